// Host side of libebag.so: argument checks, the handle and its few KB of device state, and the
// kernel launches.  Declarations and the contract of every entry point are in include/ebag.h.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "ebag.h"
#include "ebag_bwd.cuh"
#include "ebag_bwd_sorted.cuh"
#include "ebag_bwd_weights.cuh"
#include "ebag_fwd.cuh"

using namespace ebag;

namespace {

constexpr int kTableSlots = 4;   // device copies of the table-pointer array that may be in flight
constexpr int kMaxHostChunks = 16;                 // bag ranges per ebag_forward_host call
constexpr int64_t kHostChunkBytes = 64ll << 20;    // transfer size one range aims for
constexpr uint64_t kSmallCallBytesPerWarp = 16384;   // see forward_device
constexpr uint64_t kLongScratchBytes = 64ull << 20;  // partial sums of split bags, per handle
constexpr uint64_t kLongMaxParts = 8 * kMaxLongBags; // parts of split bags per launch (see forward_device)
constexpr int kAutoHostChunks = 8;                 // more ranges cost more in small copies than they hide

struct DeviceGuard {             // make the handle's device current for the duration of a call
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

bool is_rowwise8(int dtype) { return dtype == EBAG_INT8_ROWWISE || dtype == EBAG_UINT8_ROWWISE; }
int elem_bytes(int dtype) { return dtype == EBAG_F32 ? 4 : (is_rowwise8(dtype) ? 1 : 2); }

}  // namespace

struct ebag_tbe {
    int T = 0, dtype = 0, device = 0, sumD = 0, num_sms = 0;
    std::vector<int64_t> rows;
    std::vector<int32_t> D;
    TableMeta* d_meta = nullptr;
    BwdTableMeta* d_bwd_meta = nullptr;            // built by the first ebag_backward
    int32_t* d_bwd_hot = nullptr;                  // [T, kHotSlots] sampled hot rows of the current call
    int bwd_occupancy[2] = {};
    int bwd_sorted = 1;                            // 1: lookups sorted by row, summed run by run (reproducible); 0: reductions
    void* s_bwd = nullptr;                         // scratch of the sorted backward, grown with the calls
    int64_t cap_bwd = 0;
    Queue* d_queue = nullptr;
    Status* d_status = nullptr;
    // per-call pointer block [tables T][mappings T][mapping lengths T]: cached on the device,
    // re-sent only when the caller's arrays change
    const void** d_tables[kTableSlots] = {};
    const void** h_tables[kTableSlots] = {};       // pinned
    cudaEvent_t slot_event[kTableSlots] = {};
    bool slot_busy[kTableSlots] = {};
    cudaStream_t slot_stream[kTableSlots] = {};    // the stream the slot's copy was enqueued on
    int slot = -1;
    int occupancy[2][2] = {};                      // CTAs per SM, [plain, MapId][unweighted, weighted]
    unsigned width_classes = 0;                    // bit g: some table's rows are covered by 2^g lanes
    uint32_t item_bytes = 32768;
    int ctas_per_sm = 0;                           // 0: occupancy limit
    // long bags (pooled in parts by a second kernel): one device block carved into the control
    // words, the recorded bags, their arrival counters and the partial sums
    void* d_long = nullptr;
    LongParams lg = {};
    uint32_t max_stride = 0;
    int out_dtype = EBAG_F32;                      // element type of `out` (F32, F16 or BF16)
    int mapid_fused = 0;                           // ebag_forward_mapid: 1 = search inside the forward kernel
    uint32_t split_bytes = 65536;                  // a bag gathering this much or more is split; 0: never
    int64_t launches = 0;
    std::string cuda_error;
    // staging for ebag_forward_host
    int64_t* s_indices = nullptr;
    ebag::MapSlot* s_maphash = nullptr;     // hash tables of the mappings of the MapId call in flight
    int64_t cap_maphash = 0;
    uint32_t* d_map_base = nullptr;   // [T] first slot of every table's hash table (written by the build kernel)
    int64_t cap_map_base = 0;
    int mapid_hash = 1;
    int64_t* s_offsets = nullptr;
    float* s_weights = nullptr;
    float* s_out = nullptr;
    int64_t cap_indices = 0, cap_offsets = 0, cap_weights = 0, cap_out = 0;
    // ebag_forward_host pipelines copies and kernels over ranges of bags
    cudaStream_t s_h2d = nullptr, s_d2h = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaEvent_t ev_in[kMaxHostChunks] = {}, ev_done[kMaxHostChunks] = {};
    int host_chunks = 0;                           // 0: pick from the transfer size
};

namespace {

ebag_status cuda_fail(ebag_tbe* h, cudaError_t e) {
    if (h) h->cuda_error = cudaGetErrorString(e);
    cudaGetLastError();   // clear the sticky-less error state
    return EBAG_ERR_CUDA;
}

#define EBAG_CUDA(h, call)                                 \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) return cuda_fail(h, e__);  \
    } while (0)

void free_handle(ebag_tbe* h) {
    if (!h) return;
    cudaFree(h->d_meta);
    cudaFree(h->d_bwd_meta);
    cudaFree(h->d_bwd_hot);
    cudaFree(h->d_queue);
    cudaFree(h->d_status);
    cudaFree(h->d_long);
    for (int i = 0; i < kTableSlots; ++i) {
        cudaFree(h->d_tables[i]);
        if (h->h_tables[i]) cudaFreeHost(h->h_tables[i]);
        if (h->slot_event[i]) cudaEventDestroy(h->slot_event[i]);
    }
    if (h->s_h2d) cudaStreamDestroy(h->s_h2d);
    if (h->s_d2h) cudaStreamDestroy(h->s_d2h);
    if (h->ev_fork) cudaEventDestroy(h->ev_fork);
    if (h->ev_join) cudaEventDestroy(h->ev_join);
    for (int i = 0; i < kMaxHostChunks; ++i) {
        if (h->ev_in[i]) cudaEventDestroy(h->ev_in[i]);
        if (h->ev_done[i]) cudaEventDestroy(h->ev_done[i]);
    }
    cudaFree(h->s_indices);
    cudaFree(h->s_bwd);
    cudaFree(h->s_maphash);
    cudaFree(h->d_map_base);
    cudaFree(h->s_offsets);
    cudaFree(h->s_weights);
    cudaFree(h->s_out);
    delete h;
}

size_t fwd_smem_bytes(int T) { return (size_t)(2 * T + 1) * sizeof(int); }

cudaError_t launch_fwd(int dtype, const FwdParams& p, bool w, bool mapid, int grid, size_t smem,
                       cudaStream_t s) {
    switch (dtype) {
        case EBAG_F32: return launch_fwd_f32(p, w, mapid, grid, smem, s);
        case EBAG_F16: return launch_fwd_f16(p, w, mapid, grid, smem, s);
        case EBAG_BF16: return launch_fwd_bf16(p, w, mapid, grid, smem, s);
        default: return launch_fwd_int8(p, w, mapid, grid, smem, s);
    }
}

cudaError_t launch_fwdmax(int dtype, const FwdParams& p, int grid, size_t smem, cudaStream_t s) {
    switch (dtype) {
        case EBAG_F32: return launch_fwdmax_f32(p, grid, smem, s);
        case EBAG_F16: return launch_fwdmax_f16(p, grid, smem, s);
        case EBAG_BF16: return launch_fwdmax_bf16(p, grid, smem, s);
        default: return launch_fwdmax_int8(p, grid, smem, s);
    }
}

cudaError_t launch_parts(int dtype, const FwdParams& p, bool w, bool mapid, int grid, cudaStream_t s) {
    switch (dtype) {
        case EBAG_F32: return launch_parts_f32(p, w, mapid, grid, s);
        case EBAG_F16: return launch_parts_f16(p, w, mapid, grid, s);
        case EBAG_BF16: return launch_parts_bf16(p, w, mapid, grid, s);
        default: return launch_parts_int8(p, w, mapid, grid, s);
    }
}

cudaError_t occupancy_fwd(int dtype, bool w, bool mapid, size_t smem, int* n) {
    switch (dtype) {
        case EBAG_F32: return occupancy_fwd_f32(w, mapid, smem, n);
        case EBAG_F16: return occupancy_fwd_f16(w, mapid, smem, n);
        case EBAG_BF16: return occupancy_fwd_bf16(w, mapid, smem, n);
        default: return occupancy_fwd_int8(w, mapid, smem, n);
    }
}

// Checks shared by ebag_forward and ebag_forward_host (pointers may be host or device).
ebag_status check_forward_args(ebag_tbe* h, const void* const* tables, const int32_t* D,
                               const int64_t* indices, int64_t n_indices, const int64_t* offsets,
                               const float* weights, int64_t B, ebag_mode mode, float* out) {
    if (!h || !tables || !D || !offsets || B < 0 || n_indices < 0) return EBAG_ERR_INVALID_ARG;
    if (mode != EBAG_SUM && mode != EBAG_MEAN && mode != EBAG_MAX) return EBAG_ERR_INVALID_ARG;
    if (mode == EBAG_MAX && weights) return EBAG_ERR_UNSUPPORTED;
    if (n_indices > 0 && !indices) return EBAG_ERR_INVALID_ARG;
    if (B > 0 && !out) return EBAG_ERR_INVALID_ARG;
    if ((int64_t)h->T * B >= (1ll << 31)) return EBAG_ERR_UNSUPPORTED;
    for (int t = 0; t < h->T; ++t) {
        if (D[t] != h->D[t]) return EBAG_ERR_INVALID_ARG;
        if (!tables[t] && h->rows[t] > 0) return EBAG_ERR_INVALID_ARG;
        if ((uintptr_t)tables[t] & 15u) return EBAG_ERR_INVALID_ARG;
    }
    return EBAG_OK;
}

// Device copy of the caller's pointer block (tables, and for the MapId variant the mapping
// pointers and lengths); re-sent only when it changed.
ebag_status stage_tables(ebag_tbe* h, const void* const* tables, const int64_t* const* mappings,
                         const int64_t* mapping_len, cudaStream_t stream, const void* const** d_out) {
    const int T = h->T;
    const size_t bytes = (size_t)3 * T * sizeof(void*);
    std::vector<const void*> blob(3 * (size_t)T, nullptr);
    for (int t = 0; t < T; ++t) {
        blob[t] = tables[t];
        if (mappings) blob[T + t] = mappings[t];
        if (mapping_len) std::memcpy(&blob[2 * T + t], &mapping_len[t], sizeof(int64_t));
    }
    if (h->slot >= 0 && std::memcmp(h->h_tables[h->slot], blob.data(), bytes) == 0) {
        // the copy of this block was enqueued on the stream of an earlier call: a launch on
        // another stream has to be ordered behind it (a device-side wait, the host does not block)
        if (h->slot_stream[h->slot] != stream)
            EBAG_CUDA(h, cudaStreamWaitEvent(stream, h->slot_event[h->slot], 0));
        *d_out = h->d_tables[h->slot];
        return EBAG_OK;
    }
    const int s = (h->slot + 1) % kTableSlots;
    if (h->slot_busy[s]) {   // an older launch may still read this slot's staging memory
        EBAG_CUDA(h, cudaEventSynchronize(h->slot_event[s]));
        h->slot_busy[s] = false;
    }
    std::memcpy(h->h_tables[s], blob.data(), bytes);
    EBAG_CUDA(h, cudaMemcpyAsync(h->d_tables[s], h->h_tables[s], bytes, cudaMemcpyHostToDevice, stream));
    EBAG_CUDA(h, cudaEventRecord(h->slot_event[s], stream));
    h->slot_busy[s] = true;
    h->slot_stream[s] = stream;
    h->slot = s;
    *d_out = h->d_tables[s];
    return EBAG_OK;
}

// Builds the hash tables of a call's mappings in the handle's scratch when that pays (defined
// with the MapId kernels below); *used says whether it did.
ebag_status prepare_map_hash(ebag_tbe* h, const void* const* d_block, const int64_t* mapping_len,
                             int64_t n_values, cudaStream_t stream, bool* used);

// Launch on device pointers for bags [b0, b1) of every table; arguments already checked.
// offsets and out are the buffers of the WHOLE call (B bags per table).
ebag_status forward_device(ebag_tbe* h, const void* const* tables, const int64_t* indices,
                           int64_t n_indices, const int64_t* offsets, const float* weights,
                           int64_t B, int64_t b0, int64_t b1, ebag_mode mode, float* out,
                           cudaStream_t stream, const int64_t* const* mappings = nullptr,
                           const int64_t* mapping_len = nullptr, bool idx32 = false) {
    if (b1 <= b0) return EBAG_OK;
    if (((uintptr_t)out & 15u) || ((uintptr_t)indices & (idx32 ? 3u : 7u)) || ((uintptr_t)offsets & 7u) ||
        ((uintptr_t)weights & 3u))
        return EBAG_ERR_INVALID_ARG;
    const void* const* d_tables = nullptr;
    ebag_status st = stage_tables(h, tables, mappings, mapping_len, stream, &d_tables);
    if (st != EBAG_OK) return st;

    FwdParams p;
    p.tables = d_tables;
    p.meta = h->d_meta;
    p.indices = indices;
    p.offsets = offsets + b0;
    p.weights = weights;
    p.out16 = h->out_dtype == EBAG_F16 ? 1 : (h->out_dtype == EBAG_BF16 ? 2 : 0);
    // (a 16-bit `out` is addressed in elements inside the kernel; the range offset is applied here in bytes)
    p.out = reinterpret_cast<float*>(reinterpret_cast<char*>(out) +
                                     b0 * (int64_t)h->sumD * (p.out16 ? 2 : 4));
    p.queue = h->d_queue;
    p.status = h->d_status;
    p.mappings = reinterpret_cast<const int64_t* const*>(d_tables + h->T);
    p.mapping_len = reinterpret_cast<const int64_t*>(d_tables + 2 * h->T);
    p.map_slots = nullptr;
    p.map_base = nullptr;
    if (mappings) {   // fused MapId: look ids up through hash tables when the call pays for building them
        bool hashed = false;
        if ((st = prepare_map_hash(h, d_tables, mapping_len, n_indices, stream, &hashed)) != EBAG_OK) return st;
        if (hashed) {
            p.map_slots = h->s_maphash;
            p.map_base = h->d_map_base;
        }
    }
    p.n_indices = n_indices;
    p.B = b1 - b0;
    p.off_stride = B;
    p.T = h->T;
    p.sumD = h->sumD;
    p.mean = mode == EBAG_MEAN ? 1 : 0;
    p.idx32 = idx32 ? 1 : 0;
    p.code_zero = h->dtype == EBAG_UINT8_ROWWISE ? 0.0f : 128.0f;
    p.item_bytes = h->item_bytes;
    // Long bags.  The bytes this call can gather are at most n_indices * (widest row), so at most
    // that / long_bytes bags can reach long_bytes; with long_bytes = 4 * part_bytes (a power of two) and
    // part_bytes >= 2 * bound / max_parts, at most max_parts / 8 bags are recorded and they ask
    // for at most bound / part_bytes + (bags) <= 5/8 max_parts parts: both always fit, so which
    // bags are split never depends on timing.  A call too small to hold a long bag skips the
    // second launch altogether.
    p.lg = h->lg;
    const uint64_t bound = (uint64_t)n_indices * std::max<uint32_t>(h->max_stride, kLongMinRowBytes);
    if (h->split_bytes == 0 || bound < h->split_bytes) {
        p.lg.ctl = nullptr;
    } else {
        const uint64_t fit = (2 * bound + p.lg.max_parts - 1) / p.lg.max_parts;
        const uint64_t part_bytes = std::max<uint64_t>(h->split_bytes / 4, fit);
        p.lg.part_shift = 8;
        while ((1ull << p.lg.part_shift) < part_bytes) ++p.lg.part_shift;   // a power of two: no division on the device
        p.lg.long_bytes = 4ull << p.lg.part_shift;
    }
    const bool w = weights != nullptr;
    const bool mapid = mappings != nullptr;
    int per_sm = h->occupancy[mapid ? 1 : 0][w ? 1 : 0];
    if (h->ctas_per_sm > 0) {
        if (h->ctas_per_sm < per_sm) per_sm = h->ctas_per_sm;
    } else {
        // A small call is over before a full grid has even started: one resident CTA per SM for
        // every kSmallCallBytesPerWarp the call can gather per warp (workload 1: 18.9 -> 15.6 us).
        const uint64_t want = bound / ((uint64_t)h->num_sms * (kThreads / 32) * kSmallCallBytesPerWarp) + 1;
        if (want < (uint64_t)per_sm) per_sm = (int)want;
    }
    const int grid = h->num_sms * per_sm;
    if (mode == EBAG_MAX) {                        // its own kernel; bags are never split
        if (mapid) return EBAG_ERR_UNSUPPORTED;
        p.lg.ctl = nullptr;
        EBAG_CUDA(h, launch_fwdmax(h->dtype, p, grid, fwd_smem_bytes(p.T), stream));
        ++h->launches;
        return EBAG_OK;
    }
    EBAG_CUDA(h, launch_fwd(h->dtype, p, w, mapid, grid, fwd_smem_bytes(p.T), stream));
    ++h->launches;
    if (p.lg.ctl) {
        EBAG_CUDA(h, launch_parts(h->dtype, p, w, mapid, grid, stream));
        ++h->launches;
    }
    return EBAG_OK;
}

template <typename T>
ebag_status grow(ebag_tbe* h, T** buf, int64_t* cap, int64_t need) {
    if (need <= *cap) return EBAG_OK;
    EBAG_CUDA(h, cudaDeviceSynchronize());
    cudaFree(*buf);
    *buf = nullptr;
    *cap = 0;
    EBAG_CUDA(h, cudaMalloc((void**)buf, (size_t)need * sizeof(T)));
    *cap = need;
    return EBAG_OK;
}

__global__ void pack_int8_rowwise_kernel(const int8_t* __restrict__ q, const float* __restrict__ scale,
                                         const float* __restrict__ bias, int64_t rows, int D,
                                         uint4* __restrict__ dst, uint32_t flip) {
    // one thread per 16-byte vector of the packed row: D/16 vectors of codes, stored biased by
    // +128 (sign bit flipped) so that the forward kernel widens them without a sign fix-up, then
    // one vector holding scale, bias and 8 bytes of zero padding
    const int vecs = D / 16 + 1;
    const int64_t total = rows * vecs;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / vecs;
        const int v = (int)(i - r * vecs);
        uint4 x;
        if (v < vecs - 1) {
            x = *reinterpret_cast<const uint4*>(q + r * D + v * 16);
            x.x ^= flip;                  // 0x80808080 for signed codes, 0 for unsigned ones
            x.y ^= flip;
            x.z ^= flip;
            x.w ^= flip;
        } else {
            x = make_uint4(__float_as_uint(scale[r]), __float_as_uint(bias[r]), 0u, 0u);
        }
        dst[i] = x;
    }
}

// ---- MapId, stand-alone kernels.  A search is a chain of dependent loads; the first ten of its
// steps are taken in shared memory: the CTA keeps up to kPivots pivots of its mapping there,
// pivot j = the LAST entry of block j of `stride` consecutive entries.  The insertion index of v
// lies in the first block whose pivot is >= v, so a search is a halving search over the pivots
// (shared memory) followed by one over that block (global memory, log2(stride) steps instead of
// log2(|M|)); mappings of up to kPivots entries never touch global memory again.
constexpr int kPivots = 1024;

__device__ __forceinline__ void load_pivots(const int64_t* __restrict__ M, uint32_t mlen, uint32_t stride,
                                            uint32_t np, int64_t* pivots) {
    for (uint32_t j = threadIdx.x; j < np; j += blockDim.x) {
        const uint64_t last = (uint64_t)(j + 1) * stride - 1;
        pivots[j] = __ldg(M + (last < mlen ? (uint32_t)last : mlen - 1));
    }
    __syncthreads();
}

// Four searches side by side (their chains of dependent loads overlap): out[k] = MapId(v[k]).
__device__ __forceinline__ void map_id4_pivots(const int64_t* __restrict__ M, uint32_t mlen, uint32_t stride,
                                               uint32_t np, int steps1, int steps2,
                                               const int64_t* pivots, const int64_t (&v)[4], int64_t (&out)[4]) {
    if (mlen == 0) {
#pragma unroll
        for (int k = 0; k < 4; ++k) out[k] = 0;
        return;
    }
    uint32_t lo[4] = {0, 0, 0, 0}, hi[4] = {np, np, np, np};
    for (int s = 0; s < steps1; ++s) {                      // first pivot >= v, in shared memory
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t mid = (lo[k] + hi[k]) >> 1;
            const int64_t pv = pivots[mid < np ? mid : np - 1];
            const bool active = lo[k] < hi[k];
            const bool right = pv < v[k];
            lo[k] = (active && right) ? mid + 1 : lo[k];
            hi[k] = (active && !right) ? mid : hi[k];
        }
    }
    uint32_t blo[4], bhi[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {                           // that block (or past the end: v > max M)
        const uint64_t b0 = (uint64_t)lo[k] * stride, b1 = b0 + stride;
        blo[k] = b0 < mlen ? (uint32_t)b0 : mlen;
        bhi[k] = b1 < mlen ? (uint32_t)b1 : mlen;
    }
    for (int s = 0; s < steps2; ++s) {                      // first entry >= v inside the block
        int64_t mv[4];
        uint32_t mid[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            mid[k] = (blo[k] + bhi[k]) >> 1;
            mv[k] = __ldg(M + (mid[k] < mlen ? mid[k] : mlen - 1));
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool active = blo[k] < bhi[k];
            const bool right = mv[k] < v[k];
            blo[k] = (active && right) ? mid[k] + 1 : blo[k];
            bhi[k] = (active && !right) ? mid[k] : bhi[k];
        }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t idx = blo[k] < mlen ? blo[k] : mlen - 1;
        out[k] = __ldg(M + idx) == v[k] ? (int64_t)idx + 1 : 0;
    }
}

struct PivotPlan {
    uint32_t stride, np;
    int steps1, steps2;
};
__device__ __forceinline__ PivotPlan plan_pivots(uint32_t mlen) {
    PivotPlan pl;
    pl.stride = mlen ? (mlen + kPivots - 1) / kPivots : 1;
    pl.np = mlen ? (mlen + pl.stride - 1) / pl.stride : 0;
    pl.steps1 = 32 - __clz(pl.np);
    pl.steps2 = 32 - __clz(pl.stride);           // bit length: enough halvings for a block of `stride`
    if (pl.stride == 1) pl.steps2 = 1;           // one-entry blocks: a single step settles lo
    return pl;
}

// MapId of values[lo, hi): every thread runs four searches at a time, on values a block-width
// apart, so that loads and stores stay coalesced.
__device__ __forceinline__ void mapid_range(const int64_t* __restrict__ values, int64_t lo, int64_t hi,
                                            const int64_t* __restrict__ M, uint32_t mlen,
                                            int64_t* __restrict__ out, int64_t first, int64_t stride,
                                            int64_t* pivots) {
    const PivotPlan pl = plan_pivots(mlen);
    if (mlen) load_pivots(M, mlen, pl.stride, pl.np, pivots);
    const int64_t step = stride * 4;
    for (int64_t i = lo + first; i < hi; i += step) {
        int64_t v[4], r[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int64_t j = i + k * stride;
            v[k] = j < hi ? __ldcs(reinterpret_cast<const long long*>(values + j)) : 0;
        }
        map_id4_pivots(M, mlen, pl.stride, pl.np, pl.steps1, pl.steps2, pivots, v, r);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int64_t j = i + k * stride;
            if (j < hi) out[j] = r[k];
        }
    }
}

__global__ void __launch_bounds__(256)
mapid_kernel(const int64_t* __restrict__ values, int64_t n, const int64_t* __restrict__ mapping,
             uint32_t mlen, int64_t* __restrict__ out) {
    __shared__ int64_t pivots[kPivots];
    mapid_range(values, 0, n, mapping, mlen, out, blockIdx.x * (int64_t)blockDim.x + threadIdx.x,
                (int64_t)gridDim.x * blockDim.x, pivots);
}

// Prefix sums over a[0..n) in shared memory, in place, by a CTA of 256 threads: a[i] becomes
// a[0] + ... + a[i].  Every thread takes a run of consecutive entries.  Ends with a barrier.
__device__ __forceinline__ void block_scan_inclusive(uint32_t* a, int n) {
    __shared__ uint32_t warp_total[8];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int per = (n + 255) / 256;
    const int i0 = threadIdx.x * per;
    const int i1 = i0 + per < n ? i0 + per : n;
    uint32_t sum = 0;
    for (int i = i0; i < i1; ++i) sum += a[i];
    uint32_t x = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, x, d);
        if (lane >= d) x += y;
    }
    if (lane == 31) warp_total[wid] = x;
    __syncthreads();
    uint32_t run = x - sum;
    for (int w = 0; w < wid; ++w) run += warp_total[w];
    for (int i = i0; i < i1; ++i) {
        run += a[i];
        a[i] = run;
    }
    __syncthreads();
}

// MapId for all tables of a TBE call in one launch.  The tables' slices of the jagged value list
// are read from the offsets array on the device (no host synchronisation) and cut into chunks of
// kMapChunk values; every CTA takes an equal run of consecutive chunks, so the work is balanced
// whatever the tables' sizes, and reloads its pivots only when its run crosses into another table.
constexpr int kMapChunk = 16384;
constexpr int kMapMaxTables = 2048;

__global__ void __launch_bounds__(256)
mapid_tbe_kernel(const int64_t* __restrict__ values, int64_t n_values, const int64_t* __restrict__ offsets,
                 int64_t B, int T, const int64_t* const* __restrict__ mappings,
                 const int64_t* __restrict__ mapping_len, int64_t* __restrict__ out) {
    __shared__ int64_t pivots[kPivots];
    __shared__ int chunk_base[kMapMaxTables + 1];           // first chunk of every table
    for (int t = threadIdx.x; t < T; t += blockDim.x) {
        int64_t lo = offsets[(int64_t)t * B], hi = offsets[(int64_t)(t + 1) * B];
        if (lo < 0) lo = 0;
        if (hi > n_values) hi = n_values;
        chunk_base[t + 1] = hi > lo ? (int)((hi - lo + kMapChunk - 1) / kMapChunk) : 0;
    }
    if (threadIdx.x == 0) chunk_base[0] = 0;
    __syncthreads();
    block_scan_inclusive(reinterpret_cast<uint32_t*>(chunk_base), T + 1);
    const int total = chunk_base[T];
    const int per_cta = (total + gridDim.x - 1) / gridDim.x;
    const int c0 = blockIdx.x * per_cta;
    const int c1 = c0 + per_cta < total ? c0 + per_cta : total;
    int cur_t = -1;
    const int64_t* M = nullptr;
    uint32_t mlen = 0;
    PivotPlan pl = plan_pivots(0);
    for (int c = c0; c < c1; ++c) {
        int lo_t = cur_t < 0 ? 0 : cur_t, hi_t = T;          // tables come in order: search from the current one
        while (hi_t - lo_t > 1) {
            const int mid = (lo_t + hi_t) >> 1;
            if (chunk_base[mid] <= c) lo_t = mid; else hi_t = mid;
        }
        if (lo_t != cur_t) {
            cur_t = lo_t;
            M = mappings[cur_t];
            const int64_t ml = mapping_len[cur_t];
            mlen = (uint32_t)(ml < 0 ? 0 : ml);
            pl = plan_pivots(mlen);
            __syncthreads();                                 // everyone is done with the old pivots
            if (mlen) load_pivots(M, mlen, pl.stride, pl.np, pivots);
        }
        int64_t lo = offsets[(int64_t)cur_t * B], hi = offsets[(int64_t)(cur_t + 1) * B];
        if (lo < 0) lo = 0;
        if (hi > n_values) hi = n_values;
        const int64_t v0 = lo + (int64_t)(c - chunk_base[cur_t]) * kMapChunk;
        const int64_t v1 = v0 + kMapChunk < hi ? v0 + kMapChunk : hi;
        for (int64_t i = v0 + threadIdx.x; i < v1; i += 4 * blockDim.x) {
            int64_t v[4], r[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int64_t j = i + k * blockDim.x;
                v[k] = j < v1 ? __ldcs(reinterpret_cast<const long long*>(values + j)) : 0;
            }
            map_id4_pivots(M, mlen, pl.stride, pl.np, pl.steps1, pl.steps2, pivots, v, r);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int64_t j = i + k * blockDim.x;
                if (j < v1) out[j] = r[k];
            }
        }
    }
}

// ---- MapId through a hash table.  When a call has many more values than mapping entries, the
// handle first builds, per table, an open-addressing table of the mapping (16-byte slots: key,
// index + 1; linear probing; at most a quarter full) and the searches become one or two loads each
// instead of log2(|M|) dependent ones.  The result is the same as the binary search's for a
// sorted mapping: equal keys are adjacent there and only the first of a run is inserted.
// slots of every table's hash table into hbase[t + 1], hbase[0] = 0: after a prefix sum over
// the T + 1 entries hbase[t] is the first slot of table t
__device__ __forceinline__ void map_hash_sizes(int T, const int64_t* __restrict__ mapping_len, uint32_t* hbase) {
    for (int t = threadIdx.x; t < T; t += blockDim.x) {
        const int64_t ml = mapping_len[t];
        hbase[t + 1] = 1u << map_hash_bits(ml < 0 ? 0 : ml);
    }
    if (threadIdx.x == 0) hbase[0] = 0;
}

__global__ void __launch_bounds__(256)
map_hash_build_kernel(int T, const int64_t* const* __restrict__ mappings,
                      const int64_t* __restrict__ mapping_len, MapSlot* __restrict__ slots,
                      uint32_t* __restrict__ table_base) {
    __shared__ uint32_t base_s;
    const int t = blockIdx.y;
    const int64_t ml = mapping_len[t];
    if (threadIdx.x == 0) base_s = 0;
    __syncthreads();
    uint32_t part = 0;                                       // slots of the tables before this one
    for (int u = threadIdx.x; u < t; u += blockDim.x) {
        const int64_t l = mapping_len[u];
        part += 1u << map_hash_bits(l < 0 ? 0 : l);
    }
    part = __reduce_add_sync(0xffffffffu, part);
    if ((threadIdx.x & 31) == 0 && part) atomicAdd(&base_s, part);
    __syncthreads();
    if (threadIdx.x == 0 && blockIdx.x == 0) table_base[t] = base_s;   // for the forward kernel's fused look-up
    if (ml <= 0) return;
    const uint32_t bits = map_hash_bits(ml), mask = (1u << bits) - 1u;
    MapSlot* tab = slots + base_s;
    const int64_t* M = mappings[t];
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < ml; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t key = M[i];
        if (i > 0 && M[i - 1] == key) continue;              // only the first of a run of equal keys
        uint32_t s = (uint32_t)(((uint64_t)key * kHashMul) >> (64 - bits));
        for (uint32_t probe = 0; probe <= mask; ++probe) {   // at most a quarter full: ends early
            if (atomicCAS(&tab[s].idx1, 0u, (uint32_t)i + 1u) == 0u) {
                tab[s].key = key;
                break;
            }
            s = (s + 1) & mask;
        }
    }
}

// four look-ups side by side
__device__ __forceinline__ void map_hash_lookup4(const MapSlot* __restrict__ tab, uint32_t bits,
                                                 const int64_t (&v)[4], int64_t (&out)[4]) {
    const uint32_t mask = (1u << bits) - 1u;
    uint32_t s[4];
    bool open[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        s[k] = (uint32_t)(((uint64_t)v[k] * kHashMul) >> (64 - bits));
        open[k] = true;
        out[k] = 0;
    }
    for (uint32_t probe = 0; probe <= mask; ++probe) {
        int4 q[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
            q[k] = open[k] ? __ldg(reinterpret_cast<const int4*>(tab + s[k])) : make_int4(0, 0, 0, 0);
        bool any = false;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int64_t key = (int64_t)(((uint64_t)(uint32_t)q[k].y << 32) | (uint32_t)q[k].x);
            const bool hit = q[k].z != 0 && key == v[k];
            if (open[k] && hit) out[k] = (int64_t)(uint32_t)q[k].z;
            open[k] = open[k] && q[k].z != 0 && !hit;        // an empty slot ends the search: not mapped
            s[k] = (s[k] + 1) & mask;
            any = any || open[k];
        }
        if (!any) break;
    }
}

__global__ void __launch_bounds__(256)
mapid_tbe_hash_kernel(const int64_t* __restrict__ values, int64_t n_values, const int64_t* __restrict__ offsets,
                      int64_t B, int T, const int64_t* __restrict__ mapping_len,
                      const MapSlot* __restrict__ slots, int64_t* __restrict__ out) {
    __shared__ int chunk_base[kMapMaxTables + 1];           // first chunk of every table
    __shared__ uint32_t hbase[kMapMaxTables + 1];
    for (int t = threadIdx.x; t < T; t += blockDim.x) {
        int64_t lo = offsets[(int64_t)t * B], hi = offsets[(int64_t)(t + 1) * B];
        if (lo < 0) lo = 0;
        if (hi > n_values) hi = n_values;
        chunk_base[t + 1] = hi > lo ? (int)((hi - lo + kMapChunk - 1) / kMapChunk) : 0;
    }
    map_hash_sizes(T, mapping_len, hbase);
    if (threadIdx.x == 0) chunk_base[0] = 0;
    __syncthreads();
    block_scan_inclusive(reinterpret_cast<uint32_t*>(chunk_base), T + 1);
    block_scan_inclusive(hbase, T + 1);
    const int total = chunk_base[T];
    const int per_cta = (total + gridDim.x - 1) / gridDim.x;
    const int c0 = blockIdx.x * per_cta;
    const int c1 = c0 + per_cta < total ? c0 + per_cta : total;
    int cur_t = 0;
    for (int c = c0; c < c1; ++c) {
        int hi_t = T;                                        // tables come in order: search from the current one
        while (hi_t - cur_t > 1) {
            const int mid = (cur_t + hi_t) >> 1;
            if (chunk_base[mid] <= c) cur_t = mid; else hi_t = mid;
        }
        const int64_t ml = mapping_len[cur_t];
        const uint32_t bits = map_hash_bits(ml < 0 ? 0 : ml);
        const MapSlot* tab = slots + hbase[cur_t];
        int64_t lo = offsets[(int64_t)cur_t * B], hi = offsets[(int64_t)(cur_t + 1) * B];
        if (lo < 0) lo = 0;
        if (hi > n_values) hi = n_values;
        const int64_t v0 = lo + (int64_t)(c - chunk_base[cur_t]) * kMapChunk;
        const int64_t v1 = v0 + kMapChunk < hi ? v0 + kMapChunk : hi;
        for (int64_t i = v0 + threadIdx.x; i < v1; i += 4 * blockDim.x) {
            int64_t v[4], r[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int64_t j = i + k * blockDim.x;
                v[k] = j < v1 ? __ldcs(reinterpret_cast<const long long*>(values + j)) : 0;
            }
            map_hash_lookup4(tab, bits, v, r);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int64_t j = i + k * blockDim.x;
                if (j < v1) __stcs(reinterpret_cast<long long*>(out + j), r[k]);
            }
        }
    }
}

// With many more values than mapping entries a hash table of the mappings pays for itself.
ebag_status prepare_map_hash(ebag_tbe* h, const void* const* d_block, const int64_t* mapping_len,
                             int64_t n_values, cudaStream_t stream, bool* used) {
    *used = false;
    int64_t hash_slots = 0, max_len = 0;
    for (int t = 0; t < h->T; ++t) {
        hash_slots += 1ll << map_hash_bits(mapping_len[t]);
        if (mapping_len[t] > max_len) max_len = mapping_len[t];
    }
    if (!h->mapid_hash || hash_slots > kMapHashMaxSlots || n_values < hash_slots || max_len <= 0) return EBAG_OK;
    ebag_status st;
    if ((st = grow(h, &h->s_maphash, &h->cap_maphash, hash_slots)) != EBAG_OK) return st;
    if ((st = grow(h, &h->d_map_base, &h->cap_map_base, (int64_t)h->T)) != EBAG_OK) return st;
    EBAG_CUDA(h, cudaMemsetAsync(h->s_maphash, 0, (size_t)hash_slots * sizeof(MapSlot), stream));
    int64_t gx = (max_len + 255) / 256;
    if (gx > 64) gx = 64;
    map_hash_build_kernel<<<dim3((unsigned)gx, (unsigned)h->T), 256, 0, stream>>>(
        h->T, reinterpret_cast<const int64_t* const*>(d_block + h->T),
        reinterpret_cast<const int64_t*>(d_block + 2 * h->T), h->s_maphash, h->d_map_base);
    EBAG_CUDA(h, cudaGetLastError());
    ++h->launches;
    *used = true;
    return EBAG_OK;
}

}  // namespace

extern "C" {

ebag_status ebag_mapid_tbe(ebag_tbe* h, const int64_t* values, int64_t n_values,
                           const int64_t* offsets, const int64_t* const* mappings,
                           const int64_t* mapping_len, int64_t B, int64_t* out, ebag_stream stream) {
    if (!h || !offsets || !mappings || !mapping_len || B < 0 || n_values < 0) return EBAG_ERR_INVALID_ARG;
    if (n_values > 0 && (!values || !out)) return EBAG_ERR_INVALID_ARG;
    if ((int64_t)h->T * B >= (1ll << 31) || h->T > kMapMaxTables) return EBAG_ERR_UNSUPPORTED;
    if (n_values / kMapChunk + h->T >= (1ll << 31)) return EBAG_ERR_UNSUPPORTED;
    for (int t = 0; t < h->T; ++t) {
        if (mapping_len[t] < 0 || mapping_len[t] >= (1ll << 31)) return EBAG_ERR_INVALID_ARG;
        if (mapping_len[t] > 0 && (!mappings[t] || ((uintptr_t)mappings[t] & 7u))) return EBAG_ERR_INVALID_ARG;
    }
    if (B == 0 || n_values == 0) return EBAG_OK;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EBAG_ERR_CUDA;
    // the pointer block carries the mappings; the table slots of the block are left empty
    std::vector<const void*> no_tables(h->T, nullptr);
    const void* const* d_block = nullptr;
    ebag_status st = stage_tables(h, no_tables.data(), mappings, mapping_len, (cudaStream_t)stream, &d_block);
    if (st != EBAG_OK) return st;
    // enough CTAs to fill the device a few times over, never more than there are chunks
    int64_t bx = n_values / kMapChunk + h->T;
    const int64_t cap = (int64_t)h->num_sms * 8;
    if (bx > cap) bx = cap;
    if (bx < 1) bx = 1;
    bool hashed = false;
    if ((st = prepare_map_hash(h, d_block, mapping_len, n_values, (cudaStream_t)stream, &hashed)) != EBAG_OK) return st;
    if (hashed) {
        mapid_tbe_hash_kernel<<<(unsigned)bx, 256, 0, (cudaStream_t)stream>>>(
            values, n_values, offsets, B, h->T, reinterpret_cast<const int64_t*>(d_block + 2 * h->T),
            h->s_maphash, out);
        EBAG_CUDA(h, cudaGetLastError());
        ++h->launches;
        return EBAG_OK;
    }
    mapid_tbe_kernel<<<(unsigned)bx, 256, 0, (cudaStream_t)stream>>>(
        values, n_values, offsets, B, h->T, reinterpret_cast<const int64_t* const*>(d_block + h->T),
        reinterpret_cast<const int64_t*>(d_block + 2 * h->T), out);
    EBAG_CUDA(h, cudaGetLastError());
    ++h->launches;
    return EBAG_OK;
}

ebag_status ebag_mapid(const int64_t* values, int64_t n, const int64_t* mapping, int64_t m,
                       int64_t* out, ebag_stream stream) {
    if (n < 0 || m < 0 || m >= (1ll << 31)) return EBAG_ERR_INVALID_ARG;
    if (n == 0) return EBAG_OK;
    if (!values || !out || (m > 0 && !mapping)) return EBAG_ERR_INVALID_ARG;
    int64_t blocks = (n + 1023) / 1024;              // four values per thread and step
    if (blocks > 148 * 8) blocks = 148 * 8;
    if (blocks < 1) blocks = 1;
    mapid_kernel<<<(int)blocks, 256, 0, (cudaStream_t)stream>>>(values, n, mapping, (uint32_t)m, out);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    return EBAG_OK;
}

ebag_status ebag_forward_mapid(ebag_tbe* h, const void* const* tables, const int32_t* D,
                               const int64_t* values, int64_t n_values, const int64_t* offsets,
                               const float* per_sample_weights, const int64_t* const* mappings,
                               const int64_t* mapping_len, int64_t B, ebag_mode mode, float* out,
                               ebag_stream stream) {
    ebag_status st = check_forward_args(h, tables, D, values, n_values, offsets, per_sample_weights,
                                        B, mode, out);
    if (st != EBAG_OK) return st;
    if (!mappings || !mapping_len) return EBAG_ERR_INVALID_ARG;
    for (int t = 0; t < h->T; ++t) {
        if (mapping_len[t] < 0 || mapping_len[t] >= (1ll << 31)) return EBAG_ERR_INVALID_ARG;
        if (mapping_len[t] > 0 && (!mappings[t] || ((uintptr_t)mappings[t] & 7u))) return EBAG_ERR_INVALID_ARG;
    }
    DeviceGuard guard(h->device);
    if (!guard.ok) return EBAG_ERR_CUDA;
    if (h->mapid_fused)
        return forward_device(h, tables, values, n_values, offsets, per_sample_weights, B, 0, B, mode,
                              out, (cudaStream_t)stream, mappings, mapping_len);
    // Default: the transform for all tables in one launch into a scratch buffer of ids that the
    // handle keeps (grown when a larger call arrives), then the plain forward.  The searches are
    // chains of dependent loads; run between the stages of the forward's row pipeline they stall
    // it, and the separate launches together are faster (2.34 against 3.82 ms on bench workload 6).
    if (B == 0) return EBAG_OK;
    if ((st = grow(h, &h->s_indices, &h->cap_indices, n_values > 0 ? n_values : 1)) != EBAG_OK) return st;
    if (n_values > 0) {
        st = ebag_mapid_tbe(h, values, n_values, offsets, mappings, mapping_len, B, h->s_indices, stream);
        if (st != EBAG_OK) return st;
    }
    return forward_device(h, tables, h->s_indices, n_values, offsets, per_sample_weights, B, 0, B, mode,
                          out, (cudaStream_t)stream);
}

int64_t ebag_row_stride(ebag_dtype dtype, int32_t D) {
    if (D <= 0 || dtype < EBAG_F32 || dtype > EBAG_UINT8_ROWWISE) return -1;
    const int64_t payload = (int64_t)D * elem_bytes(dtype);
    if (payload % 16 != 0) return -1;
    return (dtype == EBAG_INT8_ROWWISE || dtype == EBAG_UINT8_ROWWISE) ? payload + 16 : payload;
}

ebag_status ebag_create_tbe(int32_t T, const int64_t* rows, const int32_t* D, ebag_dtype dtype,
                            int device, ebag_tbe** out) {
    if (!out) return EBAG_ERR_INVALID_ARG;
    *out = nullptr;
    if (T <= 0 || !rows || !D || dtype < EBAG_F32 || dtype > EBAG_UINT8_ROWWISE)
        return EBAG_ERR_INVALID_ARG;
    if (T > EBAG_MAX_TABLES) return EBAG_ERR_UNSUPPORTED;
    std::vector<TableMeta> meta(T);
    int64_t d_off = 0;
    unsigned width_classes = 0;
    for (int t = 0; t < T; ++t) {
        const int64_t stride = ebag_row_stride(dtype, D[t]);
        if (stride < 0 || rows[t] < 0) return EBAG_ERR_INVALID_ARG;
        if (rows[t] >= (1ll << 31) || stride >= (1ll << 31)) return EBAG_ERR_UNSUPPORTED;
        TableMeta& m = meta[t];
        m.rows = rows[t];
        m.D = D[t];
        m.D_off = (int32_t)d_off;
        m.stride = (int32_t)stride;
        m.nvec = (int32_t)((int64_t)D[t] * elem_bytes(dtype) / 16);
        int g_log2 = 2;
        while ((1 << g_log2) < m.nvec && g_log2 < 5) ++g_log2;
        m.g_log2 = g_log2;
        width_classes |= 1u << g_log2;
        m.V = m.nvec <= 32 ? 1 : 2;
        d_off += D[t];
        if (d_off >= (1ll << 31)) return EBAG_ERR_UNSUPPORTED;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) {
        cudaGetLastError();
        return EBAG_ERR_CUDA;
    }
    DeviceGuard guard(device);
    if (!guard.ok) return EBAG_ERR_CUDA;
    ebag_tbe* h = new (std::nothrow) ebag_tbe;
    if (!h) return EBAG_ERR_INVALID_ARG;
    h->T = T;
    h->dtype = dtype;
    h->device = device;
    h->sumD = (int)d_off;
    h->width_classes = width_classes;
    h->rows.assign(rows, rows + T);
    h->D.assign(D, D + T);
    ebag_status st = EBAG_OK;
    auto body = [&]() -> ebag_status {
        cudaDeviceProp prop;
        EBAG_CUDA(h, cudaGetDeviceProperties(&prop, device));
        h->num_sms = prop.multiProcessorCount;
        EBAG_CUDA(h, cudaMalloc((void**)&h->d_meta, sizeof(TableMeta) * T));
        EBAG_CUDA(h, cudaMemcpy(h->d_meta, meta.data(), sizeof(TableMeta) * T, cudaMemcpyHostToDevice));
        EBAG_CUDA(h, cudaMalloc((void**)&h->d_queue, sizeof(Queue)));
        EBAG_CUDA(h, cudaMemset(h->d_queue, 0, sizeof(Queue)));
        EBAG_CUDA(h, cudaMalloc((void**)&h->d_status, sizeof(Status)));
        EBAG_CUDA(h, cudaMemset(h->d_status, 0, sizeof(Status)));
        {
            // one slot of partial sums holds a row per bag that a warp pools side by side
            uint32_t slot = 4;
            for (int t = 0; t < T; ++t) {
                slot = std::max<uint32_t>(slot, (uint32_t)(32 >> meta[t].g_log2) * (uint32_t)meta[t].D);
                h->max_stride = std::max<uint32_t>(h->max_stride, (uint32_t)meta[t].stride);
            }
            uint64_t parts = kLongScratchBytes / ((uint64_t)slot * sizeof(float));
            parts = std::min<uint64_t>(std::max<uint64_t>(parts, kMaxLongBags), kLongMaxParts);
            auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
            const size_t o_bags = up(sizeof(LongCtl));
            const size_t o_arr = o_bags + up(sizeof(LongBag) * kMaxLongBags);
            const size_t o_part = o_arr + up(sizeof(unsigned) * kMaxLongBags);
            const size_t total = o_part + (size_t)parts * slot * sizeof(float);
            EBAG_CUDA(h, cudaMalloc(&h->d_long, total));
            EBAG_CUDA(h, cudaMemset(h->d_long, 0, o_part));
            char* base = static_cast<char*>(h->d_long);
            h->lg.ctl = reinterpret_cast<LongCtl*>(base);
            h->lg.bags = reinterpret_cast<LongBag*>(base + o_bags);
            h->lg.arrivals = reinterpret_cast<unsigned*>(base + o_arr);
            h->lg.partial = reinterpret_cast<float*>(base + o_part);
            h->lg.slot_floats = slot;
            h->lg.max_parts = (uint32_t)parts;
        }
        for (int i = 0; i < kTableSlots; ++i) {
            EBAG_CUDA(h, cudaMalloc((void**)&h->d_tables[i], sizeof(void*) * 3 * T));
            EBAG_CUDA(h, cudaMallocHost((void**)&h->h_tables[i], sizeof(void*) * 3 * T));
            EBAG_CUDA(h, cudaEventCreateWithFlags(&h->slot_event[i], cudaEventDisableTiming));
        }
        EBAG_CUDA(h, cudaStreamCreateWithFlags(&h->s_h2d, cudaStreamNonBlocking));
        EBAG_CUDA(h, cudaStreamCreateWithFlags(&h->s_d2h, cudaStreamNonBlocking));
        EBAG_CUDA(h, cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming));
        EBAG_CUDA(h, cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming));
        for (int i = 0; i < kMaxHostChunks; ++i) {
            EBAG_CUDA(h, cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming));
            EBAG_CUDA(h, cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming));
        }
        for (int mp = 0; mp < 2; ++mp)
            for (int w = 0; w < 2; ++w) {
                EBAG_CUDA(h, occupancy_fwd(dtype, w != 0, mp != 0, fwd_smem_bytes(T), &h->occupancy[mp][w]));
                if (h->occupancy[mp][w] < 1) h->occupancy[mp][w] = 1;
            }
        return EBAG_OK;
    };
    st = body();
    if (st != EBAG_OK) {
        free_handle(h);
        return st;
    }
    *out = h;
    return EBAG_OK;
}

ebag_status ebag_forward(ebag_tbe* h, const void* const* tables, const int32_t* D,
                         const int64_t* indices, int64_t n_indices, const int64_t* offsets,
                         const float* per_sample_weights, int64_t B, ebag_mode mode, float* out,
                         ebag_stream stream) {
    ebag_status st = check_forward_args(h, tables, D, indices, n_indices, offsets,
                                        per_sample_weights, B, mode, out);
    if (st != EBAG_OK) return st;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EBAG_ERR_CUDA;
    return forward_device(h, tables, indices, n_indices, offsets, per_sample_weights, B, 0, B, mode,
                          out, (cudaStream_t)stream);
}

ebag_status ebag_forward_i32(ebag_tbe* h, const void* const* tables, const int32_t* D,
                             const int32_t* indices, int64_t n_indices, const int64_t* offsets,
                             const float* per_sample_weights, int64_t B, ebag_mode mode, float* out,
                             ebag_stream stream) {
    const int64_t* ids = reinterpret_cast<const int64_t*>(indices);   // width travels in idx32
    ebag_status st = check_forward_args(h, tables, D, ids, n_indices, offsets, per_sample_weights, B,
                                        mode, out);
    if (st != EBAG_OK) return st;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EBAG_ERR_CUDA;
    return forward_device(h, tables, ids, n_indices, offsets, per_sample_weights, B, 0, B, mode, out,
                          (cudaStream_t)stream, nullptr, nullptr, true);
}

ebag_status ebag_backward(ebag_tbe* h, const float* grad_out, const void* indices, int32_t index_bits,
                          int64_t n_indices, const int64_t* offsets, const float* per_sample_weights,
                          int64_t B, ebag_mode mode, float* const* grad_tables, ebag_stream stream) {
    if (!h || !offsets || !grad_tables || B < 0 || n_indices < 0) return EBAG_ERR_INVALID_ARG;
    if (index_bits != 32 && index_bits != 64) return EBAG_ERR_INVALID_ARG;
    if (mode != EBAG_SUM && mode != EBAG_MEAN) return EBAG_ERR_INVALID_ARG;
    if (n_indices > 0 && !indices) return EBAG_ERR_INVALID_ARG;
    if (B > 0 && !grad_out) return EBAG_ERR_INVALID_ARG;
    if ((int64_t)h->T * B >= (1ll << 31)) return EBAG_ERR_UNSUPPORTED;
    if (((uintptr_t)grad_out & 15u) || ((uintptr_t)indices & (index_bits == 32 ? 3u : 7u)) ||
        ((uintptr_t)offsets & 7u) || ((uintptr_t)per_sample_weights & 3u))
        return EBAG_ERR_INVALID_ARG;
    for (int t = 0; t < h->T; ++t) {
        if (h->D[t] % 4 != 0) return EBAG_ERR_UNSUPPORTED;          // fp32 gradient rows in 16-byte vectors
        if (!grad_tables[t] && h->rows[t] > 0) return EBAG_ERR_INVALID_ARG;
        if ((uintptr_t)grad_tables[t] & 15u) return EBAG_ERR_INVALID_ARG;
    }
    // (no ids is not the same as nothing to do: offsets that reach past an empty id list are
    // malformed bags, and the kernel counts them as the forward does)
    if (B == 0) return EBAG_OK;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EBAG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (!h->d_bwd_meta) {                       // first call: per-table metadata and launch geometry
        std::vector<BwdTableMeta> meta(h->T);
        int32_t d_off = 0;
        for (int t = 0; t < h->T; ++t) {
            BwdTableMeta& m = meta[t];
            m.rows = h->rows[t];
            m.D = h->D[t];
            m.D_off = d_off;
            m.nvec = h->D[t] / 4;
            int g = 0;
            while ((1 << g) < m.nvec && g < 5) ++g;
            m.g_log2 = g;
            d_off += h->D[t];
        }
        EBAG_CUDA(h, cudaMalloc((void**)&h->d_bwd_meta, sizeof(BwdTableMeta) * h->T));
        EBAG_CUDA(h, cudaMemcpy(h->d_bwd_meta, meta.data(), sizeof(BwdTableMeta) * h->T,
                                cudaMemcpyHostToDevice));
        EBAG_CUDA(h, cudaMalloc((void**)&h->d_bwd_hot, sizeof(int32_t) * kHotSlots * h->T));
        for (int w = 0; w < 2; ++w) {
            EBAG_CUDA(h, occupancy_bwd(w != 0, h->T, &h->bwd_occupancy[w]));
            if (h->bwd_occupancy[w] < 1) h->bwd_occupancy[w] = 1;
        }
    }
    const void* const* d_ptrs = nullptr;
    ebag_status st = stage_tables(h, reinterpret_cast<const void* const*>(grad_tables), nullptr, nullptr,
                                  s, &d_ptrs);
    if (st != EBAG_OK) return st;
    BwdParams p;
    p.grad_tables = reinterpret_cast<float* const*>(const_cast<void* const*>(d_ptrs));
    p.meta = h->d_bwd_meta;
    p.indices = indices;
    p.offsets = offsets;
    p.weights = per_sample_weights;
    p.grad_out = grad_out;
    p.status = h->d_status;
    p.n_indices = n_indices;
    p.B = B;
    p.T = h->T;
    p.sumD = h->sumD;
    p.mean = mode == EBAG_MEAN ? 1 : 0;
    p.idx32 = index_bits == 32 ? 1 : 0;
    p.hot = h->d_bwd_hot;
    p.use_cache = 1;
    p.only_if = nullptr;
    const bool w = per_sample_weights != nullptr;
    // The reproducible path: lookups sorted by row, every run of equal rows added up in the order
    // of the lookups and written once.  It needs offsets that do not decrease (checked on the
    // device: if they do, its kernels return at once and the reduction kernel below runs instead).
    int64_t max_rows = 1;
    int max_d = 4;
    for (int t = 0; t < h->T; ++t) {
        max_rows = std::max<int64_t>(max_rows, h->rows[t]);
        max_d = std::max<int>(max_d, h->D[t]);
    }
    if (h->bwd_sorted && n_indices > 0 && n_indices < (1ll << 32) && max_d <= kSortedMaxD) {
        const bool scaled = w || mode == EBAG_MEAN;
        const size_t need = bwd_sorted_scratch_bytes(n_indices, h->T, max_d, scaled);
        char* scratch = static_cast<char*>(h->s_bwd);
        const bool have_scratch = grow(h, &scratch, &h->cap_bwd, (int64_t)need) == EBAG_OK;
        h->s_bwd = scratch;
        if (!have_scratch) {             // no room for the sorted lists: the reduction kernel needs none
            h->cuda_error.clear();
            cudaGetLastError();
        }
        BwdSortedParams q;
        q.grad_tables = p.grad_tables;
        q.meta = p.meta;
        q.indices = indices;
        q.offsets = offsets;
        q.weights = per_sample_weights;
        q.grad_out = grad_out;
        q.status = h->d_status;
        q.n_indices = n_indices;
        q.B = B;
        q.T = h->T;
        q.sumD = h->sumD;
        q.mean = p.mean;
        q.idx32 = p.idx32;
        if (have_scratch) bwd_sorted_carve(q, h->s_bwd, n_indices, h->T, max_d, scaled);
        int bits = 1;
        while (bits < 32 && (1ll << bits) <= max_rows) ++bits;       // the key of a skipped id is rows[t] itself
        q.passes = (bits + 7) / 8;
        if (have_scratch) {
            int launches = 0;
            EBAG_CUDA(h, launch_bwd_sorted(q, h->num_sms, s, &launches));
            h->launches += launches;
            p.only_if = q.ctl;
        }
    }
    const int grid = h->num_sms * h->bwd_occupancy[w ? 1 : 0];
    EBAG_CUDA(h, launch_bwd(p, w, grid, s));
    h->launches += 2;                           // the hot-row sampler, then the backward kernel
    return EBAG_OK;
}

namespace {
// ebag_forward_host and ebag_forward_host_i32: `indices` holds 8-byte ids, or 4-byte ids when
// idx32; `out` holds elements of the handle's out_dtype.
ebag_status forward_host(ebag_tbe* h, const void* const* tables, const int32_t* D,
                         const int64_t* indices, int64_t n_indices, const int64_t* offsets,
                         const float* per_sample_weights, int64_t B, ebag_mode mode,
                         float* out, ebag_stream stream, bool idx32) {
    ebag_status st = check_forward_args(h, tables, D, indices, n_indices, offsets,
                                        per_sample_weights, B, mode, out);
    if (st != EBAG_OK) return st;
    if (B == 0) return EBAG_OK;
    const size_t isz = idx32 ? sizeof(int32_t) : sizeof(int64_t);      // bytes per id
    const size_t osz = h->out_dtype == EBAG_F32 ? 4 : 2;               // bytes per output element
    const char* idx_b = reinterpret_cast<const char*>(indices);
    char* out_b = reinterpret_cast<char*>(out);
    DeviceGuard guard(h->device);
    if (!guard.ok) return EBAG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t n_off = (int64_t)h->T * B + 1;
    const int64_t n_out = B * (int64_t)h->sumD;
    if ((st = grow(h, &h->s_indices, &h->cap_indices, n_indices > 0 ? n_indices : 1)) != EBAG_OK) return st;
    if ((st = grow(h, &h->s_offsets, &h->cap_offsets, n_off)) != EBAG_OK) return st;
    if (per_sample_weights &&
        (st = grow(h, &h->s_weights, &h->cap_weights, n_indices > 0 ? n_indices : 1)) != EBAG_OK)
        return st;
    if ((st = grow(h, &h->s_out, &h->cap_out, n_out)) != EBAG_OK) return st;
    // How many bag ranges: enough for copies and kernels to overlap, few enough that a range
    // still moves tens of MB.  The ranges need sane offsets at their borders (read here, on the
    // host); otherwise everything goes in one piece and the device sorts it out.
    const int64_t bytes = (int64_t)isz * n_indices + sizeof(int64_t) * n_off + (int64_t)osz * n_out +
                          (per_sample_weights ? sizeof(float) * n_indices : 0);
    // (Pieces that start small, so that the result starts travelling back sooner, and shrink again
    // towards the end were measured: 28.1 ms against 27.1 ms on the 32-table benchmark call.  A
    // piece costs one copy per table on the way in, and small copies waste the link.  Halving only
    // the first and the last piece, or quartering only the first: 27.1 and 27.4 ms, no gain.)
    int64_t cut[kMaxHostChunks + 1];
    int64_t chunks = h->host_chunks;
    if (chunks <= 0) {
        chunks = bytes / kHostChunkBytes;
        if (chunks > kAutoHostChunks) chunks = kAutoHostChunks;
    }
    if (chunks > kMaxHostChunks) chunks = kMaxHostChunks;
    if (chunks > B) chunks = B;
    if (chunks < 1) chunks = 1;
    for (int64_t c = 0; c <= chunks; ++c) cut[c] = c * B / chunks;
    if (chunks > 1) {                      // a full scan costs far less than the copies it guards
        int64_t prev = 0;
        for (int64_t i = 0; i < n_off && chunks > 1; ++i) {
            const int64_t v = offsets[i];
            if (v < prev || v > n_indices) chunks = 1;
            prev = v;
        }
    }
    if (chunks == 1) {
        if (n_indices > 0)
            EBAG_CUDA(h, cudaMemcpyAsync(h->s_indices, indices, isz * n_indices, cudaMemcpyHostToDevice, s));
        EBAG_CUDA(h, cudaMemcpyAsync(h->s_offsets, offsets, sizeof(int64_t) * n_off, cudaMemcpyHostToDevice, s));
        if (per_sample_weights && n_indices > 0)
            EBAG_CUDA(h, cudaMemcpyAsync(h->s_weights, per_sample_weights, sizeof(float) * n_indices, cudaMemcpyHostToDevice, s));
        st = forward_device(h, tables, h->s_indices, n_indices, h->s_offsets,
                            per_sample_weights ? h->s_weights : nullptr, B, 0, B, mode, h->s_out, s, nullptr,
                            nullptr, idx32);
        if (st != EBAG_OK) return st;
        EBAG_CUDA(h, cudaMemcpyAsync(out, h->s_out, osz * n_out, cudaMemcpyDeviceToHost, s));
        return EBAG_OK;
    }
    // Pipeline: inputs of piece k+1 travel while the kernel works on piece k and the result of
    // piece k-1 travels back.  Kernels stay on the caller's stream.
    EBAG_CUDA(h, cudaEventRecord(h->ev_fork, s));
    EBAG_CUDA(h, cudaStreamWaitEvent(h->s_h2d, h->ev_fork, 0));
    EBAG_CUDA(h, cudaStreamWaitEvent(h->s_d2h, h->ev_fork, 0));
    // all offsets first, in one copy (every piece's item sizing reads the table boundaries)
    EBAG_CUDA(h, cudaMemcpyAsync(h->s_offsets, offsets, sizeof(int64_t) * n_off, cudaMemcpyHostToDevice, h->s_h2d));
    // pieces are ranges of bags: per table one block of ids (and weights) in, one block of rows out
    for (int64_t c = 0; c < chunks; ++c) {
        const int64_t b0 = cut[c], b1 = cut[c + 1];
        for (int t = 0; t < h->T; ++t) {
            const int64_t g = (int64_t)t * B;
            const int64_t lo = offsets[g + b0], hi = offsets[g + b1];
            if (hi > lo) {
                EBAG_CUDA(h, cudaMemcpyAsync(reinterpret_cast<char*>(h->s_indices) + isz * lo, idx_b + isz * lo,
                                             isz * (hi - lo), cudaMemcpyHostToDevice, h->s_h2d));
                if (per_sample_weights)
                    EBAG_CUDA(h, cudaMemcpyAsync(h->s_weights + lo, per_sample_weights + lo,
                                                 sizeof(float) * (hi - lo), cudaMemcpyHostToDevice, h->s_h2d));
            }
        }
        EBAG_CUDA(h, cudaEventRecord(h->ev_in[c], h->s_h2d));
        EBAG_CUDA(h, cudaStreamWaitEvent(s, h->ev_in[c], 0));
        st = forward_device(h, tables, h->s_indices, n_indices, h->s_offsets,
                            per_sample_weights ? h->s_weights : nullptr, B, b0, b1, mode, h->s_out, s, nullptr,
                            nullptr, idx32);
        if (st != EBAG_OK) return st;
        EBAG_CUDA(h, cudaEventRecord(h->ev_done[c], s));
        EBAG_CUDA(h, cudaStreamWaitEvent(h->s_d2h, h->ev_done[c], 0));
        EBAG_CUDA(h, cudaMemcpyAsync(out_b + osz * b0 * h->sumD, reinterpret_cast<char*>(h->s_out) + osz * b0 * h->sumD,
                                     osz * (b1 - b0) * h->sumD, cudaMemcpyDeviceToHost, h->s_d2h));
    }
    EBAG_CUDA(h, cudaEventRecord(h->ev_join, h->s_d2h));
    EBAG_CUDA(h, cudaStreamWaitEvent(s, h->ev_join, 0));
    return EBAG_OK;
}
}  // namespace

ebag_status ebag_forward_host(ebag_tbe* h, const void* const* tables, const int32_t* D,
                              const int64_t* indices, int64_t n_indices, const int64_t* offsets,
                              const float* per_sample_weights, int64_t B, ebag_mode mode,
                              float* out, ebag_stream stream) {
    return forward_host(h, tables, D, indices, n_indices, offsets, per_sample_weights, B, mode, out, stream,
                        false);
}

ebag_status ebag_forward_host_i32(ebag_tbe* h, const void* const* tables, const int32_t* D,
                                  const int32_t* indices, int64_t n_indices, const int64_t* offsets,
                                  const float* per_sample_weights, int64_t B, ebag_mode mode,
                                  float* out, ebag_stream stream) {
    return forward_host(h, tables, D, reinterpret_cast<const int64_t*>(indices), n_indices, offsets,
                        per_sample_weights, B, mode, out, stream, true);
}

ebag_status ebag_backward_weights(ebag_tbe* h, const void* const* tables, const int32_t* D,
                                  const float* grad_out, const void* indices, int32_t index_bits,
                                  int64_t n_indices, const int64_t* offsets, int64_t B, ebag_mode mode,
                                  float* grad_weights, ebag_stream stream) {
    if (!h || !tables || !D || !offsets || B < 0 || n_indices < 0) return EBAG_ERR_INVALID_ARG;
    if (index_bits != 32 && index_bits != 64) return EBAG_ERR_INVALID_ARG;
    if (mode != EBAG_SUM && mode != EBAG_MEAN) return EBAG_ERR_INVALID_ARG;
    if (n_indices > 0 && (!indices || !grad_weights)) return EBAG_ERR_INVALID_ARG;
    if (B > 0 && !grad_out) return EBAG_ERR_INVALID_ARG;
    if ((int64_t)h->T * B >= (1ll << 31)) return EBAG_ERR_UNSUPPORTED;
    if (((uintptr_t)grad_out & 15u) || ((uintptr_t)indices & (index_bits == 32 ? 3u : 7u)) ||
        ((uintptr_t)offsets & 7u) || ((uintptr_t)grad_weights & 3u))
        return EBAG_ERR_INVALID_ARG;
    for (int t = 0; t < h->T; ++t) {
        if (D[t] != h->D[t]) return EBAG_ERR_INVALID_ARG;
        if (h->D[t] % 4 != 0) return EBAG_ERR_UNSUPPORTED;          // grad_out slices in 16-byte vectors
        if (!tables[t] && h->rows[t] > 0) return EBAG_ERR_INVALID_ARG;
        if ((uintptr_t)tables[t] & 15u) return EBAG_ERR_INVALID_ARG;
    }
    if (B == 0) return EBAG_OK;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EBAG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const void* const* d_tables = nullptr;
    ebag_status st = stage_tables(h, tables, nullptr, nullptr, s, &d_tables);
    if (st != EBAG_OK) return st;
    BwdWeightsParams p;
    p.tables = d_tables;
    p.meta = h->d_meta;
    p.indices = indices;
    p.offsets = offsets;
    p.grad_out = grad_out;
    p.grad_w = grad_weights;
    p.status = h->d_status;
    p.n_indices = n_indices;
    p.B = B;
    p.T = h->T;
    p.sumD = h->sumD;
    p.mean = mode == EBAG_MEAN ? 1 : 0;
    p.idx32 = index_bits == 32 ? 1 : 0;
    p.code_zero = h->dtype == EBAG_UINT8_ROWWISE ? 0.0f : 128.0f;
    int launches = 0;
    EBAG_CUDA(h, launch_bwd_weights(h->dtype == EBAG_UINT8_ROWWISE ? (int)EBAG_INT8_ROWWISE : h->dtype, p,
                                    h->width_classes, h->num_sms, s, &launches));
    h->launches += launches;
    return EBAG_OK;
}

ebag_status ebag_last_status(ebag_tbe* h, ebag_stream stream, int64_t* n_oob, int64_t* n_bad_offsets) {
    if (!h) return EBAG_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (!guard.ok) return EBAG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    Status host;
    EBAG_CUDA(h, cudaMemcpyAsync(&host, h->d_status, sizeof host, cudaMemcpyDeviceToHost, s));
    EBAG_CUDA(h, cudaMemsetAsync(h->d_status, 0, sizeof(Status), s));
    EBAG_CUDA(h, cudaStreamSynchronize(s));
    if (n_oob) *n_oob = (int64_t)host.n_oob;
    if (n_bad_offsets) *n_bad_offsets = (int64_t)host.n_bad_offsets;
    if (host.n_bad_offsets) return EBAG_ERR_BAD_OFFSETS;
    if (host.n_oob) return EBAG_ERR_INDEX_OOB;
    return EBAG_OK;
}

namespace {
ebag_status pack_rowwise8(const void* q, const float* scale, const float* bias, int64_t rows, int32_t D,
                          void* dst, uint32_t flip, ebag_stream stream) {
    if (rows < 0 || ebag_row_stride(EBAG_INT8_ROWWISE, D) < 0) return EBAG_ERR_INVALID_ARG;
    if (rows == 0) return EBAG_OK;
    if (!q || !scale || !bias || !dst) return EBAG_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15u) || ((uintptr_t)dst & 15u)) return EBAG_ERR_INVALID_ARG;
    const int64_t total = rows * (D / 16 + 1);
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    pack_int8_rowwise_kernel<<<(int)blocks, 256, 0, (cudaStream_t)stream>>>(
        static_cast<const int8_t*>(q), scale, bias, rows, D, static_cast<uint4*>(dst), flip);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    return EBAG_OK;
}
}  // namespace

ebag_status ebag_pack_int8_rowwise(const int8_t* q, const float* scale, const float* bias,
                                   int64_t rows, int32_t D, void* dst, ebag_stream stream) {
    return pack_rowwise8(q, scale, bias, rows, D, dst, 0x80808080u, stream);
}

ebag_status ebag_pack_uint8_rowwise(const uint8_t* q, const float* scale, const float* bias,
                                    int64_t rows, int32_t D, void* dst, ebag_stream stream) {
    return pack_rowwise8(q, scale, bias, rows, D, dst, 0u, stream);
}

ebag_status ebag_set_param(ebag_tbe* h, const char* name, int64_t value) {
    if (!h || !name) return EBAG_ERR_INVALID_ARG;
    if (std::strcmp(name, "item_bytes") == 0) {
        if (value < 256 || value > (1ll << 30)) return EBAG_ERR_INVALID_ARG;
        h->item_bytes = (uint32_t)value;
        return EBAG_OK;
    }
    if (std::strcmp(name, "bwd_sorted") == 0) {
        if (value != 0 && value != 1) return EBAG_ERR_INVALID_ARG;
        h->bwd_sorted = (int)value;
        return EBAG_OK;
    }
    if (std::strcmp(name, "split_bytes") == 0) {
        if (value != 0 && (value < 1024 || value > (1ll << 31) - 1)) return EBAG_ERR_INVALID_ARG;
        h->split_bytes = (uint32_t)value;
        return EBAG_OK;
    }
    if (std::strcmp(name, "mapid_fused") == 0) {
        if (value != 0 && value != 1) return EBAG_ERR_INVALID_ARG;
        h->mapid_fused = (int)value;
        return EBAG_OK;
    }
    if (std::strcmp(name, "mapid_hash") == 0) {
        if (value != 0 && value != 1) return EBAG_ERR_INVALID_ARG;
        h->mapid_hash = (int)value;
        return EBAG_OK;
    }
    if (std::strcmp(name, "out_dtype") == 0) {
        if (value != EBAG_F32 && value != EBAG_F16 && value != EBAG_BF16) return EBAG_ERR_INVALID_ARG;
        h->out_dtype = (int)value;
        return EBAG_OK;
    }
    if (std::strcmp(name, "host_chunks") == 0) {
        if (value < 0 || value > kMaxHostChunks) return EBAG_ERR_INVALID_ARG;
        h->host_chunks = (int)value;
        return EBAG_OK;
    }
    if (std::strcmp(name, "ctas_per_sm") == 0) {
        if (value < 0 || value > 32) return EBAG_ERR_INVALID_ARG;
        h->ctas_per_sm = (int)value;
        return EBAG_OK;
    }
    return EBAG_ERR_INVALID_ARG;
}

int64_t ebag_launch_count(const ebag_tbe* h) { return h ? h->launches : 0; }

const char* ebag_last_cuda_error(const ebag_tbe* h) { return h ? h->cuda_error.c_str() : ""; }

void ebag_destroy(ebag_tbe* h) {
    if (!h) return;
    DeviceGuard guard(h->device);
    cudaDeviceSynchronize();
    free_handle(h);
}

const char* ebag_status_string(ebag_status s) {
    switch (s) {
        case EBAG_OK: return "ok";
        case EBAG_ERR_INVALID_ARG: return "invalid argument";
        case EBAG_ERR_UNSUPPORTED: return "unsupported";
        case EBAG_ERR_CUDA: return "CUDA error";
        case EBAG_ERR_INDEX_OOB: return "out-of-range ids were skipped";
        case EBAG_ERR_BAD_OFFSETS: return "malformed bags were treated as empty";
        default: return "unknown status";
    }
}

}  // extern "C"
