// ebag_forward_noalloc: the pooled forward for callers that must not allocate device memory.
//
// Some processes cannot call cudaMalloc at the time they need a forward: code running inside a
// memory pool whose owner forbids side allocations, a plugin loaded into a host application
// that has already handed all device memory to its own allocator, a latency-critical serving
// thread for which an allocation (and the implicit synchronisation it may bring) is not
// acceptable.  The regular path needs a handle, and creating a handle allocates.  This entry
// point needs no handle: the few KB of device scratch the forward kernel uses (work-queue
// counters, status words, the table-pointer array and the per-table metadata) live in a
// file-scope device array that the loaded library carries on every GPU until the process ends.
//
// The forward kernel itself is the library's regular one; only where its scratch lives differs.
#include <cuda_runtime.h>

#include <mutex>

#include "ebag.h"
#include "ebag_fwd.cuh"

using namespace ebag;

namespace {

constexpr int kMaxTables = EBAG_NOALLOC_MAX_TABLES;
constexpr int kMaxDevices = 64;

struct Scratch {                     // layout of the static array
    Queue queue;                     // must be zero when the forward kernel starts
    Status status;                   // used when the caller passes no status buffer
    const void* tables[kMaxTables];
    TableMeta meta[kMaxTables];
};
static_assert(sizeof(Scratch) <= EBAG_NOALLOC_SCRATCH_BYTES, "scratch layout outgrew its array");

// Every GPU that loads the library holds these bytes until the process exits.  In host code this
// name is only a stand-in for the symbol, never a device address: the address is asked for once
// per device with cudaGetSymbolAddress (below) and that pointer is what kernels are given.
static __device__ __align__(256) unsigned char g_noalloc_scratch[EBAG_NOALLOC_SCRATCH_BYTES];

struct SetupArgs {                   // passed by value as a kernel parameter (about 2.6 KB)
    const void* tables[kMaxTables];
    TableMeta meta[kMaxTables];
    int T;
};

// Fills the metadata part of the scratch and clears what must start at zero.  Device code may
// name the array directly.
__global__ void noalloc_setup_kernel(const SetupArgs a) {
    Scratch* s = reinterpret_cast<Scratch*>(g_noalloc_scratch);
    const int i = threadIdx.x;
    if (i < a.T) {
        s->tables[i] = a.tables[i];
        s->meta[i] = a.meta[i];
    }
    if (i == 0) {
        s->queue.next = 0;
        s->queue.done = 0;
        s->status.n_oob = 0;
        s->status.n_bad_offsets = 0;
    }
}

struct DeviceState {
    bool ready = false;
    Scratch* scratch = nullptr;      // device address of g_noalloc_scratch on this device
    int num_sms = 0;
    int occupancy[4][2] = {};        // CTAs per SM by dtype and weighted
};
DeviceState g_state[kMaxDevices];
std::mutex g_mutex;

int elem_bytes(int dtype) { return dtype == EBAG_F32 ? 4 : (dtype >= EBAG_INT8_ROWWISE ? 1 : 2); }

size_t fwd_smem_bytes(int T) { return (size_t)(2 * T + 1) * sizeof(int); }

cudaError_t launch(int dtype, const FwdParams& p, bool w, int grid, size_t smem, cudaStream_t s) {
    switch (dtype) {
        case EBAG_F32: return launch_fwd_f32(p, w, false, grid, smem, s);
        case EBAG_F16: return launch_fwd_f16(p, w, false, grid, smem, s);
        case EBAG_BF16: return launch_fwd_bf16(p, w, false, grid, smem, s);
        default: return launch_fwd_int8(p, w, false, grid, smem, s);
    }
}

cudaError_t occupancy(int dtype, bool w, size_t smem, int* n) {
    switch (dtype) {
        case EBAG_F32: return occupancy_fwd_f32(w, false, smem, n);
        case EBAG_F16: return occupancy_fwd_f16(w, false, smem, n);
        case EBAG_BF16: return occupancy_fwd_bf16(w, false, smem, n);
        default: return occupancy_fwd_int8(w, false, smem, n);
    }
}

// Once per device, with that device current: resolve the symbol's device address and cache the
// launch geometry.  Nothing here allocates.
ebag_status setup_device(int device, DeviceState** out) {
    if (device < 0 || device >= kMaxDevices) return EBAG_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& st = g_state[device];
    if (!st.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return EBAG_ERR_CUDA;
        }
        if (cudaDeviceGetAttribute(&st.num_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
            cudaGetLastError();
            return EBAG_ERR_CUDA;
        }
        for (int dt = 0; dt < 4; ++dt)
            for (int w = 0; w < 2; ++w) {
                int n = 0;
                if (occupancy(dt, w != 0, fwd_smem_bytes(kMaxTables), &n) != cudaSuccess) {
                    cudaGetLastError();
                    return EBAG_ERR_CUDA;
                }
                st.occupancy[dt][w] = n < 1 ? 1 : n;
            }
        st.scratch = static_cast<Scratch*>(ptr);
        st.ready = true;
    }
    *out = &st;
    return EBAG_OK;
}

}  // namespace

extern "C" ebag_status ebag_forward_noalloc(int32_t T, const int64_t* rows, const int32_t* D,
                                            ebag_dtype dtype, const void* const* tables,
                                            const int64_t* indices, int64_t n_indices,
                                            const int64_t* offsets,
                                            const float* per_sample_weights, int64_t B,
                                            ebag_mode mode, float* out,
                                            unsigned long long* status_counts,
                                            ebag_stream stream) {
    if (T <= 0 || !rows || !D || !tables || !offsets || B < 0 || n_indices < 0)
        return EBAG_ERR_INVALID_ARG;
    if (dtype < EBAG_F32 || dtype > EBAG_UINT8_ROWWISE) return EBAG_ERR_INVALID_ARG;
    if (mode == EBAG_MAX) return EBAG_ERR_UNSUPPORTED;
    if (mode != EBAG_SUM && mode != EBAG_MEAN) return EBAG_ERR_INVALID_ARG;
    if (T > kMaxTables) return EBAG_ERR_UNSUPPORTED;       // beyond the static scratch
    if ((int64_t)T * B >= (1ll << 31)) return EBAG_ERR_UNSUPPORTED;
    if (n_indices > 0 && !indices) return EBAG_ERR_INVALID_ARG;
    if (B > 0 && !out) return EBAG_ERR_INVALID_ARG;
    if (((uintptr_t)out & 15u) || ((uintptr_t)indices & 7u) || ((uintptr_t)offsets & 7u) ||
        ((uintptr_t)per_sample_weights & 3u) || ((uintptr_t)status_counts & 7u))
        return EBAG_ERR_INVALID_ARG;

    SetupArgs args;
    int64_t d_off = 0;
    for (int t = 0; t < T; ++t) {
        const int64_t stride = ebag_row_stride(dtype, D[t]);
        if (stride < 0 || rows[t] < 0) return EBAG_ERR_INVALID_ARG;
        if (rows[t] >= (1ll << 31) || stride >= (1ll << 31)) return EBAG_ERR_UNSUPPORTED;
        if (!tables[t] && rows[t] > 0) return EBAG_ERR_INVALID_ARG;
        if ((uintptr_t)tables[t] & 15u) return EBAG_ERR_INVALID_ARG;
        TableMeta& m = args.meta[t];
        m.rows = rows[t];
        m.D = D[t];
        m.D_off = (int32_t)d_off;
        m.stride = (int32_t)stride;
        m.nvec = (int32_t)((int64_t)D[t] * elem_bytes(dtype) / 16);
        int g_log2 = 2;
        while ((1 << g_log2) < m.nvec && g_log2 < 5) ++g_log2;
        m.g_log2 = g_log2;
        m.V = m.nvec <= 32 ? 1 : 2;
        args.tables[t] = tables[t];
        d_off += D[t];
        if (d_off >= (1ll << 31)) return EBAG_ERR_UNSUPPORTED;
    }
    args.T = T;
    if (B == 0) return EBAG_OK;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) {
        cudaGetLastError();
        return EBAG_ERR_CUDA;
    }
    DeviceState* st = nullptr;
    ebag_status rc = setup_device(device, &st);
    if (rc != EBAG_OK) return rc;

    cudaStream_t s = (cudaStream_t)stream;
    noalloc_setup_kernel<<<1, kMaxTables, 0, s>>>(args);
    if (cudaGetLastError() != cudaSuccess) return EBAG_ERR_CUDA;

    FwdParams p;
    p.tables = st->scratch->tables;          // device addresses inside the static array
    p.meta = st->scratch->meta;
    p.indices = indices;
    p.offsets = offsets;
    p.weights = per_sample_weights;
    p.out = out;
    p.queue = &st->scratch->queue;
    p.mappings = nullptr;
    p.mapping_len = nullptr;
    p.map_slots = nullptr;
    p.map_base = nullptr;
    p.status = status_counts ? reinterpret_cast<Status*>(status_counts) : &st->scratch->status;
    p.n_indices = n_indices;
    p.B = B;
    p.off_stride = B;
    p.T = T;
    p.sumD = (int32_t)d_off;
    p.mean = mode == EBAG_MEAN ? 1 : 0;
    p.idx32 = 0;
    p.out16 = 0;
    p.code_zero = dtype == EBAG_UINT8_ROWWISE ? 0.0f : 128.0f;
    p.item_bytes = 32768;
    p.lg = LongParams{};                     // no room for partial sums here: bags are not split
    const bool w = per_sample_weights != nullptr;
    const int kernel_of = dtype > EBAG_INT8_ROWWISE ? EBAG_INT8_ROWWISE : dtype;   // both 8-bit types share kernels
    const int grid = st->num_sms * st->occupancy[kernel_of][w ? 1 : 0];
    if (launch(dtype, p, w, grid, fwd_smem_bytes(T), s) != cudaSuccess) {
        cudaGetLastError();
        return EBAG_ERR_CUDA;
    }
    return EBAG_OK;
}
