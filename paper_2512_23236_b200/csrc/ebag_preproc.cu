// Preprocessing producers of embedding ids that sit in front of the pooled forward
// (paper Sec. 5.4 "Data Preprocessing Kernels on MTIA").  Contracts are in include/ebag.h.
#include <cuda_runtime.h>

#include "ebag.h"

namespace {

constexpr int kThreads = 256;
constexpr int kSmemBorders = 64;     // border lists up to this long are counted linearly from smem
constexpr int kIlp = 8;              // values per thread in flight (8 x 4 B x 2048 threads = 64 KB per SM)

// MergeBucketizedDense (Sec. 5.4.2): out[f, i] = #borders of feature f below values[f, i] + off[f].
// blockIdx.y is the feature.  "Below" is written !(x <= b) so that NaN lands in the last bin,
// like the library routine the paper's pseudocode calls.  Short lists are counted linearly
// (the vectorised counting the paper's kernel uses), long ones by a branch-free halving search.
__global__ void __launch_bounds__(kThreads)
mbdt_kernel(const float* __restrict__ values, int64_t B, const float* __restrict__ borders,
            const int64_t* __restrict__ border_offsets, const int64_t* __restrict__ out_offsets,
            int64_t* __restrict__ out) {
    __shared__ float sb[kSmemBorders];
    const int f = blockIdx.y;
    const int64_t b0 = border_offsets[f];
    const int64_t K64 = border_offsets[f + 1] - b0;
    const int K = K64 < 0 ? 0 : (K64 > 0x7fffffff ? 0x7fffffff : (int)K64);
    const float* __restrict__ bf = borders + b0;
    const int64_t add = out_offsets[f];
    if (K <= kSmemBorders) {
        for (int k = threadIdx.x; k < K; k += kThreads) sb[k] = bf[k];
        __syncthreads();
    }
    const float* __restrict__ vf = values + (int64_t)f * B;
    int64_t* __restrict__ of = out + (int64_t)f * B;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < B; i += kIlp * stride) {
        float x[kIlp];
        int n[kIlp];
#pragma unroll
        for (int k = 0; k < kIlp; ++k) n[k] = 0;
#pragma unroll
        for (int k = 0; k < kIlp; ++k) x[k] = i + k * stride < B ? __ldcs(vf + i + k * stride) : 0.0f;
        if (K <= kSmemBorders) {
            for (int j = 0; j < K; ++j) {
                const float b = sb[j];
#pragma unroll
                for (int k = 0; k < kIlp; ++k) n[k] += !(x[k] <= b);
            }
        } else {
            const int steps = 32 - __clz(K);
            int lo[kIlp], hi[kIlp];
#pragma unroll
            for (int k = 0; k < kIlp; ++k) {
                lo[k] = 0;
                hi[k] = K;
            }
            for (int s = 0; s < steps; ++s) {
#pragma unroll
                for (int k = 0; k < kIlp; ++k) {
                    const int mid = (lo[k] + hi[k]) >> 1;
                    const float b = __ldg(bf + (mid < K ? mid : K - 1));
                    const bool active = lo[k] < hi[k];
                    const bool right = !(x[k] <= b);
                    lo[k] = (active && right) ? mid + 1 : lo[k];
                    hi[k] = (active && !right) ? mid : hi[k];
                }
            }
#pragma unroll
            for (int k = 0; k < kIlp; ++k) n[k] = lo[k];
        }
#pragma unroll
        for (int k = 0; k < kIlp; ++k)
            if (i + k * stride < B) __stcs(reinterpret_cast<long long*>(of + i + k * stride), (long long)(n[k] + add));
    }
}

}  // namespace

extern "C" ebag_status ebag_mbdt(const float* values, int32_t F, int64_t B, const float* borders,
                                 const int64_t* border_offsets, const int64_t* out_offsets,
                                 int64_t* out, ebag_stream stream) {
    if (F < 0 || B < 0 || F > 65535) return EBAG_ERR_INVALID_ARG;
    if (F == 0 || B == 0) return EBAG_OK;
    if (!values || !border_offsets || !out_offsets || !out) return EBAG_ERR_INVALID_ARG;
    // one wave: as many blocks as fit on the device at once, split evenly over the features
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, mbdt_kernel, kThreads, 0) != cudaSuccess) {
        cudaGetLastError();
        return EBAG_ERR_CUDA;
    }
    int64_t bx = (B + kIlp * kThreads - 1) / (kIlp * kThreads);
    int64_t cap = (int64_t)sms * per_sm / F;
    if (cap < 1) cap = 1;
    if (bx > cap) bx = cap;
    mbdt_kernel<<<dim3((unsigned)bx, (unsigned)F), kThreads, 0, (cudaStream_t)stream>>>(
        values, B, borders, border_offsets, out_offsets, out);
    if (cudaGetLastError() != cudaSuccess) return EBAG_ERR_CUDA;
    return EBAG_OK;
}

// ---------------------------------------------------------------------------------------------
// Batch Event Truncate (paper Sec. 5.5): keep the first N events of every user in every feature
// of a nested jagged batch, all features in a constant number of launches.  The kept events of a
// user are a prefix of that user's events, so per feature a user's kept inner lengths and kept
// values are each ONE contiguous range; only user-level prefix sums are needed:
//   1. scan outer lengths            -> first event of every user, before and after (1 CTA)
//   2. per (feature, user) sums      -> values held / kept by the user           (1 warp each)
//   3. scan those per feature        -> first value of every user, before and after (1 CTA each)
//   4. copy the two ranges per (feature, user)                                    (1 warp each)
namespace {

constexpr int kScanThreads = 1024;

struct BetWorkspace {        // carved out of the caller's workspace; all int64
    int64_t* ev_in;          // [U+1] first event of user u in the input
    int64_t* ev_out;         // [U+1] ... in the output
    int64_t* v_all;          // [F, U] values user u holds in feature f
    int64_t* v_keep;         // [F, U] values of its kept events
    int64_t* v_in;           // [F, U+1] first value of user u in the input (relative to the feature)
    int64_t* v_out;          // [F, U+1] ... in the output
};

__host__ __device__ inline BetWorkspace carve(void* ws, int F, int64_t U) {
    int64_t* p = static_cast<int64_t*>(ws);
    BetWorkspace w;
    w.ev_in = p;  p += U + 1;
    w.ev_out = p; p += U + 1;
    w.v_all = p;  p += (int64_t)F * U;
    w.v_keep = p; p += (int64_t)F * U;
    w.v_in = p;   p += (int64_t)F * (U + 1);
    w.v_out = p;
    return w;
}

// exclusive prefix sums of a[0..n) and b[0..n) by one CTA, totals written at index n.
// Every thread owns kScanItems consecutive entries per round (negative entries count as 0).
constexpr int kScanItems = 4;
__device__ void block_exscan2(const int64_t* __restrict__ a, const int64_t* __restrict__ b, int64_t n,
                              int64_t* __restrict__ sa, int64_t* __restrict__ sb) {
    __shared__ int64_t warp_a[32], warp_b[32], carry[2];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (tid == 0) carry[0] = carry[1] = 0;
    __syncthreads();
    for (int64_t base = 0; base < n; base += (int64_t)kScanThreads * kScanItems) {
        const int64_t i0 = base + (int64_t)tid * kScanItems;
        int64_t xa[kScanItems], xb[kScanItems];
        int64_t ta = 0, tb = 0;                      // this thread's totals
#pragma unroll
        for (int k = 0; k < kScanItems; ++k) {
            xa[k] = i0 + k < n ? a[i0 + k] : 0;
            xb[k] = i0 + k < n ? b[i0 + k] : 0;
            if (xa[k] < 0) xa[k] = 0;
            if (xb[k] < 0) xb[k] = 0;
            ta += xa[k];
            tb += xb[k];
        }
        int64_t ia = ta, ib = tb;                    // inclusive over the threads of the warp
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int64_t ya = __shfl_up_sync(0xffffffffu, ia, d), yb = __shfl_up_sync(0xffffffffu, ib, d);
            if (lane >= d) { ia += ya; ib += yb; }
        }
        if (lane == 31) { warp_a[wid] = ia; warp_b[wid] = ib; }
        __syncthreads();
        if (wid == 0) {
            int64_t wa = warp_a[lane], wb = warp_b[lane];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int64_t ya = __shfl_up_sync(0xffffffffu, wa, d), yb = __shfl_up_sync(0xffffffffu, wb, d);
                if (lane >= d) { wa += ya; wb += yb; }
            }
            warp_a[lane] = wa; warp_b[lane] = wb;      // inclusive over warps
        }
        __syncthreads();
        int64_t ra = carry[0] + (wid ? warp_a[wid - 1] : 0) + ia - ta;   // exclusive for this thread
        int64_t rb = carry[1] + (wid ? warp_b[wid - 1] : 0) + ib - tb;
#pragma unroll
        for (int k = 0; k < kScanItems; ++k) {
            if (i0 + k < n) { sa[i0 + k] = ra; sb[i0 + k] = rb; }
            ra += xa[k];
            rb += xb[k];
        }
        __syncthreads();
        if (tid == 0) { carry[0] += warp_a[31]; carry[1] += warp_b[31]; }
        __syncthreads();
    }
    if (tid == 0) { sa[n] = carry[0]; sb[n] = carry[1]; }
}

__global__ void __launch_bounds__(kScanThreads)
bet_scan_outer(const int64_t* __restrict__ outer, int64_t U, int64_t N, int64_t* __restrict__ outer_out,
               BetWorkspace w, int64_t* __restrict__ counts_out) {
    for (int64_t u = threadIdx.x; u < U; u += kScanThreads) {
        int64_t n = outer[u];
        if (n < 0) n = 0;
        outer_out[u] = n < N ? n : N;
    }
    __syncthreads();
    block_exscan2(outer, outer_out, U, w.ev_in, w.ev_out);
    __syncthreads();
    if (threadIdx.x == 0) counts_out[0] = w.ev_out[U];
}

// one warp per (feature, user): how many values the user holds and how many its kept events hold
__global__ void bet_user_sums(const int64_t* __restrict__ inner, int64_t E, int64_t U, BetWorkspace w) {
    const int f = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int64_t u = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5);
    if (u >= U) return;
    int64_t e0 = w.ev_in[u], e1 = w.ev_in[u + 1];
    const int64_t keep = w.ev_out[u + 1] - w.ev_out[u];
    if (e1 > E) e1 = E;                               // never read past the caller's array
    if (e0 > e1) e0 = e1;
    const int64_t* __restrict__ row = inner + (int64_t)f * E;
    int64_t all = 0, kept = 0;
    for (int64_t j = lane; j < e1 - e0; j += 32) {
        int64_t n = __ldcs(reinterpret_cast<const long long*>(row + e0 + j));
        if (n < 0) n = 0;
        all += n;
        if (j < keep) kept += n;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        all += __shfl_xor_sync(0xffffffffu, all, d);
        kept += __shfl_xor_sync(0xffffffffu, kept, d);
    }
    if (lane == 0) {
        w.v_all[(int64_t)f * U + u] = all;
        w.v_keep[(int64_t)f * U + u] = kept;
    }
}

__global__ void __launch_bounds__(kScanThreads)
bet_scan_values(int64_t U, BetWorkspace w, int64_t* __restrict__ counts_out) {
    const int f = blockIdx.x;
    block_exscan2(w.v_all + (int64_t)f * U, w.v_keep + (int64_t)f * U, U, w.v_in + (int64_t)f * (U + 1),
                  w.v_out + (int64_t)f * (U + 1));
    __syncthreads();
    if (threadIdx.x == 0) counts_out[1 + f] = w.v_out[(int64_t)f * (U + 1) + U];
}

// one warp per (feature, user): copy the kept inner lengths and the kept values, both contiguous
__global__ void __launch_bounds__(256)
bet_copy(const int64_t* __restrict__ inner, int64_t E, const int64_t* __restrict__ values,
         const int64_t* __restrict__ value_offsets, int64_t U, BetWorkspace w,
         int64_t* __restrict__ inner_out, int64_t* __restrict__ values_out) {
    const int f = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t vbase = value_offsets[f], vend = value_offsets[f + 1];
    for (int64_t u = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); u < U; u += warps) {
        const int64_t e_in = w.ev_in[u], e_out = w.ev_out[u];
        int64_t keep = w.ev_out[u + 1] - e_out;
        if (e_in + keep > E) keep = E > e_in ? E - e_in : 0;
        const int64_t v_in = vbase + w.v_in[(int64_t)f * (U + 1) + u];
        const int64_t v_out = vbase + w.v_out[(int64_t)f * (U + 1) + u];
        int64_t nv = w.v_keep[(int64_t)f * U + u];
        if (v_in + nv > vend) nv = vend > v_in ? vend - v_in : 0;      // stay inside the feature's values
        const int64_t* __restrict__ src_i = inner + (int64_t)f * E + e_in;
        int64_t* __restrict__ dst_i = inner_out + (int64_t)f * E + e_out;
        for (int64_t j = lane; j < keep; j += 32) {
            const int64_t n = __ldcs(reinterpret_cast<const long long*>(src_i + j));
            __stcs(reinterpret_cast<long long*>(dst_i + j), (long long)(n < 0 ? 0 : n));
        }
        for (int64_t j = lane; j < nv; j += 32)
            __stcs(reinterpret_cast<long long*>(values_out + v_out + j),
                   __ldcs(reinterpret_cast<const long long*>(values + v_in + j)));
    }
}

}  // namespace

extern "C" int64_t ebag_bet_workspace_bytes(int32_t F, int64_t U) {
    if (F < 0 || U < 0) return -1;
    return (int64_t)sizeof(int64_t) * (2 * (U + 1) + 2 * (int64_t)F * U + 2 * (int64_t)F * (U + 1));
}

extern "C" ebag_status ebag_batch_event_truncate(const int64_t* outer_lengths, int64_t U,
                                                 const int64_t* inner_lengths, int64_t E,
                                                 const int64_t* values, const int64_t* value_offsets,
                                                 int32_t F, int64_t N, int64_t* outer_out,
                                                 int64_t* inner_out, int64_t* values_out,
                                                 int64_t* counts_out, void* workspace,
                                                 int64_t workspace_bytes, ebag_stream stream) {
    if (F < 0 || F > 65535 || U < 0 || E < 0 || N < 0) return EBAG_ERR_INVALID_ARG;
    if (!counts_out) return EBAG_ERR_INVALID_ARG;
    if (U > 0 && (!outer_lengths || !outer_out)) return EBAG_ERR_INVALID_ARG;
    if (F > 0 && (!value_offsets || (E > 0 && (!inner_lengths || !inner_out)))) return EBAG_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < ebag_bet_workspace_bytes(F, U) || ((uintptr_t)workspace & 7u))
        return EBAG_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    const BetWorkspace w = carve(workspace, F, U);
    bet_scan_outer<<<1, kScanThreads, 0, s>>>(outer_lengths, U, N, outer_out, w, counts_out);
    if (F > 0 && U > 0) {
        const int warps = 8;
        bet_user_sums<<<dim3((unsigned)((U + warps - 1) / warps), (unsigned)F), warps * 32, 0, s>>>(
            inner_lengths, E, U, w);
    }
    if (F > 0) bet_scan_values<<<F, kScanThreads, 0, s>>>(U, w, counts_out);
    if (F > 0 && U > 0) {
        int64_t bx = (U + 7) / 8;
        const int64_t cap = 148 * 8 * 4 / F + 1;           // a few waves of 8-warp CTAs
        if (bx > cap) bx = cap;
        bet_copy<<<dim3((unsigned)bx, (unsigned)F), 256, 0, s>>>(inner_lengths, E, values, value_offsets, U, w,
                                                                 inner_out, values_out);
    }
    if (cudaGetLastError() != cudaSuccess) return EBAG_ERR_CUDA;
    return EBAG_OK;
}
