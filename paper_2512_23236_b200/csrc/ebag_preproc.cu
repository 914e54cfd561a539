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
