// Gradient of the pooled forward with respect to the per-sample weights (sm_100a).
//
// The forward is linear in the weights (the scores of the paper's weighted sparse features,
// Sec. 2.2 "Feature Types and Memory Layout"), so for lookup i of bag (t, b)
//     grad_w[i] = sum_d grad_out[b, Doff[t] + d] * value(t, indices[i], d)      (EBAG_MEAN: / L)
// one dot product per lookup between the bag's slice of grad_out and the looked-up row.  It is the
// forward's gather with the roles swapped: the bag's slice sits in registers (G lanes x one
// 16-byte row vector each, wider rows in column tiles of G vectors), every looked-up row is read
// once with 16-byte loads, four rows of a bag in flight, the products are summed over the lanes
// of the group with shuffles in a fixed order (so the result is reproducible bit for bit) and the
// group's first lane writes the lookup's gradient.  32/G bags run side by side in a warp; work is
// dealt statically in table-major order.  Ids outside the table give 0 and are counted,
// malformed bags are skipped and counted, as everywhere else.
#include <cuda_runtime.h>
#include <stdint.h>

#include "ebag_bwd_weights.cuh"

namespace ebag {

namespace {

constexpr int kGwThreads = 256;
constexpr int kGwWarps = kGwThreads / 32;
constexpr int kGwRows = 4;            // rows of a bag in flight per group

// sum_k g[k] * widen(d)[k] over the elements of one 16-byte row vector.  Rowwise 8-bit: the
// element is scale * (code - zero) + bias with product and sum rounded separately, as the value
// is defined.
template <int DT>
__device__ __forceinline__ float dot_vec(const float* g, const uint4& d, float scale, float bias, float code_zero) {
    const uint32_t r[4] = {d.x, d.y, d.z, d.w};
    float s = 0.0f;
    if constexpr (DT == DT_F32) {
#pragma unroll
        for (int i = 0; i < 4; ++i) s = fmaf(g[i], __uint_as_float(r[i]), s);
    } else if constexpr (DT == DT_BF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            s = fmaf(g[2 * i], __uint_as_float(r[i] << 16), s);
            s = fmaf(g[2 * i + 1], __uint_as_float(r[i] & 0xffff0000u), s);
        }
    } else if constexpr (DT == DT_F16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&r[i]));
            s = fmaf(g[2 * i], f.x, s);
            s = fmaf(g[2 * i + 1], f.y, s);
        }
    } else {
        const float zero = 8388608.0f + code_zero;       // 2^23 + the byte that means code 0
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float q = __uint_as_float(__byte_perm(r[i], 0x4B000000u, 0x7440 + k)) - zero;   // exact
                s = fmaf(g[4 * i + k], __fadd_rn(__fmul_rn(scale, q), bias), s);
            }
    }
    return s;
}

template <int DT>
__global__ void __launch_bounds__(kGwThreads) ebag_bwd_weights_kernel(const BwdWeightsParams p) {
    constexpr int NACC = Elem<DT>::kAcc;                // elements per 16-byte row vector
    extern __shared__ int item_base[];                  // [T+1] first item of each table
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    for (int t = tid; t < p.T; t += kGwThreads) {
        const int ng = 32 >> p.meta[t].g_log2;
        item_base[t + 1] = (int)((p.B + ng - 1) / ng);
    }
    __syncthreads();
    if (tid == 0) {
        item_base[0] = 0;
        for (int t = 0; t < p.T; ++t) item_base[t + 1] += item_base[t];
    }
    __syncthreads();
    const int64_t total = item_base[p.T];
    const int64_t warps = (int64_t)gridDim.x * kGwWarps;
    unsigned n_oob = 0, n_bad = 0;

    for (int64_t item = (int64_t)blockIdx.x * kGwWarps + wid; item < total; item += warps) {
        int lo_t = 0, hi_t = p.T;
        while (hi_t - lo_t > 1) {
            const int mid = (lo_t + hi_t) >> 1;
            if (item_base[mid] <= item) lo_t = mid; else hi_t = mid;
        }
        const int t = lo_t;
        const TableMeta m = p.meta[t];
        const int G = 1 << m.g_log2, ng = 32 >> m.g_log2;
        const int lig = lane & (G - 1), grp = lane >> m.g_log2;
        const int64_t b = (item - item_base[t]) * ng + grp;
        int64_t lo = 0, hi = 0;
        if (b < p.B) {
            const int64_t g = (int64_t)t * p.B + b;
            lo = p.offsets[g];
            hi = p.offsets[g + 1];
            if (lo < 0 || hi < lo || hi > p.n_indices) {
                if (lig == 0) ++n_bad;
                lo = hi = 0;
            }
        }
        const int64_t L = hi - lo;
        const int64_t Lmax = __reduce_max_sync(0xffffffffu, (unsigned)(L > 0x7fffffffll ? 0x7fffffff : L));
        const char* __restrict__ tbase = static_cast<const char*>(p.tables[t]);
        const float* __restrict__ go = p.grad_out + b * (int64_t)p.sumD + m.D_off;
        const bool inv_on = p.mean && L > 0;

        for (int c0 = 0; c0 < m.nvec; c0 += G) {                  // column tiles of G row vectors
            const int vec = c0 + lig;
            const bool on = vec < m.nvec && L > 0;
            float g[NACC];
#pragma unroll
            for (int k = 0; k < NACC; k += 4) {
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (on) x = __ldg(reinterpret_cast<const float4*>(go + (size_t)vec * NACC + k));
                g[k] = x.x; g[k + 1] = x.y; g[k + 2] = x.z; g[k + 3] = x.w;
            }
            // the ids of the next batch are requested before the current batch's rows
            int64_t rn[kGwRows];
            auto fetch_ids = [&](int64_t j0) {
#pragma unroll
                for (int k = 0; k < kGwRows; ++k) {
                    rn[k] = -1;
                    if (j0 + k < L)
                        rn[k] = p.idx32 ? (int64_t)__ldg(reinterpret_cast<const int*>(p.indices) + lo + j0 + k)
                                        : (int64_t)__ldg(reinterpret_cast<const long long*>(p.indices) + lo + j0 + k);
                }
            };
            fetch_ids(0);
            for (int64_t j0 = 0; j0 < Lmax; j0 += kGwRows) {
                int64_t r[kGwRows];
                bool valid[kGwRows];
                uint4 d[kGwRows];
                float2 sb[kGwRows];
#pragma unroll
                for (int k = 0; k < kGwRows; ++k) {
                    const bool live = j0 + k < L;
                    r[k] = rn[k];
                    valid[k] = live && (uint64_t)r[k] < (uint64_t)m.rows;
                    if (live && !valid[k] && lig == 0 && c0 == 0) ++n_oob;
                }
                fetch_ids(j0 + kGwRows);
#pragma unroll
                for (int k = 0; k < kGwRows; ++k) {
                    d[k] = make_uint4(0u, 0u, 0u, 0u);
                    sb[k] = make_float2(0.0f, 0.0f);
                    if (valid[k] && on) {
                        const char* row = tbase + (uint64_t)r[k] * (uint32_t)m.stride;
                        d[k] = __ldg(reinterpret_cast<const uint4*>(row) + vec);
                        if (DT == DT_INT8) sb[k] = __ldg(reinterpret_cast<const float2*>(row + m.D));
                    }
                }
#pragma unroll
                for (int k = 0; k < kGwRows; ++k) {
                    float s = (valid[k] && on) ? dot_vec<DT>(g, d[k], sb[k].x, sb[k].y, p.code_zero) : 0.0f;
                    // the lanes of the group, added in a fixed (butterfly) order
                    for (int o = G >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                    if (lig == 0 && j0 + k < L) {
                        if (!valid[k]) s = 0.0f;
                        float* out = p.grad_w + lo + j0 + k;
                        if (c0 > 0) s += *out;                       // later column tiles add to the first one's
                        if (inv_on && c0 + G >= m.nvec) s = __fdiv_rn(s, (float)L);
                        *out = s;
                    }
                }
            }
        }
    }
    n_oob = __reduce_add_sync(0xffffffffu, n_oob);
    n_bad = __reduce_add_sync(0xffffffffu, n_bad);
    if (lane == 0) {
        if (n_oob) atomicAdd(&p.status->n_oob, (unsigned long long)n_oob);
        if (n_bad) atomicAdd(&p.status->n_bad_offsets, (unsigned long long)n_bad);
    }
}

}  // namespace

size_t bwd_weights_smem_bytes(int T) { return (size_t)(T + 1) * sizeof(int); }

cudaError_t launch_bwd_weights(int dtype, const BwdWeightsParams& p, int grid, cudaStream_t s) {
    const size_t smem = bwd_weights_smem_bytes(p.T);
    switch (dtype) {
        case DT_F32: ebag_bwd_weights_kernel<DT_F32><<<grid, kGwThreads, smem, s>>>(p); break;
        case DT_F16: ebag_bwd_weights_kernel<DT_F16><<<grid, kGwThreads, smem, s>>>(p); break;
        case DT_BF16: ebag_bwd_weights_kernel<DT_BF16><<<grid, kGwThreads, smem, s>>>(p); break;
        default: ebag_bwd_weights_kernel<DT_INT8><<<grid, kGwThreads, smem, s>>>(p); break;
    }
    return cudaGetLastError();
}

}  // namespace ebag
