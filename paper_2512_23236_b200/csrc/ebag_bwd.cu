// Backward of the pooled embedding-bag forward (sm_100a): scatter-add of w_i * grad_out into
// the rows the bags looked up.
//
// grad_t[indices[i], d] += w_i * grad_out[b, Doff[t] + d] * (1/L in mean mode)
// for every lookup i of every bag (t, b); gradient tables are dense fp32 [rows_t, D_t] that the
// caller owns and zeroes (or keeps accumulating into).
//
// A bag's slice of grad_out is the same for all its lookups, so it is read once into registers
// (G lanes x 16 bytes cover it; G in {1,2,..,32} by row width, wider rows in column tiles of
// G x kTileVecs vectors) and then sent to each looked-up row with 16-byte vector reductions
// (`red.global.add.v4.f32`): fire-and-forget, resolved in L2, no return value to wait for.
// 32/G bags run side by side in one warp.  Work is dealt statically: warp w takes the groups of
// 32/G consecutive bags numbered w, w + W, ... in table-major order; the ids of a bag are read
// four at a time (every lane of a group reads the same id, one transaction).
//
// The order in which the contributions to a row arrive is not fixed, so results are
// reproducible only up to fp32 rounding.  Ids outside the table and malformed bags are skipped
// and counted, as in the forward.
#include <cuda_runtime.h>
#include <stdint.h>

#include "ebag_bwd.cuh"

namespace ebag {

namespace {

constexpr int kBwdThreads = 256;
constexpr int kTileVecs = 2;          // 16-byte vectors of grad_out a lane holds per column tile
constexpr int kIdBatch = 4;           // ids of a bag fetched together

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

template <bool WEIGHTED>
__global__ void __launch_bounds__(kBwdThreads) ebag_bwd_kernel(const BwdParams p) {
    extern __shared__ int item_base[];                        // [T+1] first item of each table
    const int tid = threadIdx.x, lane = tid & 31;
    // ---- items: groups of 32/G consecutive bags of a table
    for (int t = tid; t < p.T; t += kBwdThreads) {
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
    const int64_t warps = (int64_t)gridDim.x * (kBwdThreads / 32);
    unsigned n_oob = 0, n_bad = 0;

    for (int64_t item = (int64_t)blockIdx.x * (kBwdThreads / 32) + (tid >> 5); item < total; item += warps) {
        int lo_t = 0, hi_t = p.T;
        while (hi_t - lo_t > 1) {
            const int mid = (lo_t + hi_t) >> 1;
            if (item_base[mid] <= item) lo_t = mid; else hi_t = mid;
        }
        const int t = lo_t;
        const BwdTableMeta m = p.meta[t];
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
        float* __restrict__ gt = p.grad_tables[t];
        const float* __restrict__ go = p.grad_out + b * (int64_t)p.sumD + m.D_off;
        const int64_t Lmax = __reduce_max_sync(0xffffffffu, (unsigned)(L > 0x7fffffffll ? 0x7fffffff : L));

        for (int c0 = 0; c0 < m.nvec; c0 += G * kTileVecs) {       // column tiles
            float4 gv[kTileVecs];
            bool on[kTileVecs];
#pragma unroll
            for (int v = 0; v < kTileVecs; ++v) {
                const int vec = c0 + v * G + lig;
                on[v] = vec < m.nvec && L > 0;
                gv[v] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (on[v]) {
                    gv[v] = __ldcs(reinterpret_cast<const float4*>(go) + vec);
                    if (p.mean) {
                        // the forward divides the pooled sum by L: its transpose divides grad_out by L
                        gv[v].x = __fdiv_rn(gv[v].x, (float)L); gv[v].y = __fdiv_rn(gv[v].y, (float)L);
                        gv[v].z = __fdiv_rn(gv[v].z, (float)L); gv[v].w = __fdiv_rn(gv[v].w, (float)L);
                    }
                }
            }
            for (int64_t j0 = 0; j0 < Lmax; j0 += kIdBatch) {
                int64_t r[kIdBatch];
                float w[kIdBatch];
#pragma unroll
                for (int k = 0; k < kIdBatch; ++k) {
                    const int64_t i = lo + j0 + k;
                    r[k] = -1;
                    w[k] = 1.0f;
                    if (j0 + k < L) {
                        r[k] = p.idx32 ? (int64_t)__ldg(reinterpret_cast<const int*>(p.indices) + i)
                                       : __ldg(reinterpret_cast<const long long*>(p.indices) + i);
                        if (WEIGHTED) w[k] = __ldg(p.weights + i);
                    }
                }
#pragma unroll
                for (int k = 0; k < kIdBatch; ++k) {
                    if (j0 + k >= L) continue;
                    if ((uint64_t)r[k] >= (uint64_t)m.rows) {
                        if (lig == 0 && c0 == 0) ++n_oob;
                        continue;
                    }
                    float* row = gt + r[k] * (int64_t)m.D;
#pragma unroll
                    for (int v = 0; v < kTileVecs; ++v)
                        if (on[v]) {
                            float* a = row + (size_t)(c0 + v * G + lig) * 4;
                            if (WEIGHTED) red_add_v4(a, w[k] * gv[v].x, w[k] * gv[v].y, w[k] * gv[v].z, w[k] * gv[v].w);
                            else red_add_v4(a, gv[v].x, gv[v].y, gv[v].z, gv[v].w);
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

cudaError_t launch_bwd(const BwdParams& p, bool weighted, int grid, cudaStream_t s) {
    const size_t smem = (size_t)(p.T + 1) * sizeof(int);
    if (weighted) ebag_bwd_kernel<true><<<grid, kBwdThreads, smem, s>>>(p);
    else ebag_bwd_kernel<false><<<grid, kBwdThreads, smem, s>>>(p);
    return cudaGetLastError();
}

cudaError_t occupancy_bwd(bool weighted, int T, int* ctas_per_sm) {
    const size_t smem = (size_t)(T + 1) * sizeof(int);
    return weighted ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, ebag_bwd_kernel<true>,
                                                                     kBwdThreads, smem)
                    : cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, ebag_bwd_kernel<false>,
                                                                     kBwdThreads, smem);
}

}  // namespace ebag
