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
// Hot rows.  Reductions to one address are applied one after the other in L2, and with skewed
// (Zipf) ids a handful of rows per table take a large share of its lookups: the whole grid then
// queues on them (measured: 13 times slower than uniform ids).  So a first, small kernel samples
// the ids of every table and puts its most frequent rows into a small hashed table of K slots
// (K = 2048 / D, at most 32); every warp of the main kernel sums the contributions to those
// rows in its own 8 KB of shared memory (plain loads and stores: a lane owns its columns, and
// groups of lanes that hit one row at the same step take turns) and sends each sum to L2 once
// per table it passes through.
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
constexpr int kBwdWarps = kBwdThreads / 32;
constexpr int kTileVecs = 2;          // 16-byte vectors of grad_out a lane holds per column tile
constexpr int kIdBatch = 4;           // ids of a bag fetched together
#ifndef EBAG_HOT_USE
#define EBAG_HOT_USE 32
#endif
constexpr int kHotUse = EBAG_HOT_USE;   // slots in use at most (<= kHotSlots)
constexpr int kSampleIds = 2048;      // ids of a table the hot-row kernel looks at
constexpr int kSampleSlots = 4096;    // its hash table (32 KB of shared memory)

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}

__device__ __forceinline__ int64_t load_id(const void* indices, int idx32, int64_t i) {
    return idx32 ? (int64_t)__ldg(reinterpret_cast<const int*>(indices) + i)
                 : (int64_t)__ldg(reinterpret_cast<const long long*>(indices) + i);
}

// ---- the most frequent rows of every table, from an evenly spaced sample of its ids.  One CTA
// per table: the sampled ids are counted in a shared-memory hash table (linear probing), then
// the kHotRows largest counts are picked one after the other.  A row must show up at least
// three times in the sample to be named.
__global__ void __launch_bounds__(kBwdThreads) bwd_hot_rows_kernel(const BwdParams p) {
    if (p.only_if && *p.only_if == 0) return;
    __shared__ int keys[kSampleSlots];
    __shared__ int counts[kSampleSlots];
    __shared__ unsigned long long best;
    const int t = blockIdx.x, tid = threadIdx.x;
    for (int i = tid; i < kSampleSlots; i += kBwdThreads) {
        keys[i] = -1;
        counts[i] = 0;
    }
    __syncthreads();
    int64_t o0 = p.offsets[(int64_t)t * p.B], o1 = p.offsets[(int64_t)(t + 1) * p.B];
    if (o0 < 0) o0 = 0;
    if (o1 > p.n_indices) o1 = p.n_indices;
    const int64_t n = o1 > o0 ? o1 - o0 : 0;
    const int64_t S = n < kSampleIds ? n : kSampleIds;
    const int64_t rows = p.meta[t].rows;
    for (int64_t i = tid; i < S; i += kBwdThreads) {
        const int64_t r = load_id(p.indices, p.idx32, o0 + i * n / S);
        if ((uint64_t)r >= (uint64_t)rows) continue;
        unsigned slot = ((unsigned)r * 2654435761u) >> 20;                 // 12 bits
        for (int probe = 0; probe < kSampleSlots; ++probe) {
            const int old = atomicCAS(&keys[slot], -1, (int)r);
            if (old == -1 || old == (int)r) {
                atomicAdd(&counts[slot], 1);
                break;
            }
            slot = (slot + 1) & (kSampleSlots - 1);
        }
    }
    __syncthreads();
    // candidates by decreasing count; each goes to the first of its two hash slots that is still free
    const int D = p.meta[t].D;
    int K = 1;
    while (K * 2 <= kHotUse && K * 2 * D <= kCacheFloats) K *= 2;
    if (D > kCacheFloats) K = 0;
    if (tid < kHotSlots) p.hot[t * kHotSlots + tid] = -1;
    __syncthreads();
    for (int k = 0; k < 2 * K; ++k) {
        if (tid == 0) best = 0;
        __syncthreads();
        unsigned long long mine = 0;
        for (int i = tid; i < kSampleSlots; i += kBwdThreads)
            if (counts[i] >= 3) {
                const unsigned long long v = ((unsigned long long)counts[i] << 32) | (unsigned)i;
                if (v > mine) mine = v;
            }
        if (mine) atomicMax(&best, mine);
        __syncthreads();
        const unsigned long long got = best;
        if (got == 0) break;                                               // uniform: no candidates left
        if (tid == 0) {
            const int slot = (int)(got & 0xffffffffu);
            const int row = keys[slot];
            counts[slot] = 0;                                              // taken
            int* d1 = p.hot + t * kHotSlots + hot_slot((uint32_t)row, K);
            int* d2 = p.hot + t * kHotSlots + hot_slot2((uint32_t)row, K);
            if (*d1 < 0) *d1 = row;
            else if (*d2 < 0) *d2 = row;
        }
        __syncthreads();
    }
}

template <bool WEIGHTED>
__global__ void __launch_bounds__(kBwdThreads, 3) ebag_bwd_kernel(const BwdParams p) {
    if (p.only_if && *p.only_if == 0) return;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // per warp: kCacheFloats floats of sums, then kHotSlots ids and kHotSlots flags; after all
    // warps: item_base[T+1]
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    float* cache = reinterpret_cast<float*>(smem_raw) + (size_t)wid * kCacheFloats;
    int* hot_s = reinterpret_cast<int*>(smem_raw + (size_t)kBwdWarps * kCacheFloats * sizeof(float)) +
                 wid * 2 * kHotSlots;                                     // [ids | touched]
    int* item_base = reinterpret_cast<int*>(smem_raw + (size_t)kBwdWarps * kCacheFloats * sizeof(float)) +
                     kBwdWarps * 2 * kHotSlots;                           // [T+1] first item of each table
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
    const int64_t warps = (int64_t)gridDim.x * kBwdWarps;
    unsigned n_oob = 0, n_bad = 0;
    int cur_t = -1;                       // table whose hot rows this warp holds (-1: none)
    int cur_K = 0;                        // its slots in use (0: not cached)

    // sends the warp's cached sums of table `t` to the gradient table
    auto flush = [&](int t, int K) {
        const BwdTableMeta m = p.meta[t];
        float* __restrict__ gt = p.grad_tables[t];
        for (int k = 0; k < K; ++k) {
            const int row = hot_s[k];
            if (row < 0 || !hot_s[kHotSlots + k]) continue;
            for (int vec = lane; vec < m.nvec; vec += 32) {
                const float4 x = *reinterpret_cast<const float4*>(cache + (size_t)k * m.D + vec * 4);
                red_add_v4(gt + row * (int64_t)m.D + vec * 4, x.x, x.y, x.z, x.w);
            }
        }
    };

    for (int64_t item = (int64_t)blockIdx.x * kBwdWarps + wid; item < total; item += warps) {
        int lo_t = 0, hi_t = p.T;
        while (hi_t - lo_t > 1) {
            const int mid = (lo_t + hi_t) >> 1;
            if (item_base[mid] <= item) lo_t = mid; else hi_t = mid;
        }
        const int t = lo_t;
        const BwdTableMeta m = p.meta[t];
        if (t != cur_t) {                 // a new table: hand in the old sums, learn the new hot rows
            __syncwarp();
            if (cur_t >= 0 && cur_K > 0) flush(cur_t, cur_K);
            __syncwarp();
            cur_t = t;
            cur_K = 0;
            if (p.use_cache && m.D <= kCacheFloats) {
                cur_K = 1;
                while (cur_K * 2 <= kHotUse && cur_K * 2 * m.D <= kCacheFloats) cur_K *= 2;
                hot_s[lane] = p.hot[t * kHotSlots + lane];                 // kHotSlots == 32 lanes
                hot_s[kHotSlots + lane] = 0;
                for (int i = lane; i < cur_K * m.D / 4; i += 32)
                    reinterpret_cast<float4*>(cache)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            __syncwarp();
        }
        const int G = 1 << m.g_log2, ng = 32 >> m.g_log2;
        const int lig = lane & (G - 1), grp = lane >> m.g_log2;
        const unsigned leaders = ng > 1 ? 0xffffffffu / ((1u << G) - 1u) : 1u;   // first lane of every group
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
            // the ids of the next batch are requested before the current batch is worked on
            int64_t rn[kIdBatch];
            float wn[kIdBatch];
            auto fetch = [&](int64_t j0) {
#pragma unroll
                for (int k = 0; k < kIdBatch; ++k) {
                    const int64_t i = lo + j0 + k;
                    rn[k] = -1;
                    wn[k] = 1.0f;
                    if (j0 + k < L) {
                        rn[k] = load_id(p.indices, p.idx32, i);
                        if (WEIGHTED) wn[k] = __ldg(p.weights + i);
                    }
                }
            };
            fetch(0);
            for (int64_t j0 = 0; j0 < Lmax; j0 += kIdBatch) {
                int64_t r[kIdBatch];
                float w[kIdBatch];
#pragma unroll
                for (int k = 0; k < kIdBatch; ++k) {
                    r[k] = rn[k];
                    w[k] = wn[k];
                }
                fetch(j0 + kIdBatch);
                auto add_hot = [&](int slot, int k) {
                    float* crow = cache + (size_t)slot * m.D;
#pragma unroll
                    for (int v = 0; v < kTileVecs; ++v)
                        if (on[v]) {
                            float4* a = reinterpret_cast<float4*>(crow + (size_t)(c0 + v * G + lig) * 4);
                            const float ww = WEIGHTED ? w[k] : 1.0f;
                            float4 c = *a;
                            c.x += ww * gv[v].x; c.y += ww * gv[v].y; c.z += ww * gv[v].z; c.w += ww * gv[v].w;
                            *a = c;
                        }
                };
#pragma unroll
                for (int k = 0; k < kIdBatch; ++k) {
                    // (no lane leaves this iteration early: the groups of a warp vote below)
                    const bool live = j0 + k < L;
                    const bool valid = live && (uint64_t)r[k] < (uint64_t)m.rows;
                    if (live && !valid && lig == 0 && c0 == 0) ++n_oob;
                    int slot = -1;
                    if (valid && cur_K > 0) {
                        const int h1 = hot_slot((uint32_t)r[k], cur_K), h2 = hot_slot2((uint32_t)r[k], cur_K);
                        if (hot_s[h1] == (int)r[k]) slot = h1;
                        else if (hot_s[h2] == (int)r[k]) slot = h2;
                    }
                    // A hot row is summed here, in this warp's shared memory.  A lane owns its
                    // columns, so within one group of lanes the sums need no atomics; groups that
                    // run side by side and hit the same row at the same step take turns.
                    if (slot >= 0 && lig == 0) hot_s[kHotSlots + slot] = 1;
                    if (ng > 1) {
                        if (__any_sync(0xffffffffu, slot >= 0)) {
                            const unsigned same = __match_any_sync(0xffffffffu, slot);
                            // groups before mine that want the same slot
                            const int rank = slot >= 0 ? __popc(same & leaders & ((1u << (grp << m.g_log2)) - 1u)) : 0;
                            const int turns = __reduce_max_sync(0xffffffffu, (unsigned)rank);
                            for (int turn = 0; turn <= turns; ++turn) {
                                if (slot >= 0 && rank == turn) add_hot(slot, k);
                                __syncwarp();
                            }
                        }
                    } else if (slot >= 0) {
                        add_hot(slot, k);
                    }
                    if (slot >= 0 || !valid) continue;
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
    __syncwarp();
    if (cur_t >= 0 && cur_K > 0) flush(cur_t, cur_K);
    n_oob = __reduce_add_sync(0xffffffffu, n_oob);
    n_bad = __reduce_add_sync(0xffffffffu, n_bad);
    if (lane == 0) {
        if (n_oob) atomicAdd(&p.status->n_oob, (unsigned long long)n_oob);
        if (n_bad) atomicAdd(&p.status->n_bad_offsets, (unsigned long long)n_bad);
    }
}

template <typename K>
cudaError_t allow_smem(K kernel, size_t bytes) {
    return cudaFuncSetAttribute(reinterpret_cast<const void*>(kernel),
                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace

size_t bwd_smem_bytes(int T) {
    return (size_t)kBwdWarps * kCacheFloats * sizeof(float) + (size_t)kBwdWarps * 2 * kHotSlots * sizeof(int) +
           (size_t)(T + 1) * sizeof(int);
}

cudaError_t launch_bwd(const BwdParams& p, bool weighted, int grid, cudaStream_t s) {
    if (p.use_cache) {
        bwd_hot_rows_kernel<<<p.T, kBwdThreads, 0, s>>>(p);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    const size_t smem = bwd_smem_bytes(p.T);
    if (weighted) ebag_bwd_kernel<true><<<grid, kBwdThreads, smem, s>>>(p);
    else ebag_bwd_kernel<false><<<grid, kBwdThreads, smem, s>>>(p);
    return cudaGetLastError();
}

cudaError_t occupancy_bwd(bool weighted, int T, int* ctas_per_sm) {
    const size_t smem = bwd_smem_bytes(T);
    cudaError_t e = weighted ? allow_smem(ebag_bwd_kernel<true>, bwd_smem_bytes(2048))
                             : allow_smem(ebag_bwd_kernel<false>, bwd_smem_bytes(2048));
    if (e != cudaSuccess) return e;
    return weighted ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, ebag_bwd_kernel<true>,
                                                                     kBwdThreads, smem)
                    : cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, ebag_bwd_kernel<false>,
                                                                     kBwdThreads, smem);
}

}  // namespace ebag
