// Device code of the pooled embedding-bag forward (sm_100a).
//
// One persistent kernel serves all T tables of a call.  Work is cut into ITEMS: runs of
// consecutive bags of one table, sized on the device from the offsets array (which is the prefix
// sum of the bag lengths) so that every item gathers about `item_bytes` of rows whatever the
// table's row size and mean bag length.  Warps pull items from a global counter in table-major
// order, so a table's hot rows stay in L2 while that table is being processed and bags of very
// unequal length are balanced dynamically.
//
// Inside an item a warp is split into row groups of G lanes (G*16 bytes cover one row, G in
// {4,8,16,32}; rows above 512 bytes take V = 2 or 4 vectors per lane).  Each group owns one bag
// at a time.  The lanes of a group read G ids (and weights) of their bag with one coalesced load,
// one chunk ahead of use; each id is then broadcast inside the group with a shuffle and up to
// ROWS_IN_FLIGHT rows are requested with 128-bit loads before the first is consumed.  Widening
// (bf16/fp16), rowwise-int8 dequantisation and the per-sample weight are fused into the fp32
// accumulation; the result is written once with 128-bit streaming stores.
//
// Ids outside the table and malformed bags never fault: they are skipped, counted and reported
// through the handle's status words.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ebag {

enum : int { DT_F32 = 0, DT_F16 = 1, DT_BF16 = 2, DT_INT8 = 3 };

constexpr int kThreads = 256;            // 8 warps per CTA
constexpr int kWarps = kThreads / 32;
constexpr int kMaxItemBags = 32;         // an item's offsets live in one register per lane
constexpr uint32_t kInvalidRow = 0xFFFFFFFFu;

struct TableMeta {       // per table, built at create, lives in device memory
    int64_t rows;
    int32_t D;
    int32_t D_off;       // first output column of this table
    int32_t stride;      // bytes between stored rows
    int32_t nvec;        // 16-byte vectors of payload per row (int8: of codes)
    int32_t g_log2;      // log2 of lanes per row group
    int32_t V;           // vectors per lane (1, 2 or 4); nvec > 32*4 is walked in column tiles
};

struct Queue {           // handle-owned scratch; both zero between launches
    unsigned int next;   // next item to hand out
    unsigned int done;   // CTAs that have left the item loop
};

struct Status {
    unsigned long long n_oob;
    unsigned long long n_bad_offsets;
};

struct FwdParams {
    const void* const* tables;   // device [T]
    const TableMeta* meta;       // device [T]
    const int64_t* indices;
    const int64_t* offsets;
    const float* weights;
    float* out;
    Queue* queue;
    Status* status;
    int64_t n_indices;
    int64_t B;
    int32_t T;
    int32_t sumD;
    int32_t mean;                // 1: divide by the bag length
    uint32_t item_bytes;
};

// ------------------------------------------------------------------ memory access helpers
__device__ __forceinline__ uint4 ld_row16(const void* p) {
    // read-only path, default L1/L2 policy: hot (Zipf) rows are meant to be caught by L1/L2
    return __ldg(reinterpret_cast<const uint4*>(p));
}
__device__ __forceinline__ int64_t ld_stream_i64(const int64_t* p) {
    // ids and offsets are read once: streaming (evict-first) so they do not displace table rows
    return __ldcs(reinterpret_cast<const long long*>(p));
}
__device__ __forceinline__ float ld_stream_f32(const float* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream16(float* p, float a, float b, float c, float d) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(a, b, c, d));
}

__device__ __forceinline__ int64_t shfl64(int64_t v, int src) {
    int lo = __shfl_sync(0xffffffffu, (int)(v & 0xffffffffll), src);
    int hi = __shfl_sync(0xffffffffu, (int)(v >> 32), src);
    return ((int64_t)hi << 32) | (uint32_t)lo;
}

// ------------------------------------------------------------------ per-dtype accumulation
template <int DT> struct Elem;
template <> struct Elem<DT_F32>  { static constexpr int kAcc = 4; };
template <> struct Elem<DT_F16>  { static constexpr int kAcc = 8; };
template <> struct Elem<DT_BF16> { static constexpr int kAcc = 8; };
template <> struct Elem<DT_INT8> { static constexpr int kAcc = 16; };

// acc[0..kAcc) += w * widen(d)        (int8: w is w*scale; the bias term is summed separately)
template <int DT, bool WEIGHTED>
__device__ __forceinline__ void accumulate(float* acc, const uint4& d, float w) {
    const uint32_t r[4] = {d.x, d.y, d.z, d.w};
    if constexpr (DT == DT_F32) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float x = __uint_as_float(r[i]);
            acc[i] = WEIGHTED ? fmaf(w, x, acc[i]) : acc[i] + x;
        }
    } else if constexpr (DT == DT_BF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float lo = __uint_as_float(r[i] << 16);
            const float hi = __uint_as_float(r[i] & 0xffff0000u);
            acc[2 * i] = WEIGHTED ? fmaf(w, lo, acc[2 * i]) : acc[2 * i] + lo;
            acc[2 * i + 1] = WEIGHTED ? fmaf(w, hi, acc[2 * i + 1]) : acc[2 * i + 1] + hi;
        }
    } else if constexpr (DT == DT_F16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&r[i]));
            acc[2 * i] = WEIGHTED ? fmaf(w, f.x, acc[2 * i]) : acc[2 * i] + f.x;
            acc[2 * i + 1] = WEIGHTED ? fmaf(w, f.y, acc[2 * i + 1]) : acc[2 * i + 1] + f.y;
        }
    } else {
        // int8 code q -> float without the conversion pipe: flip the sign bit (u = q + 128),
        // drop the byte into the mantissa of 2^23, subtract 2^23 + 128.  Exact.
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t u = r[i] ^ 0x80808080u;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float f = __uint_as_float(__byte_perm(u, 0x4B000000u, 0x7440 + k));
                const float q = f - 8388736.0f;                     // 2^23 + 128
                acc[4 * i + k] = fmaf(w, q, acc[4 * i + k]);
            }
        }
    }
}

// ------------------------------------------------------------------ one item
// Bags [bag0, bag0 + cnt) of table t; cnt <= 32.  G lanes per row, V vectors per lane.
// vec0: first 16-byte vector of the column tile this call covers (0 unless the row is wider
// than 32*4 vectors).
template <int DT, bool WEIGHTED, int G, int V>
__device__ __forceinline__ void process_item(const FwdParams& p, const TableMeta& m,
                                             const char* __restrict__ tbase, int t, int64_t bag0,
                                             int cnt, int vec0, int lane, unsigned& n_oob,
                                             unsigned& n_bad) {
    constexpr int NG = 32 / G;                       // row groups (bags in progress) per warp
    constexpr int NACC = Elem<DT>::kAcc;
    constexpr int U = (8 / V) < G ? (8 / V) : G;     // rows requested before the first is used
    const int lig = lane & (G - 1);
    const int grp = lane / G;
    const int64_t g0 = (int64_t)t * p.B + bag0;

    // the item's offsets: lane i holds the bounds of bag i
    int64_t off_lo = 0, off_hi = 0;
    if (lane < cnt) {
        off_lo = ld_stream_i64(p.offsets + g0 + lane);
        off_hi = ld_stream_i64(p.offsets + g0 + lane + 1);
        if (off_hi < off_lo || off_lo < 0 || off_hi > p.n_indices) {
            if (vec0 == 0) ++n_bad;
            off_lo = off_hi = 0;
        }
    }

    bool col_on[V];
    int col_byte[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int vec = vec0 + v * G + lig;
        col_on[v] = vec < m.nvec;
        col_byte[v] = vec * 16;
    }
    const uint32_t stride = (uint32_t)m.stride;
    const uint64_t rows = (uint64_t)m.rows;

    // ids (validated, narrowed to 32 bits) and weights of one chunk: lane `lig` of a group
    // holds entry pos + lig of the group's bag
    auto load_chunk = [&](int64_t pos, int64_t end, uint32_t& ridx, float& w) {
        ridx = kInvalidRow;
        w = 0.0f;
        const int64_t i = pos + lig;
        if (i < end) {
            const int64_t r = ld_stream_i64(p.indices + i);
            float wl = 1.0f;
            if (WEIGHTED) wl = ld_stream_f32(p.weights + i);
            if ((uint64_t)r < rows) {
                ridx = (uint32_t)r;
                w = wl;
            } else if (vec0 == 0) {
                ++n_oob;
            }
        }
    };

    const int nslots = (cnt + NG - 1) / NG;
    int slot = 0;
    int64_t s, e;
    {
        const int j = grp;                            // slot 0
        s = shfl64(off_lo, j < cnt ? j : 0);
        e = shfl64(off_hi, j < cnt ? j : 0);
        if (j >= cnt) s = e = 0;
    }
    int64_t pos = s;
    uint32_t cur_r, nxt_r = kInvalidRow;
    float cur_w, nxt_w = 0.0f;
    load_chunk(pos, e, cur_r, cur_w);

    float acc[V][NACC];
    float acc_bias = 0.0f;                            // int8: sum of w * bias[row]
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int a = 0; a < NACC; ++a) acc[v][a] = 0.0f;

    while (true) {
        // ---- prefetch the ids of the next chunk (same bag, or first chunk of the next slot)
        const int64_t pos_next = pos + G;
        const bool more = __any_sync(0xffffffffu, pos_next < e);
        int64_t s2 = 0, e2 = 0;
        if (more) {
            load_chunk(pos_next, e, nxt_r, nxt_w);
        } else if (slot + 1 < nslots) {
            const int j = (slot + 1) * NG + grp;
            s2 = shfl64(off_lo, j < cnt ? j : 0);
            e2 = shfl64(off_hi, j < cnt ? j : 0);
            if (j >= cnt) s2 = e2 = 0;
            load_chunk(s2, e2, nxt_r, nxt_w);
        }

        // ---- gather and accumulate the rows of the current chunk
        int64_t left = e - pos;
        const int nval = left <= 0 ? 0 : (left > G ? G : (int)left);
        const int nmax = __reduce_max_sync(0xffffffffu, nval);
#pragma unroll
        for (int j0 = 0; j0 < G; j0 += U) {
            if (j0 < nmax) {
                uint32_t r[U];
                float w[U];
                uint4 d[U][V];
                float sb[U][2];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    r[u] = __shfl_sync(0xffffffffu, cur_r, j0 + u, G);
                    w[u] = WEIGHTED ? __shfl_sync(0xffffffffu, cur_w, j0 + u, G) : 1.0f;
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const char* row = tbase + (uint64_t)r[u] * stride;
                    const bool ok = r[u] != kInvalidRow;
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        d[u][v] = make_uint4(0u, 0u, 0u, 0u);
                        if (ok && col_on[v]) d[u][v] = ld_row16(row + col_byte[v]);
                    }
                    if (DT == DT_INT8) {
                        sb[u][0] = 0.0f;
                        sb[u][1] = 0.0f;
                        if (ok) {
                            const float2 c = __ldg(reinterpret_cast<const float2*>(row + m.D));
                            sb[u][0] = c.x;
                            sb[u][1] = c.y;
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    float wu = w[u];
                    if (!WEIGHTED && r[u] == kInvalidRow) wu = 0.0f;
                    if (DT == DT_INT8) {
                        acc_bias = fmaf(wu, sb[u][1], acc_bias);
                        wu *= sb[u][0];
                    }
#pragma unroll
                    for (int v = 0; v < V; ++v) accumulate<DT, WEIGHTED || DT == DT_INT8>(acc[v], d[u][v], wu);
                }
            }
        }

        if (more) {
            pos = pos_next;
        } else {
            // ---- the bags of this slot are complete: finalise and store
            const int j = slot * NG + grp;
            if (j < cnt) {
                const int64_t L = e - s;
                float* orow = p.out + (bag0 + j) * (int64_t)p.sumD + m.D_off;
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    if (!col_on[v]) continue;
                    float* o = orow + (size_t)(vec0 + v * G + lig) * NACC;
#pragma unroll
                    for (int a = 0; a < NACC; ++a) {
                        float x = acc[v][a];
                        if (DT == DT_INT8) x += acc_bias;
                        if (p.mean && L > 0) x = __fdiv_rn(x, (float)L);
                        acc[v][a] = x;
                    }
#pragma unroll
                    for (int a = 0; a < NACC; a += 4)
                        st_stream16(o + a, acc[v][a], acc[v][a + 1], acc[v][a + 2], acc[v][a + 3]);
                }
            }
            ++slot;
            if (slot >= nslots) break;
            s = s2;
            e = e2;
            pos = s;
            acc_bias = 0.0f;
#pragma unroll
            for (int v = 0; v < V; ++v)
#pragma unroll
                for (int a = 0; a < NACC; ++a) acc[v][a] = 0.0f;
        }
        cur_r = nxt_r;
        cur_w = nxt_w;
    }
}

// ------------------------------------------------------------------ the kernel
template <int DT, bool WEIGHTED>
__global__ void __launch_bounds__(kThreads)
ebag_fwd_kernel(const FwdParams p) {
    extern __shared__ int smem_i[];
    int* item_base = smem_i;                 // [T+1] first item of each table
    int* item_bags = smem_i + p.T + 1;       // [T]   bags per item of each table
    const int tid = threadIdx.x;
    const int lane = tid & 31;

    // ---- size the items of every table from its share of the offsets prefix sum
    for (int t = tid; t < p.T; t += kThreads) {
        const TableMeta m = p.meta[t];
        const int64_t n0 = p.offsets[(int64_t)t * p.B];
        const int64_t n1 = p.offsets[(int64_t)(t + 1) * p.B];
        int64_t nt = n1 - n0;
        if (nt < 0) nt = 0;
        if (nt > p.n_indices) nt = p.n_indices;
        const int ng = 32 >> m.g_log2;
        const float mean_len = (float)nt / (float)p.B;
        const float want = (float)p.item_bytes / ((float)m.stride * fmaxf(mean_len, 1e-6f));
        int ib = want >= (float)kMaxItemBags ? kMaxItemBags : (int)want;
        ib = (ib / ng) * ng;
        if (ib < ng) ib = ng;
        item_bags[t] = ib;
        item_base[t + 1] = (int)((p.B + ib - 1) / ib);
    }
    __syncthreads();
    if (tid < 32) {                           // exclusive scan of the item counts (warp 0)
        int carry = 0;
        for (int t0 = 0; t0 < p.T; t0 += 32) {
            const int t = t0 + lane;
            int x = t < p.T ? item_base[t + 1] : 0;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, x, d);
                if (lane >= d) x += y;
            }
            if (t < p.T) item_base[t + 1] = carry + x;
            carry += __shfl_sync(0xffffffffu, x, 31);
        }
        if (lane == 0) item_base[0] = 0;
    }
    __syncthreads();
    const unsigned total = (unsigned)item_base[p.T];

    unsigned n_oob = 0, n_bad = 0;
    while (true) {
        unsigned q = 0;
        if (lane == 0) q = atomicAdd(&p.queue->next, 1u);
        q = __shfl_sync(0xffffffffu, q, 0);
        if (q >= total) break;
        // table of item q: last t with item_base[t] <= q
        int lo = 0, hi = p.T;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if ((unsigned)item_base[mid] <= q) lo = mid; else hi = mid;
        }
        const int t = lo;
        const TableMeta m = p.meta[t];
        const int ib = item_bags[t];
        const int64_t bag0 = (int64_t)(q - (unsigned)item_base[t]) * ib;
        const int64_t rest = p.B - bag0;
        const int cnt = rest < ib ? (int)rest : ib;
        const char* tbase = static_cast<const char*>(p.tables[t]);

        if (m.V == 1) {
            switch (m.g_log2) {
                case 2: process_item<DT, WEIGHTED, 4, 1>(p, m, tbase, t, bag0, cnt, 0, lane, n_oob, n_bad); break;
                case 3: process_item<DT, WEIGHTED, 8, 1>(p, m, tbase, t, bag0, cnt, 0, lane, n_oob, n_bad); break;
                case 4: process_item<DT, WEIGHTED, 16, 1>(p, m, tbase, t, bag0, cnt, 0, lane, n_oob, n_bad); break;
                default: process_item<DT, WEIGHTED, 32, 1>(p, m, tbase, t, bag0, cnt, 0, lane, n_oob, n_bad); break;
            }
        } else if (m.V == 2) {
            process_item<DT, WEIGHTED, 32, 2>(p, m, tbase, t, bag0, cnt, 0, lane, n_oob, n_bad);
        } else {
            if constexpr (DT == DT_INT8) {
                for (int vec0 = 0; vec0 < m.nvec; vec0 += 64)
                    process_item<DT, WEIGHTED, 32, 2>(p, m, tbase, t, bag0, cnt, vec0, lane, n_oob, n_bad);
            } else {
                for (int vec0 = 0; vec0 < m.nvec; vec0 += 128)
                    process_item<DT, WEIGHTED, 32, 4>(p, m, tbase, t, bag0, cnt, vec0, lane, n_oob, n_bad);
            }
        }
    }

    // ---- report what was skipped; the last CTA out re-arms the queue for the next launch
    n_oob = __reduce_add_sync(0xffffffffu, n_oob);
    n_bad = __reduce_add_sync(0xffffffffu, n_bad);
    if (lane == 0) {
        if (n_oob) atomicAdd(&p.status->n_oob, (unsigned long long)n_oob);
        if (n_bad) atomicAdd(&p.status->n_bad_offsets, (unsigned long long)n_bad);
    }
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned prev = atomicAdd(&p.queue->done, 1u);
        if (prev == gridDim.x - 1) {
            p.queue->next = 0;
            p.queue->done = 0;
            __threadfence();
        }
    }
}

// one launcher per dtype, each compiled in its own translation unit
cudaError_t launch_fwd_f32(const FwdParams& p, bool weighted, int grid, size_t smem, cudaStream_t s);
cudaError_t launch_fwd_f16(const FwdParams& p, bool weighted, int grid, size_t smem, cudaStream_t s);
cudaError_t launch_fwd_bf16(const FwdParams& p, bool weighted, int grid, size_t smem, cudaStream_t s);
cudaError_t launch_fwd_int8(const FwdParams& p, bool weighted, int grid, size_t smem, cudaStream_t s);
cudaError_t occupancy_fwd_f32(bool weighted, size_t smem, int* ctas_per_sm);
cudaError_t occupancy_fwd_f16(bool weighted, size_t smem, int* ctas_per_sm);
cudaError_t occupancy_fwd_bf16(bool weighted, size_t smem, int* ctas_per_sm);
cudaError_t occupancy_fwd_int8(bool weighted, size_t smem, int* ctas_per_sm);

#define EBAG_DEFINE_LAUNCHERS(NAME, DT)                                                          \
    cudaError_t launch_fwd_##NAME(const FwdParams& p, bool weighted, int grid, size_t smem,       \
                                  cudaStream_t s) {                                              \
        if (weighted) ebag_fwd_kernel<DT, true><<<grid, kThreads, smem, s>>>(p);                  \
        else ebag_fwd_kernel<DT, false><<<grid, kThreads, smem, s>>>(p);                          \
        return cudaGetLastError();                                                               \
    }                                                                                            \
    cudaError_t occupancy_fwd_##NAME(bool weighted, size_t smem, int* n) {                        \
        return weighted ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(                         \
                              n, ebag_fwd_kernel<DT, true>, kThreads, smem)                       \
                        : cudaOccupancyMaxActiveBlocksPerMultiprocessor(                         \
                              n, ebag_fwd_kernel<DT, false>, kThreads, smem);                     \
    }

}  // namespace ebag
