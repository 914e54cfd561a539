// Device code of the pooled embedding-bag forward (sm_100a).
//
// One persistent kernel serves all T tables of a call.  Work is cut into ITEMS: runs of up to 32
// consecutive bags of one table, sized on the device from the offsets array (which is the prefix
// sum of the bag lengths) so that every item gathers about `item_bytes` of rows whatever the
// table's row size and mean bag length (less when the whole call is small, so that every warp
// still gets work).  Warps pull items from a global counter in table-major order, so a table's
// hot rows stay in L2 while that table is being processed and bags of very unequal length are
// balanced dynamically.
//
// Inside an item a warp is split into row groups of G lanes (G*16 bytes cover one row, G in
// {4,8,16,32}, a run-time property of the table; rows above 512 bytes take 2 vectors per lane, in
// column tiles of 1 KB).  Each group owns one bag at a time; the 32/G bags that run side by side
// are picked after sorting the item's bags by length, so the groups finish together.  The lanes
// of a group read G ids (and weights) of their bag with one coalesced load, two chunks ahead of
// use; each id is then broadcast inside the group with a shuffle and the row is requested with
// 16-byte cp.async copies (through L1) into a per-warp two-stage ring in shared memory, one
// stage (4 row vectors per lane) ahead of the stage being accumulated.  Row fetches therefore
// stay in flight across stage, id-chunk and bag boundaries and occupy no registers.  Widening
// (bf16/fp16), rowwise-int8 dequantisation and the per-sample weight are fused into the fp32
// accumulation; the result is written once with 128-bit streaming stores.
//
// Ids outside the table and malformed bags never fault: they are skipped, counted and reported
// through the handle's status words.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#ifndef EBAG_MIN_BLOCKS
#define EBAG_MIN_BLOCKS 4
#endif

namespace ebag {

enum : int { DT_F32 = 0, DT_F16 = 1, DT_BF16 = 2, DT_INT8 = 3 };

constexpr int kThreads = 256;            // 8 warps per CTA
constexpr int kWarps = kThreads / 32;
constexpr int kMaxItemBags = 32;         // an item's offsets live in one register per lane
constexpr int kItemsPerWarp = 4;         // small calls: aim for at least this many items per warp
constexpr float kSortedItemFactor = 4.0f; // item size multiplier for tables with several bags per warp
constexpr uint32_t kInvalidRow = 0xFFFFFFFFu;

struct TableMeta {       // per table, built at create, lives in device memory
    int64_t rows;
    int32_t D;
    int32_t D_off;       // first output column of this table
    int32_t stride;      // bytes between stored rows
    int32_t nvec;        // 16-byte vectors of payload per row (int8: of codes)
    int32_t g_log2;      // log2 of lanes per row group
    int32_t V;           // vectors per lane (1 or 2); nvec > 64 is walked in 1 KB column tiles
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
    const int64_t* const* mappings;   // MapId variant: device [T] sorted id lists (else unused)
    const int64_t* mapping_len;       // MapId variant: device [T] their lengths
    int64_t n_indices;
    int64_t B;                   // bags per table in this launch
    int64_t off_stride;          // offsets of table t start at offsets[t * off_stride] (B for a
                                 // whole call; the full B when a launch covers a range of bags)
    int32_t T;
    int32_t sumD;
    int32_t mean;                // 1: divide by the bag length
    uint32_t item_bytes;
};

// ------------------------------------------------------------------ memory access helpers
__device__ __forceinline__ int64_t ld_stream_i64(const int64_t* p) {
    // ids and offsets are read once: streaming (evict-first) so they do not displace table rows
    return __ldcs(reinterpret_cast<const long long*>(p));
}
__device__ __forceinline__ float ld_stream_f32(const float* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream16(float* p, float a, float b, float c, float d) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(a, b, c, d));
}

// Asynchronous copies global -> shared (through L1, so hot rows still hit there): the data does
// not occupy registers while it is in flight.
// (`smem` is an address in the shared window, from __cvta_generic_to_shared)
__device__ __forceinline__ void cp_async16(uint32_t smem, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem), "l"(gmem));
}
__device__ __forceinline__ void cp_async8(uint32_t smem, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

__device__ __forceinline__ int64_t shfl64(int64_t v, int src) {
    int lo = __shfl_sync(0xffffffffu, (int)(v & 0xffffffffll), src);
    int hi = __shfl_sync(0xffffffffu, (int)(v >> 32), src);
    return ((int64_t)hi << 32) | (uint32_t)lo;
}

// acc += widen(h) for a 16-bit float held in the low half of `h` (mixed-precision add, one
// instruction on sm_100a)
__device__ __forceinline__ void add_bf16(float& acc, uint32_t h) {
    asm("add.rn.f32.bf16 %0, %1, %0;" : "+f"(acc) : "h"((unsigned short)h));
}
__device__ __forceinline__ void add_f16(float& acc, uint32_t h) {
    asm("add.rn.f32.f16 %0, %1, %0;" : "+f"(acc) : "h"((unsigned short)h));
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
            if constexpr (WEIGHTED) {
                acc[2 * i] = fmaf(w, __uint_as_float(r[i] << 16), acc[2 * i]);
                acc[2 * i + 1] = fmaf(w, __uint_as_float(r[i] & 0xffff0000u), acc[2 * i + 1]);
            } else {
                add_bf16(acc[2 * i], r[i]);
                add_bf16(acc[2 * i + 1], r[i] >> 16);
            }
        }
    } else if constexpr (DT == DT_F16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if constexpr (WEIGHTED) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&r[i]));
                acc[2 * i] = fmaf(w, f.x, acc[2 * i]);
                acc[2 * i + 1] = fmaf(w, f.y, acc[2 * i + 1]);
            } else {
                add_f16(acc[2 * i], r[i]);
                add_f16(acc[2 * i + 1], r[i] >> 16);
            }
        }
    } else {
        // Stored code u = q + 128 (0..255).  Dropping the byte into the mantissa of 2^23 gives the
        // float 2^23 + u; subtracting 2^23 + 128 leaves q, exactly, without the conversion pipe.
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float f = __uint_as_float(__byte_perm(r[i], 0x4B000000u, 0x7440 + k));
                acc[4 * i + k] = fmaf(w, f - 8388736.0f, acc[4 * i + k]);
            }
        }
    }
}

// Sort 32 keys, one per lane, in descending order (bitonic network, 15 exchange steps).
__device__ __forceinline__ uint32_t warp_sort_desc(uint32_t v, int lane) {
#pragma unroll
    for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            const uint32_t o = __shfl_xor_sync(0xffffffffu, v, j);
            const bool lower = (lane & j) == 0;
            const bool desc = (lane & k) == 0;
            v = (lower == desc) ? max(v, o) : min(v, o);
        }
    }
    return v;
}

// ------------------------------------------------------------------ MapId (paper Sec. 5.4.1)
// 1-based position of v in the sorted list M, 0 if v is not in it: insertion index by binary
// search, clamp to the last entry, compare.  The search runs a fixed number of branch-free
// halving steps (the bit length of |M|), as the paper's kernel does with its fixed 20.
// (Stepping by fixed powers of two instead was measured 1.9x slower: its probes sit at
// power-of-two strides and collide in the cache sets.)
__device__ __forceinline__ int64_t map_id(const int64_t* __restrict__ M, uint32_t mlen, int steps,
                                          int64_t v) {
    if (mlen == 0) return 0;
    uint32_t lo = 0, hi = mlen;                      // first position with M[pos] >= v is in [lo, hi]
    for (int s = 0; s < steps; ++s) {
        const uint32_t mid = (lo + hi) >> 1;
        const int64_t mv = __ldg(M + (mid < mlen ? mid : mlen - 1));
        const bool active = lo < hi;
        const bool right = mv < v;
        lo = (active && right) ? mid + 1 : lo;
        hi = (active && !right) ? mid : hi;
    }
    const uint32_t idx = lo < mlen ? lo : mlen - 1;
    return __ldg(M + idx) == v ? (int64_t)idx + 1 : 0;
}

// Four searches side by side (independent dependent-load chains overlap): out[k] = map_id(v[k]).
__device__ __forceinline__ void map_id4(const int64_t* __restrict__ M, uint32_t mlen, int steps,
                                        const int64_t (&v)[4], int64_t (&out)[4]) {
    if (mlen == 0) {
#pragma unroll
        for (int k = 0; k < 4; ++k) out[k] = 0;
        return;
    }
    uint32_t lo[4] = {0, 0, 0, 0}, hi[4] = {mlen, mlen, mlen, mlen};
    for (int s = 0; s < steps; ++s) {
        int64_t mv[4];
        uint32_t mid[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            mid[k] = (lo[k] + hi[k]) >> 1;
            mv[k] = __ldg(M + (mid[k] < mlen ? mid[k] : mlen - 1));
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool active = lo[k] < hi[k];
            const bool right = mv[k] < v[k];
            lo[k] = (active && right) ? mid[k] + 1 : lo[k];
            hi[k] = (active && !right) ? mid[k] : hi[k];
        }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t idx = lo[k] < mlen ? lo[k] : mlen - 1;
        out[k] = __ldg(M + idx) == v[k] ? (int64_t)idx + 1 : 0;
    }
}

// ------------------------------------------------------------------ one item, staged in smem
// Bags [bag0, bag0 + cnt) of table t; cnt <= 32.  V vectors per lane; the lanes per row (G) are
// a run-time property of the table so that one instance of this code serves every row width.
// vec0: first 16-byte vector of the column tile this call covers (0 unless the row is wider than
// 64 vectors).  Rows travel with cp.async into this warp's ring `wbuf` of kStages stages
// (kStageVecs 16-byte vectors per lane each) and are consumed one stage behind.  Every lane reads
// back only the slots it copied itself, so its own wait_group is all the synchronisation the row
// data needs (the int8 scale/bias slots are shared by a group and take a __syncwarp).
#ifndef EBAG_STAGE_VECS
#define EBAG_STAGE_VECS 4
#endif
constexpr int kStageVecs = EBAG_STAGE_VECS;      // 16-byte vectors per lane per stage
constexpr int kStages = 2;

struct IdChunk {          // ids of up to G consecutive entries of the bags one slot works on
    uint32_t r;           // per lane: validated row id of entry `lig`, or kInvalidRow
    float w;              // per lane: its weight
    int nmax;             // warp-uniform: most entries any group has in this chunk
    int nmin;             // warp-uniform: fewest
    bool clean;           // warp-uniform: no id was rejected (set when the chunk is first requested)
    int slot;             // warp-uniform
    bool last;            // warp-uniform: last chunk of its slot
    bool valid;
};

template <int DT, bool WEIGHTED, bool MAPID, int V>
__device__ __forceinline__ void process_item(const FwdParams& p, const TableMeta& m,
                                                   const char* __restrict__ tbase, int t,
                                                   int64_t bag0, int cnt, int vec0, int lane,
                                                   unsigned& n_oob, unsigned& n_bad,
                                                   uint4* __restrict__ wbuf,
                                                   float2* __restrict__ sbbuf) {
    constexpr int NACC = Elem<DT>::kAcc;
    constexpr int CR = kStageVecs / V;               // rows per stage
    const int G = 1 << m.g_log2;
    const int NG = 32 >> m.g_log2;
    const int lig = lane & (G - 1);
    const int grp = lane >> m.g_log2;
    const int64_t g0 = (int64_t)t * p.off_stride + bag0;

    const int64_t base_raw = ld_stream_i64(p.offsets + g0);
    const int64_t base = base_raw < 0 ? 0 : (base_raw > p.n_indices ? p.n_indices : base_raw);
    const int64_t room = p.n_indices - base;
    uint32_t off_lo = 0, off_hi = 0;
    uint32_t key = (uint32_t)lane;
    if (lane < cnt) {
        const int64_t lo = ld_stream_i64(p.offsets + g0 + lane) - base;
        const int64_t hi = ld_stream_i64(p.offsets + g0 + lane + 1) - base;
        if (base_raw != base || lo < 0 || hi < lo || hi > room || hi > 0x7fffffffll) {
            if (vec0 == 0) ++n_bad;
        } else {
            off_lo = (uint32_t)lo;
            off_hi = (uint32_t)hi;
        }
        const uint32_t len = off_hi - off_lo;
        key = (((len > 0x3FFFFFEu ? 0x3FFFFFEu : len) + 1u) << 5) | (uint32_t)lane;
    }
    if (NG > 1 && cnt > NG) key = warp_sort_desc(key, lane);
    const int64_t* __restrict__ idx_base = p.indices + base;
    const float* __restrict__ w_base = WEIGHTED ? p.weights + base : nullptr;

    bool col_on[V];
    const char* lane_base[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int vec = vec0 + v * G + lig;
        col_on[v] = vec < m.nvec;
        lane_base[v] = tbase + vec * 16;
    }
    const uint32_t stride = (uint32_t)m.stride;
    const uint64_t rows = (uint64_t)m.rows;
    const char* sb_base = tbase + m.D;
    const int nslots = (cnt + NG - 1) >> (5 - m.g_log2);

    const int64_t* __restrict__ map_ptr = MAPID ? p.mappings[t] : nullptr;
    const int64_t map_len64 = MAPID ? p.mapping_len[t] : 0;
    const uint32_t map_len = (uint32_t)(map_len64 < 0 ? 0 : map_len64);
    const int map_steps = 32 - __clz(map_len);
    auto load_chunk = [&](uint32_t pos, uint32_t end, uint32_t& ridx, float& w) {
        ridx = kInvalidRow;
        w = 0.0f;
        const uint32_t i = pos + lig;
        if (i < end) {
            int64_t r = ld_stream_i64(idx_base + i);
            float wl = 1.0f;
            if (WEIGHTED) wl = ld_stream_f32(w_base + i);
            if (MAPID) r = map_id(map_ptr, map_len, map_steps, r);     // raw id -> row
            if ((uint64_t)r < rows) {
                ridx = (uint32_t)r;
                w = wl;
            } else if (vec0 == 0) {
                ++n_oob;
            }
        }
    };
    auto slot_bag = [&](int pos_in_item, uint32_t& s, uint32_t& e, int& orig) {
        const uint32_t k = __shfl_sync(0xffffffffu, key, pos_in_item & 31);
        orig = (int)(k & 31u);
        s = __shfl_sync(0xffffffffu, off_lo, orig);
        e = __shfl_sync(0xffffffffu, off_hi, orig);
        if (pos_in_item >= cnt) s = e = 0;
    };

    // ---- generator of id chunks, in the order they are consumed
    int gslot = -1;
    uint32_t ge = 0, gpos = 0;
    bool gmore = false;
    auto gen = [&](IdChunk& c) {
        if (gslot >= 0 && gmore) {
            gpos += G;
        } else {
            ++gslot;
            if (gslot >= nslots) {
                c.valid = false;
                return;
            }
            uint32_t gs;
            int o;
            slot_bag(gslot * NG + grp, gs, ge, o);
            gpos = gs;
        }
        load_chunk(gpos, ge, c.r, c.w);
        const uint32_t left = ge - gpos;
        const int nval = left > (uint32_t)G ? G : (int)left;
        c.nmax = __reduce_max_sync(0xffffffffu, nval);
        c.nmin = __reduce_min_sync(0xffffffffu, nval);
        c.clean = false;
        gmore = __any_sync(0xffffffffu, gpos + G < ge);
        c.slot = gslot;
        c.last = !gmore;
        c.valid = true;
    };

    // ---- request / use one stage (CR rows of chunk c starting at entry j0)
    bool my_cols = true;
#pragma unroll
    for (int v = 0; v < V; ++v) my_cols = my_cols && col_on[v];
    const bool cols_full = __all_sync(0xffffffffu, my_cols);
    // this lane's slots: vector k of stage st is at my_rows[(st * kStageVecs + k) * 32]
    const uint4* my_rows = wbuf + lane;
    const uint32_t my_rows_s = (uint32_t)__cvta_generic_to_shared(wbuf) + lane * 16;
    const float2* my_sb = sbbuf + grp;               // int8: scale/bias of row u at [(st*kStageVecs+u)*8]
    const uint32_t my_sb_s = (uint32_t)__cvta_generic_to_shared(sbbuf) + grp * 8;
    auto issue = [&](const IdChunk& c, int j0, int st) {
        if (c.clean && j0 + CR <= c.nmin) {          // full stage, nothing to check
#pragma unroll
            for (int u = 0; u < CR; ++u) {
                const uint32_t r = __shfl_sync(0xffffffffu, c.r, j0 + u, G);
                const uint64_t roff = (uint64_t)r * stride;
#pragma unroll
                for (int v = 0; v < V; ++v)
                    cp_async16(my_rows_s + (st * kStageVecs + u * V + v) * 512, lane_base[v] + roff);
                if (DT == DT_INT8 && lig == 0)
                    cp_async8(my_sb_s + (st * kStageVecs + u) * 64, sb_base + roff);
            }
            return;
        }
#pragma unroll
        for (int u = 0; u < CR; ++u) {
            const uint32_t r = __shfl_sync(0xffffffffu, c.r, j0 + u, G);
            if (j0 + u < c.nmax && r != kInvalidRow) {
                const uint64_t roff = (uint64_t)r * stride;
#pragma unroll
                for (int v = 0; v < V; ++v)
                    if (col_on[v])
                        cp_async16(my_rows_s + (st * kStageVecs + u * V + v) * 512, lane_base[v] + roff);
                if (DT == DT_INT8 && lig == 0)
                    cp_async8(my_sb_s + (st * kStageVecs + u) * 64, sb_base + roff);
            }
        }
    };
    float acc[V][NACC];
    float acc_bias = 0.0f;
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int a = 0; a < NACC; ++a) acc[v][a] = 0.0f;
    auto consume = [&](const IdChunk& c, int j0, int st) {
        if (c.clean && j0 + CR <= c.nmin) {
#pragma unroll
            for (int u = 0; u < CR; ++u) {
                float wu = WEIGHTED ? __shfl_sync(0xffffffffu, c.w, j0 + u, G) : 1.0f;
                if (DT == DT_INT8) {
                    const float2 sb = my_sb[(st * kStageVecs + u) * 8];
                    acc_bias = fmaf(wu, sb.y, acc_bias);
                    wu *= sb.x;
                }
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const uint4 d = my_rows[(st * kStageVecs + u * V + v) * 32];
                    accumulate<DT, WEIGHTED || DT == DT_INT8>(acc[v], d, wu);
                }
            }
            return;
        }
#pragma unroll
        for (int u = 0; u < CR; ++u) {
            const uint32_t r = __shfl_sync(0xffffffffu, c.r, j0 + u, G);
            float wu = WEIGHTED ? __shfl_sync(0xffffffffu, c.w, j0 + u, G) : 1.0f;
            if (j0 + u < c.nmax && r != kInvalidRow) {
                if (DT == DT_INT8) {
                    const float2 sb = my_sb[(st * kStageVecs + u) * 8];
                    acc_bias = fmaf(wu, sb.y, acc_bias);
                    wu *= sb.x;
                }
#pragma unroll
                for (int v = 0; v < V; ++v)
                    if (col_on[v]) {
                        const uint4 d = my_rows[(st * kStageVecs + u * V + v) * 32];
                        accumulate<DT, WEIGHTED || DT == DT_INT8>(acc[v], d, wu);
                    }
            }
        }
    };
    auto finalize = [&](int slot) {
        uint32_t s, e;
        int orig;
        slot_bag(slot * NG + grp, s, e, orig);
        if (slot * NG + grp < cnt) {
            const uint32_t L = e - s;
            float* orow = p.out + (bag0 + orig) * (int64_t)p.sumD + m.D_off;
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
        acc_bias = 0.0f;
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int a = 0; a < NACC; ++a) acc[v][a] = 0.0f;
    };

    // ---- pipeline: the request side runs one stage ahead of the consuming side
    static_assert(kStages == 2, "the consuming side assumes it is exactly one stage behind");
    IdChunk cons, iss, pre;
    gen(iss);                       // nslots >= 1, so the first chunk always exists
    gen(pre);
    int ji = 0;                     // next entry of chunk `iss` to request
    bool iss_done = false;
    // request the next stage (into stage ST) and close its copy group
    auto issue_next = [&](int st) {
        if (!iss_done) {
            if (ji > 0 && ji >= iss.nmax) {              // chunk exhausted: move to the next one
                if (pre.valid) {
                    iss = pre;
                    gen(pre);
                    ji = 0;
                } else {
                    iss_done = true;
                }
            }
            if (!iss_done) {
                if (ji == 0)        // first request of this chunk: its ids are needed now anyway
                    iss.clean = cols_full &&
                                __all_sync(0xffffffffu, lig >= iss.nmin || iss.r != kInvalidRow);
                issue(iss, ji, st);
                ji += CR;
            }
        }
        cp_async_commit();          // one group per step, empty or not, keeps the counting uniform
    };
    int jc = 0;
    issue_next(0);                  // stage 0 of the first chunk (cannot leave that chunk)
    cons = iss;
    int st = 0;                     // stage being consumed; the next request goes to the other one
    while (true) {
        issue_next(st ^ 1);
        cp_async_wait<1>();         // everything but the newest group has landed
        if (DT == DT_INT8) __syncwarp();                 // scale/bias slots are shared by a group
        consume(cons, jc, st);
        if (DT == DT_INT8) __syncwarp();
        jc += CR;
        st ^= 1;
        if (jc >= cons.nmax) {                           // chunk consumed (an empty chunk is one step)
            const bool was_last = cons.last;
            const int slot = cons.slot;
            if (was_last) finalize(slot);
            if (was_last && slot == nslots - 1) break;
            cons = iss;                                  // the request side is already in the next chunk
            jc = 0;
        }
    }
    cp_async_wait<0>();
}

// ------------------------------------------------------------------ the kernel
template <int DT, bool WEIGHTED, bool MAPID>
__global__ void __launch_bounds__(kThreads, EBAG_MIN_BLOCKS)
ebag_fwd_kernel(const FwdParams p) {
    extern __shared__ int smem_i[];
    int* item_base = smem_i;                                   // [T+1] first item of each table
    int* item_bags = smem_i + p.T + 1;                         // [T]   bags per item of each table
    float* bag_bytes = reinterpret_cast<float*>(item_bags);    // [T]   (first pass) bytes per bag
    __shared__ float total_bytes;
    __shared__ uint4 stage_buf[kWarps * kStages * kStageVecs * 32];          // 4 KB per warp
    __shared__ float2 sb_buf[DT == DT_INT8 ? kWarps * kStages * kStageVecs * 8 : 1];
    uint4* wbuf = stage_buf + (threadIdx.x >> 5) * (kStages * kStageVecs * 32);
    float2* sbbuf = sb_buf + (DT == DT_INT8 ? (threadIdx.x >> 5) * (kStages * kStageVecs * 8) : 0);
    const int tid = threadIdx.x;
    const int lane = tid & 31;

    // ---- size the items of every table from its share of the offsets prefix sum
    if (tid == 0) total_bytes = 0.0f;
    __syncthreads();
    for (int t = tid; t < p.T; t += kThreads) {
        const int64_t n0 = p.offsets[(int64_t)t * p.off_stride];
        const int64_t n1 = p.offsets[(int64_t)t * p.off_stride + p.B];
        int64_t nt = n1 - n0;
        if (nt < 0) nt = 0;
        if (nt > p.n_indices) nt = p.n_indices;
        const float bytes = (float)nt * (float)p.meta[t].stride;
        bag_bytes[t] = fmaxf(bytes / (float)p.B, 1.0f);
        atomicAdd(&total_bytes, bytes);
    }
    __syncthreads();
    // small calls: shrink the items so that every warp of the grid gets a few of them
    const float spread = total_bytes / (float)(gridDim.x * kWarps * kItemsPerWarp);
    const float item_bytes = fminf((float)p.item_bytes, spread);
    __syncthreads();
    for (int t = tid; t < p.T; t += kThreads) {
        const int ng = 32 >> p.meta[t].g_log2;
        // bags that run side by side are matched by length inside an item: more bags per item,
        // better matches (measured: cfg 5 6.70 -> 5.75 ms, cfg 3 2.35 -> 2.12 ms)
        const float want = (ng > 1 ? kSortedItemFactor * item_bytes : item_bytes) / bag_bytes[t];
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
    unsigned q = 0;
    if (lane == 0) q = atomicAdd(&p.queue->next, 1u);
    q = __shfl_sync(0xffffffffu, q, 0);
    while (q < total) {
        // ask for the next item now; the answer is needed only after this one is done
        unsigned q_next = 0;
        if (lane == 0) q_next = atomicAdd(&p.queue->next, 1u);

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
            process_item<DT, WEIGHTED, MAPID, 1>(p, m, tbase, t, bag0, cnt, 0, lane, n_oob, n_bad, wbuf, sbbuf);
        } else {
            // rows above 512 bytes: two vectors per lane, 1 KB column tiles
            for (int vec0 = 0; vec0 < m.nvec; vec0 += 64)
                process_item<DT, WEIGHTED, MAPID, 2>(p, m, tbase, t, bag0, cnt, vec0, lane, n_oob, n_bad, wbuf, sbbuf);
        }
        q = __shfl_sync(0xffffffffu, q_next, 0);
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
#define EBAG_DECLARE_LAUNCHERS(NAME)                                                             \
    cudaError_t launch_fwd_##NAME(const FwdParams& p, bool weighted, bool mapid, int grid,        \
                                  size_t smem, cudaStream_t s);                                  \
    cudaError_t occupancy_fwd_##NAME(bool weighted, bool mapid, size_t smem, int* ctas_per_sm);
EBAG_DECLARE_LAUNCHERS(f32)
EBAG_DECLARE_LAUNCHERS(f16)
EBAG_DECLARE_LAUNCHERS(bf16)
EBAG_DECLARE_LAUNCHERS(int8)

#define EBAG_DEFINE_LAUNCHERS(NAME, DT)                                                          \
    cudaError_t launch_fwd_##NAME(const FwdParams& p, bool weighted, bool mapid, int grid,        \
                                  size_t smem, cudaStream_t s) {                                 \
        if (mapid) {                                                                             \
            if (weighted) ebag_fwd_kernel<DT, true, true><<<grid, kThreads, smem, s>>>(p);        \
            else ebag_fwd_kernel<DT, false, true><<<grid, kThreads, smem, s>>>(p);                \
        } else {                                                                                 \
            if (weighted) ebag_fwd_kernel<DT, true, false><<<grid, kThreads, smem, s>>>(p);       \
            else ebag_fwd_kernel<DT, false, false><<<grid, kThreads, smem, s>>>(p);               \
        }                                                                                        \
        return cudaGetLastError();                                                               \
    }                                                                                            \
    cudaError_t occupancy_fwd_##NAME(bool weighted, bool mapid, size_t smem, int* n) {            \
        const void* k = mapid ? (weighted ? (const void*)ebag_fwd_kernel<DT, true, true>          \
                                          : (const void*)ebag_fwd_kernel<DT, false, true>)        \
                              : (weighted ? (const void*)ebag_fwd_kernel<DT, true, false>         \
                                          : (const void*)ebag_fwd_kernel<DT, false, false>);      \
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(n, k, kThreads, smem);              \
    }

}  // namespace ebag
