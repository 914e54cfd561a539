// Device code of the pooled embedding-bag forward (sm_100a).
//
// One persistent kernel serves all T tables of a call.  Work is cut into ITEMS: runs of up to 32
// consecutive bags of one table, sized on the device from the offsets array (which is the prefix
// sum of the bag lengths) so that an item gathers about `item_bytes` of rows (eight times that
// for rows of one vector per lane; less for the last tables of a call and when the whole call is
// small, so that every warp still gets work and the slowest one finishes soon after the rest).
// Warps pull items from a global counter in table-major order, so a table's hot rows stay in L2
// while that table is being processed and bags of very unequal length are balanced dynamically.
// A bag too long for one warp is not pooled here: it is recorded, and a second, short kernel
// (ebag_parts_kernel, below) pools the recorded bags in parts over the whole grid.
//
// Inside an item a warp is split into row groups of G lanes (G*16 bytes cover one row, G in
// {4,8,16,32}, a run-time property of the table; rows above 512 bytes take 2 vectors per lane, in
// column tiles of 1 KB).  Each group owns one bag at a time; the 32/G bags that run side by side
// are picked after sorting the item's bags by length, so the groups finish together (the bags'
// ranges and the sorted order sit in shared memory).  The lanes of a group read G ids (and
// weights) of their bag with one coalesced load, two chunks ahead of use; each id is then
// broadcast inside the group with a shuffle and the row is requested with 16-byte cp.async
// copies (through L1: the hot rows of a skewed workload are served from there, bypassing it was
// measured five times slower) into a per-warp two-stage ring in shared memory, one stage (4 row
// vectors per lane) ahead of the stage being accumulated.  Row fetches therefore stay in flight
// across stage, id-chunk and bag boundaries and occupy no registers.  Widening (bf16/fp16),
// rowwise 8-bit dequantisation and the per-sample weight are fused into the fp32 accumulation
// (or the element-wise maximum, for max pooling); the result is written once with streaming
// stores, as fp32 or rounded to fp16 / bf16.
//
// Both kernels are launched with programmatic stream serialization and start with
// griddepcontrol.wait: a launch may become resident while the kernel ahead of it on the stream
// drains, and reads nothing before that kernel has finished.
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

constexpr int kMaxTablesAny = 2048;      // EBAG_MAX_TABLES
constexpr size_t kMaxItemTableBytes = (2 * kMaxTablesAny + 1) * sizeof(int);   // the kernel's dynamic shared memory at most
constexpr int kThreads = 256;            // 8 warps per CTA
constexpr int kWarps = kThreads / 32;
constexpr int kMaxItemBags = 32;         // an item's offsets live in one register per lane
constexpr int kItemsPerWarp = 4;         // small calls: aim for at least this many items per warp
constexpr float kSortedItemFactor = 8.0f; // item size multiplier for tables whose rows take one vector per lane
constexpr float kSmallCallFactor = 4.0f;  // the same in a call so small that the items are shrunk
constexpr float kTailItemFactor = 2.0f;   // the same for the last tables of a call (1 / 2 / 4 measured: 2 is best)
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

// ---- long bags.  A bag whose rows add up to `long_bytes` or more is not pooled by the warp that
// meets it in the forward kernel: that warp records it, and a second kernel pools the recorded
// bags in PARTS (equal runs of lookups), one part per warp, each row group of the warp leaving a
// row of partial sums in the part's slot; the warp that delivers a bag's last part adds the
// partial sums in lookup order (so the result does not depend on which warp ran what, or when)
// and writes the output row.  The host picks `long_bytes` so that the recorded bags and their
// parts always fit (at most total bytes / long_bytes bags can be that long); should malformed
// offsets make bags overlap and the room run out all the same, the bags that do not fit are
// pooled whole by the warp that met them.
constexpr int kMaxLongBags = 2048;
constexpr uint32_t kLongMinRowBytes = 256;   // narrow rows count as this much: a lone warp is latency bound
constexpr int kMaxPartsPerBag = 2048;

struct LongCtl {                         // all zero between launches
    unsigned int count;                  // bags the forward kernel recorded
    unsigned int part_next;              // next part to pool
    unsigned int exited;                 // CTAs of the parts kernel that have finished
    unsigned int pad;
};

struct LongBag {                         // what the forward kernel leaves about a bag it did not pool
    int32_t t;
    int32_t bag;                         // bag number within the launch (of its table)
};

struct LongParams {                      // ctl == nullptr: bags are never split
    LongCtl* ctl;
    LongBag* bags;                       // [kMaxLongBags]
    unsigned int* arrivals;              // [kMaxLongBags] parts delivered per bag; zero between launches
    float* partial;                      // [max_parts * slot_floats]
    uint64_t long_bytes;                 // 4 parts' worth
    uint32_t part_shift;                 // a part aims at 2^part_shift bytes of rows
    uint32_t slot_floats;                // floats per part: (bags side by side) * D, the widest of the call
    uint32_t max_parts;                  // >= kMaxLongBags
};

struct PartArgs {                        // one part of a long bag (parts kernel only)
    int64_t base;                        // first lookup of the part
    uint32_t len;                        // lookups in the part
    float* slot;                         // where its rows of partial sums go
};

// Hash table of a MapId mapping: open addressing, linear probing, at most a quarter full, 2^bits
// slots with bits = map_hash_bits(|M|); slot of key k on the first probe = (k * kHashMul) >> (64 - bits).
struct __align__(16) MapSlot {
    int64_t key;
    uint32_t idx1;      // index + 1; 0 = empty
    uint32_t pad;
};
constexpr uint64_t kHashMul = 0x9E3779B97F4A7C15ull;     // multiplicative (Fibonacci) hashing
constexpr int64_t kMapHashMaxSlots = 1ll << 24;          // 256 MB of slots per handle at most

__host__ __device__ inline uint32_t map_hash_bits(int64_t mlen) {
    uint32_t bits = 1;
    while (bits < 31 && (1ll << bits) < 4 * mlen) ++bits;
    return bits;
}

struct FwdParams {
    const void* const* tables;   // device [T]
    const TableMeta* meta;       // device [T]
    const int64_t* indices;      // int32 ids instead when idx32 is set
    const int64_t* offsets;
    const float* weights;
    float* out;                  // [B, sumD] fp32, or 16-bit elements when out16 is set
    Queue* queue;
    Status* status;
    const int64_t* const* mappings;   // MapId variant: device [T] sorted id lists (else unused)
    const int64_t* mapping_len;       // MapId variant: device [T] their lengths
    const MapSlot* map_slots;         // MapId variant: hash tables of the mappings, or null (binary search)
    const uint32_t* map_base;         // MapId variant: device [T] first slot of table t's hash table
    int64_t n_indices;
    int64_t B;                   // bags per table in this launch
    int64_t off_stride;          // offsets of table t start at offsets[t * off_stride] (B for a
                                 // whole call; the full B when a launch covers a range of bags)
    int32_t T;
    int32_t sumD;
    int32_t mean;                // 1: divide by the bag length
    int32_t idx32;               // 1: `indices` holds 32-bit ids
    int32_t out16;               // 0: fp32 output; 1: fp16; 2: bf16 (rounded to nearest-even once, at the store)
    float code_zero;             // rowwise 8-bit tables: the stored byte that means code 0 (128 signed, 0 unsigned)
    uint32_t item_bytes;
    LongParams lg;
};

// ------------------------------------------------------------------ memory access helpers
__device__ __forceinline__ int64_t ld_stream_i64(const int64_t* p) {
    // ids and offsets are read once: streaming (evict-first) so they do not displace table rows
    return __ldcs(reinterpret_cast<const long long*>(p));
}
__device__ __forceinline__ float ld_stream_f32(const float* p) { return __ldcs(p); }
// two fp32 values rounded to nearest-even into one 32-bit word of fp16 (kind 1) or bf16 (kind 2)
__device__ __forceinline__ uint32_t pack16(float lo, float hi, int kind) {
    uint32_t r;
    if (kind == 1) asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    else asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// 32 bytes in one instruction (a whole sector; the address must be 32-byte aligned)
__device__ __forceinline__ void st_stream32(float* p, float2 a, float2 b, float2 c, float2 d) {
    asm volatile("st.global.cs.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "f"(a.x), "f"(a.y),
                 "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y), "f"(d.x), "f"(d.y)
                 : "memory");
}
__device__ __forceinline__ void st_stream16(float* p, float a, float b, float c, float d) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(a, b, c, d));
}

// Asynchronous copies global -> shared (through L1, so hot rows still hit there): the data does
// not occupy registers while it is in flight.
// (`smem` is an address in the shared window, from __cvta_generic_to_shared)
__device__ __forceinline__ void cp_async16(uint32_t smem, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem), "l"(gmem));
}
// a copy of `bytes` (16 or 0) source bytes; what is not copied of the 16 is zeroed
__device__ __forceinline__ void cp_async16_zfill(uint32_t smem, const void* gmem, uint32_t bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(smem), "l"(gmem), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async8(uint32_t smem, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem), "l"(gmem));
}
// Loads from the shared window by its 32-bit address (no generic pointer to keep alongside it).
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ float2 lds64f(uint32_t a) {
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a));
    return v;
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

// Two fp32 operations per instruction (sm_100a): the pair sits in an aligned register pair.
__device__ __forceinline__ void fma2(float2& a, float w, float x0, float x1) {
    a = __ffma2_rn(make_float2(w, w), make_float2(x0, x1), a);
}
__device__ __forceinline__ void add2(float2& a, float x0, float x1) {
    a = __fadd2_rn(a, make_float2(x0, x1));
}

// acc[0..kAcc) += w * widen(d)        (int8: w is w*scale; the bias term is summed separately)
template <int DT, bool WEIGHTED>
__device__ __forceinline__ void accumulate(float2* acc, const uint4& d, float w) {
    const uint32_t r[4] = {d.x, d.y, d.z, d.w};
    if constexpr (DT == DT_F32) {
#pragma unroll
        for (int i = 0; i < 4; i += 2) {
            const float x0 = __uint_as_float(r[i]), x1 = __uint_as_float(r[i + 1]);
            if constexpr (WEIGHTED) fma2(acc[i / 2], w, x0, x1);
            else add2(acc[i / 2], x0, x1);
        }
    } else if constexpr (DT == DT_BF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if constexpr (WEIGHTED) {
                fma2(acc[i], w, __uint_as_float(r[i] << 16),
                     __uint_as_float(r[i] & 0xffff0000u));
            } else {
                add_bf16(acc[i].x, r[i]);
                add_bf16(acc[i].y, r[i] >> 16);
            }
        }
    } else if constexpr (DT == DT_F16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if constexpr (WEIGHTED) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&r[i]));
                fma2(acc[i], w, f.x, f.y);
            } else {
                add_f16(acc[i].x, r[i]);
                add_f16(acc[i].y, r[i] >> 16);
            }
        }
    } else {
        // Stored code u = q + 128 (0..255).  The byte dropped into bits 16..23 of a zero word IS
        // the float u * 2^-133, exactly, for every u (subnormal below 128, and the subnormal to
        // normal step at 128 is seamless), so widening costs one byte-permute and no arithmetic.
        // The caller passes w = weight * scale * 2^kInt8Up, the sums come out scaled by
        // 2^(kInt8Up - 133) and are scaled back, exactly, when the bag is written; the -128 of
        // every code goes into the bias term, one scalar per row.
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
            for (int k = 0; k < 4; k += 2) {
                const float f0 = __uint_as_float(__byte_perm(r[i], 0u, 0x4044 + (k << 8)));
                const float f1 = __uint_as_float(__byte_perm(r[i], 0u, 0x4144 + (k << 8)));
                fma2(acc[2 * i + k / 2], w, f0, f1);
            }
        }
    }
}
constexpr float kInt8Up = 0x1p64f;       // weight * scale travels as weight * scale * 2^64
constexpr float kInt8Down = 0x1p69f;     // 2^(133 - 64)

// acc[0..kAcc) = max(acc, widen(d))      (max pooling; rowwise 8-bit: scale * (code - zero) + bias,
// product and sum rounded separately, as the definition is written)
template <int DT>
__device__ __forceinline__ void accumulate_max(float2* acc, const uint4& d, float scale, float bias,
                                               float code_zero) {
    const uint32_t r[4] = {d.x, d.y, d.z, d.w};
    if constexpr (DT == DT_F32) {
        acc[0].x = fmaxf(acc[0].x, __uint_as_float(r[0]));
        acc[0].y = fmaxf(acc[0].y, __uint_as_float(r[1]));
        acc[1].x = fmaxf(acc[1].x, __uint_as_float(r[2]));
        acc[1].y = fmaxf(acc[1].y, __uint_as_float(r[3]));
    } else if constexpr (DT == DT_BF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            acc[i].x = fmaxf(acc[i].x, __uint_as_float(r[i] << 16));
            acc[i].y = fmaxf(acc[i].y, __uint_as_float(r[i] & 0xffff0000u));
        }
    } else if constexpr (DT == DT_F16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&r[i]));
            acc[i].x = fmaxf(acc[i].x, f.x);
            acc[i].y = fmaxf(acc[i].y, f.y);
        }
    } else {
        const float zero = 8388608.0f + code_zero;       // 2^23 + the byte that means code 0
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float q = __uint_as_float(__byte_perm(r[i], 0x4B000000u, 0x7440 + k)) - zero;   // exact
                const float x = __fadd_rn(__fmul_rn(scale, q), bias);
                float& a = (k & 1) ? acc[2 * i + k / 2].y : acc[2 * i + k / 2].x;
                a = fmaxf(a, x);
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

// The same result through the mapping's hash table: one or two 16-byte loads instead of a chain.
__device__ __forceinline__ int64_t map_hash_lookup(const MapSlot* __restrict__ tab, uint32_t bits, int64_t v) {
    const uint32_t mask = (1u << bits) - 1u;
    uint32_t s = (uint32_t)(((uint64_t)v * kHashMul) >> (64 - bits));
    for (uint32_t probe = 0; probe <= mask; ++probe) {       // at most a quarter full: ends early
        const int4 q = __ldg(reinterpret_cast<const int4*>(tab + s));
        if (q.z == 0) return 0;                               // an empty slot: not mapped
        const int64_t key = (int64_t)(((uint64_t)(uint32_t)q.y << 32) | (uint32_t)q.x);
        if (key == v) return (int64_t)(uint32_t)q.z;
        s = (s + 1) & mask;
    }
    return 0;
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
constexpr int kWarpSmemVecs = kStages * kStageVecs * 32 + 24;   // a warp's ring, then 96 words about its item's bags

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

// Offsets of bag `lane` of an item relative to the item's first lookup (both 0 for a malformed
// bag, which is reported through `bad`).
// The offsets of an item's bags as 32-bit distances from `base`, the smallest start among the
// item's well-formed bags (with offsets that do not decrease that is the first bag's start; with
// malformed ones a later bag may start before it, and is still pooled if it is well-formed itself).
// All 32 lanes call this; lanes at or beyond `cnt` hold no bag.
__device__ __forceinline__ void load_bag_range(const FwdParams& p, int64_t g0, int lane, int cnt,
                                               int64_t& base, uint32_t& off_lo, uint32_t& off_hi,
                                               bool& bad) {
    int64_t s = 0, e = 0;
    if (lane < cnt) {
        s = ld_stream_i64(p.offsets + g0 + lane);
        e = ld_stream_i64(p.offsets + g0 + lane + 1);
    }
    bad = lane < cnt && (s < 0 || e < s || e > p.n_indices);
    // smallest start of a well-formed bag: high words first, then the low words of those
    const bool in = lane < cnt && !bad;
    const unsigned hi_w = in ? (unsigned)((uint64_t)s >> 32) : 0xffffffffu;
    const unsigned hi_min = __reduce_min_sync(0xffffffffu, hi_w);
    const unsigned lo_w = (in && hi_w == hi_min) ? (unsigned)s : 0xffffffffu;
    const unsigned lo_min = __reduce_min_sync(0xffffffffu, lo_w);
    base = hi_min == 0xffffffffu ? 0 : (int64_t)(((uint64_t)hi_min << 32) | lo_min);
    off_lo = off_hi = 0;
    if (in) {
        if (e - base > 0x7fffffffll) bad = true;       // an item that spans 2^31 lookups or more
        else {
            off_lo = (uint32_t)(s - base);
            off_hi = (uint32_t)(e - base);
        }
    }
}

// PART: the "item" is one part of a long bag (`pa`): its lookups are shared out among the row
// groups as if they were NG bags, and the rows of sums go to the part's slot, never divided.
// POOL: 0 sums (sum, mean, weighted), 1 takes the element-wise maximum.
// `skip` (forward kernel, splitting on): bit i set = bag i of the item is pooled elsewhere; the
// call for the first column tile of an item works it out, the calls for the other tiles reuse it.
template <int DT, bool WEIGHTED, bool MAPID, int V, bool PART = false, int POOL = 0>
__device__ __forceinline__ void process_item(const FwdParams& p, const TableMeta& m,
                                                   const char* __restrict__ tbase, int t,
                                                   int64_t bag0, int cnt, int vec0, int lane,
                                                   unsigned& n_oob, unsigned& n_bad,
                                                   uint4* __restrict__ wbuf,
                                                   float2* __restrict__ sbbuf,
                                                   unsigned& skip, const PartArgs& pa) {
    constexpr int NACC = Elem<DT>::kAcc;
    constexpr int CR = kStageVecs / V;               // rows per stage
    // stages with gaps: zero-filling copies instead of tests (not for max pooling, where a zero is
    // not neutral; not for rowwise 8-bit rows, whose instance has no register to spare: measured slower)
    constexpr bool kZeroFill = POOL == 0 && DT != DT_INT8;
    const int G = 1 << m.g_log2;
    const int NG = 32 >> m.g_log2;
    const int lig = lane & (G - 1);
    const int grp = lane >> m.g_log2;

    int64_t base;
    uint32_t off_lo = 0, off_hi = 0;
    uint32_t key = (uint32_t)lane;
    if constexpr (PART) {
        base = pa.base;
        if (lane < cnt) {
            off_lo = (uint32_t)((uint64_t)pa.len * (uint32_t)lane / (uint32_t)cnt);
            off_hi = (uint32_t)((uint64_t)pa.len * (uint32_t)(lane + 1) / (uint32_t)cnt);
            key = ((off_hi - off_lo + 1u) << 6) | (uint32_t)lane;
        }
    } else {
        const int64_t g0 = (int64_t)t * p.off_stride + bag0;
        bool bad;
        load_bag_range(p, g0, lane, cnt, base, off_lo, off_hi, bad);
        if (bad && vec0 == 0) ++n_bad;
        if (p.lg.ctl) {
            // ---- bags long enough to be split are recorded for the parts kernel (by the call
            // for the first column tile) and count as empty here
            if (vec0 == 0) {
                bool is_long = false;
                const uint32_t len = off_hi - off_lo;
                const uint64_t bytes = (uint64_t)len * max((uint32_t)m.stride, kLongMinRowBytes);
                if (len > 0 && bytes >= p.lg.long_bytes) {
                    const unsigned idx = atomicAdd(&p.lg.ctl->count, 1u);
                    if (idx < (unsigned)kMaxLongBags) {          // else: no room, pooled whole here
                        is_long = true;
                        p.lg.bags[idx].t = t;
                        p.lg.bags[idx].bag = (int32_t)(bag0 + lane);
                    }
                }
                skip = __ballot_sync(0xffffffffu, is_long);
            }
            if ((skip >> lane) & 1u) {
                off_hi = off_lo;
                key |= 32u;                  // carried through the sort in the key
            }
        }
        if (lane < cnt) {
            const uint32_t len = off_hi - off_lo;
            key |= ((len > 0x1FFFFFEu ? 0x1FFFFFEu : len) + 1u) << 6;
        }
    }
    if (NG > 1 && cnt > NG) key = warp_sort_desc(key, lane);
    // the item's bags, readable by every lane: [0,32) first lookup, [32,64) end, [64,96) sorted keys
    uint32_t* bagw = reinterpret_cast<uint32_t*>(wbuf + kStages * kStageVecs * 32);
    __syncwarp();                                    // the previous item's readers are done
    bagw[lane] = off_lo;
    bagw[32 + lane] = off_hi;
    bagw[64 + lane] = key;
    __syncwarp();
    // this lane's slots in the ring, as addresses in the shared window: vector k of stage st is
    // at my_rows_s + (st * kStageVecs + k) * 512 (kept opaque: not to be recomputed at every use)
    uint32_t my_rows_s = (uint32_t)__cvta_generic_to_shared(wbuf) + lane * 16;
    asm volatile("" : "+r"(my_rows_s));
    // first id of the item (ids are 8 bytes wide, or 4 when p.idx32)
    const char* __restrict__ idx_base =
        reinterpret_cast<const char*>(p.indices) + base * (p.idx32 ? 4 : 8);
    const float* __restrict__ w_base = WEIGHTED ? p.weights + base : nullptr;

    bool col_on[V];
    const char* lane_base[V];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int vec = vec0 + v * G + lig;
        col_on[v] = vec < m.nvec;
        lane_base[v] = tbase + vec * 16;
        // (a table without rows may come without memory; its copies, all of zero bytes, name the output)
        if (kZeroFill && m.rows <= 0) lane_base[v] = reinterpret_cast<const char*>(p.out) + vec * 16;
    }
    const uint32_t stride = (uint32_t)m.stride;
    const uint32_t rows = (uint32_t)m.rows;          // tables have fewer than 2^31 rows
    const int sb_delta = m.D - vec0 * 16;            // int8, lane 0 of a group: from its row vector to the scale/bias pair
    const int nslots = (cnt + NG - 1) >> (5 - m.g_log2);

    const int64_t* __restrict__ map_ptr = MAPID ? p.mappings[t] : nullptr;
    const int64_t map_len64 = MAPID ? p.mapping_len[t] : 0;
    const uint32_t map_len = (uint32_t)(map_len64 < 0 ? 0 : map_len64);
    const int map_steps = 32 - __clz(map_len);
    const MapSlot* __restrict__ map_tab = (MAPID && p.map_slots) ? p.map_slots + p.map_base[t] : nullptr;
    const uint32_t map_bits = MAPID ? map_hash_bits(map_len) : 0;
    auto load_chunk = [&](uint32_t pos, uint32_t end, uint32_t& ridx, float& w) {
        ridx = kInvalidRow;
        w = 0.0f;
        const uint32_t i = pos + lig;
        if (i < end) {
            int64_t r;
            if (p.idx32) r = __ldcs(reinterpret_cast<const int*>(idx_base) + i);
            else r = ld_stream_i64(reinterpret_cast<const int64_t*>(idx_base) + i);
            float wl = 1.0f;
            if (WEIGHTED) wl = ld_stream_f32(w_base + i);
            if (MAPID)                                                  // raw id -> row
                r = map_tab ? map_hash_lookup(map_tab, map_bits, r) : map_id(map_ptr, map_len, map_steps, r);
            if ((uint64_t)r < (uint64_t)rows) {
                ridx = (uint32_t)r;
                w = wl;
            } else if (vec0 == 0) {
                ++n_oob;
            }
        }
    };
    auto slot_bag = [&](int pos_in_item, uint32_t& s, uint32_t& e, int& orig, bool& elsewhere) {
        const uint32_t bag_s = my_rows_s - lane * 16 + kStages * kStageVecs * 512;   // after the ring
        const uint32_t k = lds32(bag_s + 256 + (pos_in_item & 31) * 4);
        orig = (int)(k & 31u);
        elsewhere = (k & 32u) != 0;
        s = lds32(bag_s + orig * 4);
        e = lds32(bag_s + 128 + orig * 4);
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
            bool unused;
            slot_bag(gslot * NG + grp, gs, ge, o, unused);
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
    uint32_t my_sb_s = (uint32_t)__cvta_generic_to_shared(sbbuf) + grp * 8;
    asm volatile("" : "+r"(my_sb_s));
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
                    cp_async8(my_sb_s + (st * kStageVecs + u) * 64, lane_base[0] + roff + sb_delta);
            }
            return;
        }
        if constexpr (kZeroFill) {
            // A stage with gaps (past a bag's end, a skipped id, a lane past the row's end): every
            // slot still gets its copy, of zero source bytes where the row is missing, which fills
            // the slot with zeros and reads nothing; the consuming side then adds zeros and has
            // nothing to test.  Only the rows past the longest bag's end (warp-uniform) are left out.
#pragma unroll
            for (int u = 0; u < CR; ++u) {
                if (j0 + u >= c.nmax) break;
                const uint32_t r = __shfl_sync(0xffffffffu, c.r, j0 + u, G);
                const bool have = r != kInvalidRow;
                const uint64_t roff = (uint64_t)(have ? r : 0u) * stride;
#pragma unroll
                for (int v = 0; v < V; ++v)
                    cp_async16_zfill(my_rows_s + (st * kStageVecs + u * V + v) * 512, lane_base[v] + roff,
                                     (have && col_on[v]) ? 16u : 0u);
            }
        } else {
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
                        cp_async8(my_sb_s + (st * kStageVecs + u) * 64, lane_base[0] + roff + sb_delta);
                }
            }
        }
    };
    float2 acc[V][NACC / 2];                         // pairs: two fp32 operations per instruction
    float acc_bias = 0.0f;
    const float acc0 = POOL == 1 ? __int_as_float(0xff800000) : 0.0f;     // -inf for max pooling
#pragma unroll
    for (int v = 0; v < V; ++v)
#pragma unroll
        for (int a = 0; a < NACC / 2; ++a) acc[v][a] = make_float2(acc0, acc0);
    auto consume = [&](const IdChunk& c, int j0, int st) {
        if (c.clean && j0 + CR <= c.nmin) {
#pragma unroll
            for (int u = 0; u < CR; ++u) {
                float wu = WEIGHTED ? __shfl_sync(0xffffffffu, c.w, j0 + u, G) : 1.0f;
                float2 sb = make_float2(1.0f, 0.0f);
                if (DT == DT_INT8) {
                    sb = lds64f(my_sb_s + (st * kStageVecs + u) * 64);
                    if (POOL == 0) {
                        // the row's constant, bias - zero * scale, rounded once; then the weight
                        acc_bias = fmaf(wu, fmaf(-p.code_zero, sb.x, sb.y), acc_bias);
                        wu *= sb.x * kInt8Up;
                    }
                }
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const uint4 d = lds128(my_rows_s + (st * kStageVecs + u * V + v) * 512);
                    if constexpr (POOL == 1) accumulate_max<DT>(acc[v], d, sb.x, sb.y, p.code_zero);
                    else accumulate<DT, WEIGHTED || DT == DT_INT8>(acc[v], d, wu);
                }
            }
            return;
        }
        if constexpr (kZeroFill) {
            // gaps hold zeros (see the request side): the same straight code, up to the longest bag's end
#pragma unroll
            for (int u = 0; u < CR; ++u) {
                if (j0 + u >= c.nmax) break;
                const float wu = WEIGHTED ? __shfl_sync(0xffffffffu, c.w, j0 + u, G) : 1.0f;
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const uint4 d = lds128(my_rows_s + (st * kStageVecs + u * V + v) * 512);
                    accumulate<DT, WEIGHTED>(acc[v], d, wu);
                }
            }
        } else {
#pragma unroll
            for (int u = 0; u < CR; ++u) {
                const uint32_t r = __shfl_sync(0xffffffffu, c.r, j0 + u, G);
                float wu = WEIGHTED ? __shfl_sync(0xffffffffu, c.w, j0 + u, G) : 1.0f;
                if (j0 + u < c.nmax && r != kInvalidRow) {
                    float2 sb = make_float2(1.0f, 0.0f);
                    if (DT == DT_INT8) {
                        sb = lds64f(my_sb_s + (st * kStageVecs + u) * 64);
                        if (POOL == 0) {
                            // the row's constant, bias - zero * scale, rounded once; then the weight
                            acc_bias = fmaf(wu, fmaf(-p.code_zero, sb.x, sb.y), acc_bias);
                            wu *= sb.x * kInt8Up;
                        }
                    }
#pragma unroll
                    for (int v = 0; v < V; ++v)
                        if (col_on[v]) {
                            const uint4 d = lds128(my_rows_s + (st * kStageVecs + u * V + v) * 512);
                            if constexpr (POOL == 1) accumulate_max<DT>(acc[v], d, sb.x, sb.y, p.code_zero);
                            else accumulate<DT, WEIGHTED || DT == DT_INT8>(acc[v], d, wu);
                        }
                }
            }
        }
    };
    auto finalize = [&](int slot) {
        uint32_t s, e;
        int orig;
        bool elsewhere;
        slot_bag(slot * NG + grp, s, e, orig, elsewhere);
        bool write = slot * NG + grp < cnt;
        if (!PART) write = write && !elsewhere;
        if (write) {
            const uint32_t L = e - s;
            float* orow = PART ? pa.slot + (size_t)orig * m.D
                               : p.out + (bag0 + orig) * (int64_t)p.sumD + m.D_off;
#pragma unroll
            for (int v = 0; v < V; ++v) {
                if (!col_on[v]) continue;
                float* o = orow + (size_t)(vec0 + v * G + lig) * NACC;
#pragma unroll
                for (int a = 0; a < NACC / 2; ++a) {
                    float2 x = acc[v][a];
                    if (POOL == 1) {                 // a bag with no valid lookup reads +0
                        if (x.x == acc0) x.x = 0.0f;
                        if (x.y == acc0) x.y = 0.0f;
                    } else if (DT == DT_INT8) {
                        x.x = fmaf(x.x, kInt8Down, acc_bias);
                        x.y = fmaf(x.y, kInt8Down, acc_bias);
                    }
                    if (POOL == 0 && !PART && p.mean && L > 0) {
                        x.x = __fdiv_rn(x.x, (float)L);
                        x.y = __fdiv_rn(x.y, (float)L);
                    }
                    acc[v][a] = x;
                }
                if (PART || p.out16 == 0) {
                    // 16- and 8-bit tables: a lane holds one or two whole 32-byte sectors of the
                    // row; written 16 bytes at a time every store instruction of the warp would
                    // write half of each sector it touches
                    bool wide = false;
                    if constexpr (NACC >= 8) wide = (reinterpret_cast<uintptr_t>(o) & 31u) == 0;
                    if (wide) {
                        if constexpr (NACC >= 8) {
#pragma unroll
                            for (int a = 0; a < NACC / 2; a += 4)
                                st_stream32(o + 2 * a, acc[v][a], acc[v][a + 1], acc[v][a + 2], acc[v][a + 3]);
                        }
                    } else {
#pragma unroll
                        for (int a = 0; a < NACC / 2; a += 2)
                            st_stream16(o + 2 * a, acc[v][a].x, acc[v][a].y, acc[v][a + 1].x, acc[v][a + 1].y);
                    }
                } else {
                    // 16-bit output: the same elements, half the bytes
                    uint32_t* o16 = reinterpret_cast<uint32_t*>(p.out) +
                                    (((bag0 + orig) * (int64_t)p.sumD + m.D_off +
                                      (int64_t)(vec0 + v * G + lig) * NACC) >> 1);
                    uint32_t wd[NACC / 2];
#pragma unroll
                    for (int a = 0; a < NACC / 2; ++a) wd[a] = pack16(acc[v][a].x, acc[v][a].y, p.out16);
                    if constexpr (NACC == 4) {
                        __stcs(reinterpret_cast<uint2*>(o16), make_uint2(wd[0], wd[1]));
                    } else if (NACC == 16 && (reinterpret_cast<uintptr_t>(o16) & 31u) == 0) {
                        // 8-bit tables: the lane's 16 elements are one whole sector
                        if constexpr (NACC == 16)
                            asm volatile("st.global.cs.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(o16),
                                         "r"(wd[0]), "r"(wd[1]), "r"(wd[2]), "r"(wd[3]), "r"(wd[4]), "r"(wd[5]),
                                         "r"(wd[6]), "r"(wd[7])
                                         : "memory");
                    } else {
#pragma unroll
                        for (int a = 0; a < NACC / 2; a += 4)
                            __stcs(reinterpret_cast<uint4*>(o16 + a), make_uint4(wd[a], wd[a + 1], wd[a + 2], wd[a + 3]));
                    }
                }
            }
        }
        acc_bias = 0.0f;
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int a = 0; a < NACC / 2; ++a) acc[v][a] = make_float2(acc0, acc0);
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
template <int DT, bool WEIGHTED, bool MAPID, int POOL = 0>
__global__ void __launch_bounds__(kThreads, EBAG_MIN_BLOCKS)
ebag_fwd_kernel(const FwdParams p) {
    extern __shared__ int smem_i[];
    int* item_base = smem_i;                                   // [T+1] first item of each table
    int* item_bags = smem_i + p.T + 1;                         // [T]   bags per item of each table
    float* bag_bytes = reinterpret_cast<float*>(item_bags);    // [T]   (first pass) bytes per bag
    __shared__ unsigned long long total_bytes_u;
    __shared__ uint4 stage_buf[kWarps * kWarpSmemVecs];      // per warp: 4 KB ring + the item's bags
    __shared__ float2 sb_buf[DT == DT_INT8 ? kWarps * kStages * kStageVecs * 8 : 1];
    int tid;
    asm volatile("mov.u32 %0, %%tid.x;" : "=r"(tid));      // read once: not re-read wherever a use is
    uint4* wbuf = stage_buf + (tid >> 5) * kWarpSmemVecs;
    float2* sbbuf = sb_buf + (DT == DT_INT8 ? (tid >> 5) * (kStages * kStageVecs * 8) : 0);
    const int lane = tid & 31;

    // This launch may have been made resident before the kernel ahead of it on the stream
    // finished: wait for it (and its writes).  In turn the kernel that follows (the parts kernel,
    // or the next forward) may take the place of CTAs that finish here; it waits the same way.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");

    // ---- size the items of every table from its share of the offsets prefix sum
    // (summed as integers: every CTA must arrive at the same item tables, bit for bit, and a
    // floating-point sum would depend on the order of the additions)
    if (tid == 0) total_bytes_u = 0ull;
    __syncthreads();
    for (int t = tid; t < p.T; t += kThreads) {
        const int64_t n0 = p.offsets[(int64_t)t * p.off_stride];
        const int64_t n1 = p.offsets[(int64_t)t * p.off_stride + p.B];
        int64_t nt = n1 - n0;
        if (nt < 0) nt = 0;
        if (nt > p.n_indices) nt = p.n_indices;
        const float bytes = (float)nt * (float)p.meta[t].stride;
        bag_bytes[t] = fmaxf(bytes / (float)p.B, 1.0f);
        atomicAdd(&total_bytes_u, (unsigned long long)nt * (unsigned long long)p.meta[t].stride);
    }
    __syncthreads();
    const float total_bytes = (float)total_bytes_u;
    // small calls: shrink the items so that every warp of the grid gets a few of them
    const float spread = total_bytes / (float)(gridDim.x * kWarps * kItemsPerWarp);
    const float item_bytes = fminf((float)p.item_bytes, spread);
    const float big_item = fminf(kSortedItemFactor * (float)p.item_bytes, kSmallCallFactor * spread);
    // The queue hands items out in table order, so the last tables decide how long the slowest
    // warp runs after the others are done: the tables that make up the last big item's worth of
    // work per warp get plain (small) items.  Marked by a negative bag size.
    if (tid == 0) {
        const float budget = big_item * (float)(gridDim.x * kWarps);
        float after = 0.0f;
        for (int t = p.T - 1; t >= 0; --t) {
            after += bag_bytes[t] * (float)p.B;
            if (after > budget) break;
            bag_bytes[t] = -bag_bytes[t];
        }
    }
    __syncthreads();
    for (int t = tid; t < p.T; t += kThreads) {
        const int ng = 32 >> p.meta[t].g_log2;
        // bags that run side by side are matched by length inside an item: more bags per item,
        // better matches (measured: cfg 5 6.70 -> 5.75 ms, cfg 3 2.35 -> 2.12 ms)
        // (also: fewer item start-ups, each of which leaves the warp's pipeline empty for a while;
        // rows of two vectors per lane gather enough per bag and balance better with small items)
        const bool tail = bag_bytes[t] < 0.0f;
        const float target = p.meta[t].V != 1 ? item_bytes : (tail ? fminf(kTailItemFactor * item_bytes, big_item) : big_item);
        const float want = target / fabsf(bag_bytes[t]);
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

        const PartArgs no_part{};
        unsigned skip = 0;
        if (m.V == 1) {
            process_item<DT, WEIGHTED, MAPID, 1, false, POOL>(p, m, tbase, t, bag0, cnt, 0, lane, n_oob, n_bad,
                                                              wbuf, sbbuf, skip, no_part);
        } else {
            // rows above 512 bytes: two vectors per lane, 1 KB column tiles
            for (int vec0 = 0; vec0 < m.nvec; vec0 += 64)
                process_item<DT, WEIGHTED, MAPID, 2, false, POOL>(p, m, tbase, t, bag0, cnt, vec0, lane, n_oob,
                                                                  n_bad, wbuf, sbbuf, skip, no_part);
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

// ------------------------------------------------------------------ the parts kernel
// Pools the long bags the forward kernel recorded (it runs after it on the same stream).  A launch
// that finds nothing recorded ends at once.
template <int DT, bool WEIGHTED, bool MAPID>
__global__ void __launch_bounds__(kThreads, EBAG_MIN_BLOCKS)
ebag_parts_kernel(const FwdParams p) {
    __shared__ uint4 stage_buf[kWarps * kWarpSmemVecs];
    __shared__ float2 sb_buf[DT == DT_INT8 ? kWarps * kStages * kStageVecs * 8 : 1];
    __shared__ unsigned part0_s[kMaxLongBags + 1];     // first part of every recorded bag
    __shared__ unsigned scan_warp_s[kWarps], scan_carry_s;
    int tid;
    asm volatile("mov.u32 %0, %%tid.x;" : "=r"(tid));      // read once: not re-read wherever a use is
    uint4* wbuf = stage_buf + (tid >> 5) * kWarpSmemVecs;
    float2* sbbuf = sb_buf + (DT == DT_INT8 ? (tid >> 5) * (kStages * kStageVecs * 8) : 0);
    const int lane = tid & 31;

    // this launch may have been made resident before the forward kernel finished: wait for it
    asm volatile("griddepcontrol.wait;" ::: "memory");
    unsigned nb = p.lg.ctl->count;
    if (nb == 0) return;                               // nothing was recorded (and nothing to re-arm)
    if (nb > (unsigned)kMaxLongBags) nb = kMaxLongBags;

    // ---- plan: parts per bag from its length, first part of every bag by a prefix sum.  Every
    // CTA works out the same plan from the same records.
    auto want_of = [&](unsigned i) -> unsigned {
        const LongBag r = p.lg.bags[i];
        const int64_t g = (int64_t)r.t * p.off_stride + r.bag;
        const uint64_t len = (uint64_t)(p.offsets[g + 1] - p.offsets[g]);   // checked by the forward kernel
        const uint64_t bytes = len * max((uint32_t)p.meta[r.t].stride, kLongMinRowBytes);
        uint64_t want = (bytes + ((1ull << p.lg.part_shift) - 1)) >> p.lg.part_shift;
        if (want > (uint64_t)kMaxPartsPerBag) want = kMaxPartsPerBag;
        if (want > len) want = len;
        return (unsigned)want;
    };
    for (int pass = 0; pass < 2; ++pass) {
        // pass 0 with the parts each bag wants; should they not fit (only overlapping bags can
        // ask for that much), pass 1 with one part per bag, which always fits
        if (tid == 0) scan_carry_s = 0;
        __syncthreads();
        for (unsigned i0 = 0; i0 < nb; i0 += kThreads) {
            const unsigned i = i0 + tid;
            unsigned x = i < nb ? (pass == 0 ? want_of(i) : 1u) : 0u;
            const unsigned mine = x;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const unsigned y = __shfl_up_sync(0xffffffffu, x, d);
                if (lane >= d) x += y;
            }
            if (lane == 31) scan_warp_s[tid >> 5] = x;
            __syncthreads();
            unsigned before = scan_carry_s;
            for (int w = 0; w < (tid >> 5); ++w) before += scan_warp_s[w];
            if (i < nb) part0_s[i] = before + x - mine;
            __syncthreads();
            if (tid == kThreads - 1) scan_carry_s = before + x;
            __syncthreads();
        }
        if (scan_carry_s <= p.lg.max_parts) break;
        __syncthreads();
    }
    const unsigned part_total = scan_carry_s;
    if (tid == 0) part0_s[nb] = part_total;
    __syncthreads();

    unsigned n_oob = 0, n_bad = 0;
    while (true) {
        unsigned pq = 0;
        if (lane == 0) pq = atomicAdd(&p.lg.ctl->part_next, 1u);
        pq = __shfl_sync(0xffffffffu, pq, 0);
        if (pq >= part_total) break;
        // the bag of part pq: last record with part0 <= pq
        unsigned blo = 0, bhi = nb;
        while (bhi - blo > 1) {
            const unsigned mid = (blo + bhi) >> 1;
            if (part0_s[mid] <= pq) blo = mid; else bhi = mid;
        }
        const unsigned bi = blo;
        const unsigned bag_part0 = part0_s[bi];
        const unsigned bag_parts = part0_s[bi + 1] - bag_part0;
        const LongBag rec = p.lg.bags[bi];
        const int t = rec.t;
        const TableMeta m = p.meta[t];
        const int ng = 32 >> m.g_log2;
        const int64_t g = (int64_t)t * p.off_stride + rec.bag;
        const int64_t lo = p.offsets[g];
        const uint64_t len = (uint64_t)(p.offsets[g + 1] - lo);
        {
            const char* tbase = static_cast<const char*>(p.tables[t]);
            const uint64_t k = pq - bag_part0;
            const uint64_t s0 = len * k / bag_parts, s1 = len * (k + 1) / bag_parts;
            unsigned no_skip = 0;
            PartArgs pa;
            pa.base = lo + (int64_t)s0;
            pa.len = (uint32_t)(s1 - s0);
            pa.slot = p.lg.partial + (size_t)pq * p.lg.slot_floats;
            if (m.V == 1) {
                process_item<DT, WEIGHTED, MAPID, 1, true>(p, m, tbase, t, 0, ng, 0, lane, n_oob, n_bad,
                                                           wbuf, sbbuf, no_skip, pa);
            } else {
                for (int vec0 = 0; vec0 < m.nvec; vec0 += 64)
                    process_item<DT, WEIGHTED, MAPID, 2, true>(p, m, tbase, t, 0, ng, vec0, lane, n_oob,
                                                               n_bad, wbuf, sbbuf, no_skip, pa);
            }
        }
        // ---- deliver the part; whoever delivers a bag's last part adds them up, in lookup order
        __threadfence();
        __syncwarp();
        unsigned prev = 0;
        if (lane == 0) prev = atomicAdd(&p.lg.arrivals[bi], 1u);
        prev = __shfl_sync(0xffffffffu, prev, 0);
        if (prev == bag_parts - 1) {
            __threadfence();
            const float* src = p.lg.partial + (size_t)bag_part0 * p.lg.slot_floats;
            float* orow = p.out + rec.bag * (int64_t)p.sumD + m.D_off;
            // rows of partial sums, in lookup order: row r is at src + (r / ng) * slot + (r % ng) * D
            const unsigned nrows = bag_parts * (unsigned)ng;
            for (int c = lane * 4; c < m.D; c += 128) {
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                constexpr int kBatch = 8;                // loads in flight; the adds stay in order
                for (unsigned r0 = 0; r0 < nrows; r0 += kBatch) {
                    float4 x[kBatch];
#pragma unroll
                    for (int i = 0; i < kBatch; ++i) {
                        const unsigned r = r0 + i;
                        x[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (r < nrows)
                            x[i] = __ldcg(reinterpret_cast<const float4*>(
                                src + (size_t)(r >> (5 - m.g_log2)) * p.lg.slot_floats +
                                (size_t)(r & (ng - 1)) * m.D + c));
                    }
#pragma unroll
                    for (int i = 0; i < kBatch; ++i)
                        if (r0 + i < nrows) {
                            acc.x += x[i].x; acc.y += x[i].y; acc.z += x[i].z; acc.w += x[i].w;
                        }
                }
                if (p.mean && len > 0) {
                    const float fl = (float)len;
                    acc.x = __fdiv_rn(acc.x, fl); acc.y = __fdiv_rn(acc.y, fl);
                    acc.z = __fdiv_rn(acc.z, fl); acc.w = __fdiv_rn(acc.w, fl);
                }
                if (p.out16 == 0) {
                    st_stream16(orow + c, acc.x, acc.y, acc.z, acc.w);
                } else {
                    uint32_t* o16 = reinterpret_cast<uint32_t*>(p.out) +
                                    ((rec.bag * (int64_t)p.sumD + m.D_off + c) >> 1);
                    __stcs(reinterpret_cast<uint2*>(o16),
                           make_uint2(pack16(acc.x, acc.y, p.out16), pack16(acc.z, acc.w, p.out16)));
                }
            }
            if (lane == 0) p.lg.arrivals[bi] = 0;       // ready for the next launch
        }
    }

    n_oob = __reduce_add_sync(0xffffffffu, n_oob);
    if (lane == 0 && n_oob) atomicAdd(&p.status->n_oob, (unsigned long long)n_oob);
    __syncthreads();
    if (tid == 0) {                                    // the last CTA out re-arms the bookkeeping
        __threadfence();
        const unsigned prev = atomicAdd(&p.lg.ctl->exited, 1u);
        if (prev == gridDim.x - 1) {
            p.lg.ctl->count = 0;
            p.lg.ctl->part_next = 0;
            p.lg.ctl->exited = 0;
            __threadfence();
        }
    }
}

// one launcher per dtype, each compiled in its own translation unit
#define EBAG_DECLARE_LAUNCHERS(NAME)                                                             \
    cudaError_t launch_fwd_##NAME(const FwdParams& p, bool weighted, bool mapid, int grid,        \
                                  size_t smem, cudaStream_t s);                                  \
    cudaError_t occupancy_fwd_##NAME(bool weighted, bool mapid, size_t smem, int* ctas_per_sm);  \
    cudaError_t launch_fwdmax_##NAME(const FwdParams& p, int grid, size_t smem, cudaStream_t s);  \
    cudaError_t launch_parts_##NAME(const FwdParams& p, bool weighted, bool mapid, int grid,      \
                                    cudaStream_t s);
EBAG_DECLARE_LAUNCHERS(f32)
EBAG_DECLARE_LAUNCHERS(f16)
EBAG_DECLARE_LAUNCHERS(bf16)
EBAG_DECLARE_LAUNCHERS(int8)

#define EBAG_DEFINE_LAUNCHERS(NAME, DT)                                                          \
    cudaError_t launch_fwd_##NAME(const FwdParams& p, bool weighted, bool mapid, int grid,        \
                                  size_t smem, cudaStream_t s) {                                 \
        /* may be made resident while the kernel before it on the stream drains: the kernel's    \
           first instruction waits for that kernel to finish and for its writes */               \
        cudaLaunchAttribute attr[1];                                                             \
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                         \
        attr[0].val.programmaticStreamSerializationAllowed = 1;                                  \
        cudaLaunchConfig_t cfg = {};                                                             \
        cfg.gridDim = dim3((unsigned)grid);                                                      \
        cfg.blockDim = dim3(kThreads);                                                           \
        cfg.dynamicSmemBytes = smem;                                                             \
        cfg.stream = s;                                                                          \
        cfg.attrs = attr;                                                                        \
        cfg.numAttrs = 1;                                                                        \
        if (mapid) {                                                                             \
            if (weighted) return cudaLaunchKernelEx(&cfg, ebag_fwd_kernel<DT, true, true>, p);    \
            return cudaLaunchKernelEx(&cfg, ebag_fwd_kernel<DT, false, true>, p);                \
        }                                                                                        \
        if (weighted) return cudaLaunchKernelEx(&cfg, ebag_fwd_kernel<DT, true, false>, p);       \
        return cudaLaunchKernelEx(&cfg, ebag_fwd_kernel<DT, false, false>, p);                   \
    }                                                                                            \
    cudaError_t launch_fwdmax_##NAME(const FwdParams& p, int grid, size_t smem, cudaStream_t s) { \
        cudaError_t e = cudaFuncSetAttribute((const void*)ebag_fwd_kernel<DT, false, false, 1>,   \
                                             cudaFuncAttributeMaxDynamicSharedMemorySize,        \
                                             (int)kMaxItemTableBytes);                           \
        if (e != cudaSuccess) return e;                                                          \
        ebag_fwd_kernel<DT, false, false, 1><<<grid, kThreads, smem, s>>>(p);                     \
        return cudaGetLastError();                                                               \
    }                                                                                            \
    cudaError_t launch_parts_##NAME(const FwdParams& p, bool weighted, bool mapid, int grid,      \
                                    cudaStream_t s) {                                            \
        /* may be made resident while the forward kernel drains (it waits for it on the device) */\
        cudaLaunchAttribute attr[1];                                                             \
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                         \
        attr[0].val.programmaticStreamSerializationAllowed = 1;                                  \
        cudaLaunchConfig_t cfg = {};                                                             \
        cfg.gridDim = dim3((unsigned)grid);                                                      \
        cfg.blockDim = dim3(kThreads);                                                           \
        cfg.dynamicSmemBytes = 0;                                                                \
        cfg.stream = s;                                                                          \
        cfg.attrs = attr;                                                                        \
        cfg.numAttrs = 1;                                                                        \
        if (mapid) {                                                                             \
            if (weighted) return cudaLaunchKernelEx(&cfg, ebag_parts_kernel<DT, true, true>, p);  \
            return cudaLaunchKernelEx(&cfg, ebag_parts_kernel<DT, false, true>, p);              \
        }                                                                                        \
        if (weighted) return cudaLaunchKernelEx(&cfg, ebag_parts_kernel<DT, true, false>, p);     \
        return cudaLaunchKernelEx(&cfg, ebag_parts_kernel<DT, false, false>, p);                 \
    }                                                                                            \
    cudaError_t occupancy_fwd_##NAME(bool weighted, bool mapid, size_t smem, int* n) {            \
        const void* k = mapid ? (weighted ? (const void*)ebag_fwd_kernel<DT, true, true>          \
                                          : (const void*)ebag_fwd_kernel<DT, false, true>)        \
                              : (weighted ? (const void*)ebag_fwd_kernel<DT, true, false>         \
                                          : (const void*)ebag_fwd_kernel<DT, false, false>);      \
        /* static + dynamic shared memory passes 48 KB when there are many tables: opt in, once   \
           and for the most tables any handle may have (the attribute belongs to the kernel, not  \
           to the handle) */                                                                     \
        cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize,      \
                                             (int)(smem > kMaxItemTableBytes ? smem : kMaxItemTableBytes)); \
        if (e != cudaSuccess) return e;                                                          \
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(n, k, kThreads, smem);              \
    }

}  // namespace ebag
