// Gradient of the pooled forward with respect to the per-sample weights (sm_100a).
//
// The forward is linear in the weights (the scores of the paper's weighted sparse features,
// Sec. 2.2 "Feature Types and Memory Layout"), so for lookup i of bag (t, b)
//     grad_w[i] = sum_d grad_out[b, Doff[t] + d] * value(t, indices[i], d)      (EBAG_MEAN: / L)
// one dot product per lookup between the bag's slice of grad_out and the looked-up row.  It is the
// forward's gather with the roles swapped: the bag's slice sits in registers (G lanes x one
// 16-byte row vector each, wider rows in column tiles of G vectors); the looked-up rows travel
// eight at a time through a ring of two stages in shared memory (asynchronous 16-byte copies into
// slots private to each lane, so no barrier is needed; the (scale, bias) pair of a rowwise 8-bit
// row is copied once per group, by its first lane, and read after a __syncwarp; the ids of the
// batch after the next are requested before that); the eight dot products of a batch are summed over the lanes of the
// group together (at every step of the butterfly a lane hands half of its values to its partner
// and keeps the other half: 7 + log2(G/8) shuffles for 8 rows instead of 8 log2(G); the tree of
// additions is the same for every row, so the result is reproducible bit for bit) and up to eight
// lanes write one gradient each.  32/G bags run side by side in a warp; work is dealt statically
// in table-major order.  Ids outside the table give 0 and are counted, malformed bags are skipped
// and counted, as everywhere else.
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "ebag_bwd_weights.cuh"

namespace ebag {

namespace {

constexpr int kGwThreads = 256;
constexpr int kGwWarps = kGwThreads / 32;
constexpr int kGwRows = 8;            // rows of a bag per batch (one stage of the ring)
constexpr uint32_t kGwNoRow = 0xffffffffu;
constexpr int kGwRingBytes = 2 * kGwRows * 512;       // per warp: two stages of kGwRows 16-byte vectors per lane
constexpr int kGwSbBytes = 2 * kGwRows * 8 * 8;       // per warp, rowwise 8-bit: (scale, bias) of every row, one copy per group (at most 8 groups)

// asynchronous copy of `bytes` (16 / 8 or 0) source bytes; the rest of the 16 / 8 are zeroed
__device__ __forceinline__ void cp_async16_zfill(uint32_t smem, const void* gmem, uint32_t bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(smem), "l"(gmem), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async8_zfill(uint32_t smem, const void* gmem, uint32_t bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(smem), "l"(gmem), "r"(bytes) : "memory");
}

// sum_k g[k] * widen(d)[k] over the elements of one 16-byte row vector, two elements per
// instruction (g as fp32 pairs).  Rowwise 8-bit: returns sum_k g[k] * (code_k - zero), the codes
// widened exactly (2^23 + byte, minus 2^23 + zero); the caller applies the row's scale and bias.
template <int DT>
__device__ __forceinline__ float dot_vec(const float2* g, const uint4& d, float code_zero) {
    const uint32_t r[4] = {d.x, d.y, d.z, d.w};
    float2 s = make_float2(0.0f, 0.0f);
    if constexpr (DT == DT_F32) {
#pragma unroll
        for (int i = 0; i < 2; ++i)
            s = __ffma2_rn(g[i], make_float2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1])), s);
    } else if constexpr (DT == DT_BF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            s = __ffma2_rn(g[i], make_float2(__uint_as_float(r[i] << 16), __uint_as_float(r[i] & 0xffff0000u)), s);
    } else if constexpr (DT == DT_F16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) s = __ffma2_rn(g[i], __half22float2(*reinterpret_cast<const __half2*>(&r[i])), s);
    } else {
        const float zero = -(8388608.0f + code_zero);       // -(2^23 + the byte that means code 0)
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int k = 0; k < 4; k += 2) {
                const float f0 = __uint_as_float(__byte_perm(r[i], 0x4B000000u, 0x7440 + k));
                const float f1 = __uint_as_float(__byte_perm(r[i], 0x4B000000u, 0x7441 + k));
                const float2 q = __fadd2_rn(make_float2(f0, f1), make_float2(zero, zero));   // exact
                s = __ffma2_rn(g[2 * i + k / 2], q, s);
            }
    }
    return s.x + s.y;
}

// One launch per width class: GL = log2 of the lanes that cover a row (or one column tile of
// it), a compile-time value, so that the butterfly and the batch have no width to branch on; the
// launch takes the tables of its class and passes the others by.
template <int DT, int GL>
__global__ void __launch_bounds__(kGwThreads, 3) ebag_bwd_weights_kernel(const BwdWeightsParams p) {
    constexpr int NACC = Elem<DT>::kAcc;                // elements per 16-byte row vector
    constexpr int R = kGwRows;
    extern __shared__ __align__(16) unsigned char gw_smem[];
    // [warps][ring], rowwise 8-bit: [warps][scale/bias ring], then [T+1] first item of each table
    int* item_base = reinterpret_cast<int*>(gw_smem + kGwWarps * (kGwRingBytes + (DT == DT_INT8 ? kGwSbBytes : 0)));
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    constexpr int G = 1 << GL, ng = 32 >> GL;
    for (int t = tid; t < p.T; t += kGwThreads)
        item_base[t + 1] = p.meta[t].g_log2 == GL ? (int)((p.B + ng - 1) / ng) : 0;
    __syncthreads();
    if (tid == 0) {
        item_base[0] = 0;
        for (int t = 0; t < p.T; ++t) item_base[t + 1] += item_base[t];
    }
    __syncthreads();
    const int64_t total = item_base[p.T];
    const int64_t warps = (int64_t)gridDim.x * kGwWarps;
    unsigned n_oob = 0, n_bad = 0;
    // this lane's slots: row u of stage st at ring_s + (st * R + u) * 512; its group's (scale, bias) of
    // that row at sb_s + (st * R + u) * ng * 8 (copied by the group's first lane, read by all after a __syncwarp)
    uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(gw_smem) + wid * kGwRingBytes + lane * 16;
    uint32_t sb_s = (uint32_t)__cvta_generic_to_shared(gw_smem) + kGwWarps * kGwRingBytes + wid * kGwSbBytes + (lane >> GL) * 8;
    asm volatile("" : "+r"(ring_s), "+r"(sb_s));

    for (int64_t item = (int64_t)blockIdx.x * kGwWarps + wid; item < total; item += warps) {
        int lo_t = 0, hi_t = p.T;
        while (hi_t - lo_t > 1) {
            const int mid = (lo_t + hi_t) >> 1;
            if (item_base[mid] <= item) lo_t = mid; else hi_t = mid;
        }
        const int t = lo_t;
        const TableMeta m = p.meta[t];
        const int lig = lane & (G - 1), grp = lane >> GL;
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
        // (a bag of 2^31 lookups or more is walked up to its first 2^31 - 1)
        const uint32_t L = hi - lo > 0x7fffffffll ? 0x7fffffffu : (uint32_t)(hi - lo);
        const uint32_t Lmax = __reduce_max_sync(0xffffffffu, L);
        const char* __restrict__ ids_bag = static_cast<const char*>(p.indices) + lo * (p.idx32 ? 4 : 8);
        float* __restrict__ gw_bag = p.grad_w + lo;
        // (a table without rows may come without memory: its copies, all of zero bytes, name grad_out)
        const char* __restrict__ tbase = m.rows > 0 ? static_cast<const char*>(p.tables[t])
                                                    : reinterpret_cast<const char*>(p.grad_out);
        const float* __restrict__ go = p.grad_out + b * (int64_t)p.sumD + m.D_off;
        const bool inv_on = p.mean && L > 0;
        const uint32_t rows = (uint32_t)m.rows;             // tables have fewer than 2^31 rows
        const uint32_t stride = (uint32_t)m.stride;
        // after the butterfly this lane holds the sums of n_mine rows of the batch, from row_mine on
        constexpr int halvings = GL < 3 ? GL : 3;
        constexpr int n_mine = R >> halvings;
        int row_mine = 0;
#pragma unroll
        for (int k = 1; k <= halvings; ++k) row_mine += ((lig >> (GL - k)) & 1) * (R >> k);
        const bool writer = (lig & ((G >> halvings) - 1)) == 0;

        for (int c0 = 0; c0 < m.nvec; c0 += G) {                  // column tiles of G row vectors
            const int vec = c0 + lig;
            const bool on = vec < m.nvec && L > 0;
            const bool last_tile = c0 + G >= m.nvec;
            float2 g[NACC / 2];
            float sum_g = 0.0f;                                  // rowwise 8-bit: what the row's bias multiplies
#pragma unroll
            for (int k = 0; k < NACC; k += 4) {
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (on) x = __ldg(reinterpret_cast<const float4*>(go + (size_t)vec * NACC + k));
                g[k / 2] = make_float2(x.x, x.y);
                g[k / 2 + 1] = make_float2(x.z, x.w);
                if (DT == DT_INT8) sum_g += (x.x + x.y) + (x.z + x.w);
            }
            const char* __restrict__ lane_base = tbase + vec * 16;
            // Ids: lane k < C of a group loads the k-th id of a batch (C = min(G, R) rows per batch),
            // two batches before its rows are used; `raw` is looked at one iteration after its load.
            constexpr int C = G < R ? G : R;
            int64_t raw = 0;
            bool raw_live = false;
            uint32_t idn = kGwNoRow;                             // lane k: row k of the batch to request next
            auto fetch_id = [&](uint32_t j0) {
                raw_live = lig < C && j0 + lig < L;
                if (raw_live)
                    raw = p.idx32 ? (int64_t)__ldg(reinterpret_cast<const int*>(ids_bag) + (j0 + lig))
                                  : (int64_t)__ldg(reinterpret_cast<const long long*>(ids_bag) + (j0 + lig));
            };
            auto check_id = [&]() {
                idn = kGwNoRow;
                if (raw_live) {
                    if ((uint64_t)raw < (uint64_t)rows) idn = (uint32_t)raw;
                    else if (c0 == 0) ++n_oob;
                }
            };
            // Request the rows of the batch in idn into stage st.  Every slot gets a copy: one of
            // zero source bytes (which fills the slot with zeros and reads nothing) where the row is
            // missing (past the bag's end, an id outside the table, a lane past the row's end), so
            // neither side has anything to branch on.  Bit k of the result: the batch's row k exists.
            auto request_rows = [&](uint32_t slot_s, uint32_t sbslot_s, auto wide) {
#pragma unroll
                for (int k = 0; k < R; ++k) {
                    uint32_t r = __shfl_sync(0xffffffffu, idn, wide.value ? k : (k & (G - 1)), G);
                    if (!wide.value && k >= G) r = kGwNoRow;
                    const bool have = r != kGwNoRow && on;
                    const uint64_t roff = (uint64_t)(have ? r : 0u) * stride;
                    cp_async16_zfill(slot_s + k * 512, lane_base + roff, have ? 16u : 0u);
                    if (DT == DT_INT8 && lig == 0) cp_async8_zfill(sbslot_s + k * (ng * 8), tbase + roff + m.D, have ? 8u : 0u);
                }
            };
            auto request = [&](uint32_t slot_s, uint32_t sbslot_s) {
                const unsigned present = __ballot_sync(0xffffffffu, idn != kGwNoRow);
                request_rows(slot_s, sbslot_s, std::integral_constant<bool, (G >= R)>());
                cp_async_commit();
                return (present >> (lane & ~(G - 1))) & ((1u << C) - 1u);
            };
            fetch_id(0);
            check_id();
            fetch_id(C);
            // the stage being used and the one being filled, as addresses in the shared window
            uint32_t slot_c = ring_s, slot_n = ring_s + R * 512;
            uint32_t sb_c = sb_s, sb_n = sb_s + R * (ng * 8);
            unsigned valid_c = request(slot_c, sb_c);
            for (uint32_t j0 = 0; j0 < Lmax; j0 += C) {
                check_id();                                      // the batch after this one: loaded an iteration ago
                fetch_id(j0 + 2 * C);
                const unsigned valid_n = request(slot_n, sb_n);
                cp_async_wait<1>();                              // everything but the newest group has landed
                if (DT == DT_INT8) __syncwarp();                 // (the pairs were copied by the groups' first lanes)
                float s[R];
#pragma unroll
                for (int k = 0; k < R; ++k) {
                    const uint4 d = lds128(slot_c + k * 512);
                    s[k] = dot_vec<DT>(g, d, p.code_zero);
                    if (DT == DT_INT8) {                         // sum g * (scale * q + bias) = scale * sum g q + bias * sum g
                        const float2 sb = lds64f(sb_c + k * (ng * 8));
                        s[k] = fmaf(sb.x, s[k], sb.y * sum_g);
                    }
                }
                // the lanes of the group, added along a butterfly (partner distances G/2, G/4, .. 1):
                // while a lane holds more than one row's value it keeps half and hands over half
                if constexpr (G >= 2) {
                    constexpr int o = G >> 1;
                    const bool up = (lig & o) != 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float keep = up ? s[i + 4] : s[i], send = up ? s[i] : s[i + 4];
                        s[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                    }
                }
                if constexpr (G >= 4) {
                    constexpr int o = G >> 2;
                    const bool up = (lig & o) != 0;
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const float keep = up ? s[i + 2] : s[i], send = up ? s[i] : s[i + 2];
                        s[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                    }
                }
                if constexpr (G >= 8) {
                    constexpr int o = G >> 3;
                    const bool up = (lig & o) != 0;
                    const float keep = up ? s[1] : s[0], send = up ? s[0] : s[1];
                    s[0] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                }
#pragma unroll
                for (int o = G >> 4; o > 0; o >>= 1) s[0] += __shfl_xor_sync(0xffffffffu, s[0], o);
                {
                    // lookups of this bag in this batch (none if the bag ended before it)
                    const int rem = L <= j0 ? 0 : (L - j0 < (uint32_t)C ? (int)(L - j0) : C);
                    auto write = [&](int row, float x) {
                        if (!((valid_c >> row) & 1u)) x = 0.0f;          // an id outside the table: 0
                        float* out = gw_bag + (j0 + row);
                        if (c0 > 0) x += *out;                           // later column tiles add to the first one's
                        if (inv_on && last_tile) x = __fdiv_rn(x, (float)L);
                        *out = x;
                    };
                    if constexpr (G >= R) {                              // one row per writing lane
                        if (writer && row_mine < rem) write(row_mine, s[0]);
                    } else if (writer) {
#pragma unroll
                        for (int i = 0; i < R; ++i)
                            if (i < n_mine && row_mine + i < rem) write(row_mine + i, s[i]);
                    }
                }
                valid_c = valid_n;
                const uint32_t x0 = slot_c, x1 = sb_c;
                slot_c = slot_n; slot_n = x0;
                sb_c = sb_n; sb_n = x1;
            }
            cp_async_wait<0>();
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

size_t bwd_weights_smem_bytes(int dtype, int T) {
    return (size_t)kGwWarps * (kGwRingBytes + (dtype == DT_INT8 ? kGwSbBytes : 0)) + (size_t)(T + 1) * sizeof(int);
}

template <int DT, int GL>
static cudaError_t launch_class(const BwdWeightsParams& p, int num_sms, cudaStream_t s) {
    const size_t smem = bwd_weights_smem_bytes(DT, p.T);
    static bool set[64] = {};                            // per device: the shared-memory limit has been raised
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !set[dev]) {
        e = cudaFuncSetAttribute(ebag_bwd_weights_kernel<DT, GL>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) set[dev] = true;
    }
    ebag_bwd_weights_kernel<DT, GL><<<num_sms * 3, kGwThreads, smem, s>>>(p);
    return cudaGetLastError();
}

template <int DT>
static cudaError_t launch_one(const BwdWeightsParams& p, unsigned classes, int num_sms, cudaStream_t s, int* launches) {
    cudaError_t e = cudaSuccess;
    if (e == cudaSuccess && (classes & 4u)) { e = launch_class<DT, 2>(p, num_sms, s); ++*launches; }
    if (e == cudaSuccess && (classes & 8u)) { e = launch_class<DT, 3>(p, num_sms, s); ++*launches; }
    if (e == cudaSuccess && (classes & 16u)) { e = launch_class<DT, 4>(p, num_sms, s); ++*launches; }
    if (e == cudaSuccess && (classes & 32u)) { e = launch_class<DT, 5>(p, num_sms, s); ++*launches; }
    return e;
}

cudaError_t launch_bwd_weights(int dtype, const BwdWeightsParams& p, unsigned classes, int num_sms, cudaStream_t s,
                               int* launches) {
    *launches = 0;
    switch (dtype) {
        case DT_F32: return launch_one<DT_F32>(p, classes, num_sms, s, launches);
        case DT_F16: return launch_one<DT_F16>(p, classes, num_sms, s, launches);
        case DT_BF16: return launch_one<DT_BF16>(p, classes, num_sms, s, launches);
        default: return launch_one<DT_INT8>(p, classes, num_sms, s, launches);
    }
}

}  // namespace ebag
