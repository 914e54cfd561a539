// Preprocessing producers of embedding ids that sit in front of the pooled forward
// (paper Sec. 5.4 "Data Preprocessing Kernels on MTIA").  Contracts are in include/ebag.h.
#include <cuda_runtime.h>

#include "ebag.h"

namespace {

constexpr int kThreads = 256;
constexpr int kSmemBorders = 64;     // border lists up to this long are counted linearly from smem
constexpr int kIlp = 16;             // values per thread in flight at 3 CTAs per SM (8, 12, 32 and 2 or 4 CTAs measured slower)

// Launches here are made with programmatic stream serialization: the CTAs of a launch may become
// resident while the launch before it on the stream drains, and wait here for its results.
__device__ __forceinline__ void wait_for_previous_launch() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
}

inline cudaLaunchConfig_t serialized_launch(dim3 grid, unsigned threads, cudaStream_t s, cudaLaunchAttribute* attr) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(threads);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cfg;
}

// MergeBucketizedDense (Sec. 5.4.2): out[f, i] = #borders of feature f below values[f, i] + off[f].
// blockIdx.y is the feature.  "Below" is written !(x <= b) so that NaN lands in the last bin,
// like the library routine the paper's pseudocode calls.  Short lists are counted linearly
// (the vectorised counting the paper's kernel uses), long ones by a branch-free halving search.
template <bool VEC>       // VEC: B is a multiple of 4, values 16-byte and out 32-byte aligned
__global__ void __launch_bounds__(kThreads, 3)
mbdt_kernel(const float* __restrict__ values, int64_t B, const float* __restrict__ borders,
            const int64_t* __restrict__ border_offsets, const int64_t* __restrict__ out_offsets,
            int64_t* __restrict__ out) {
    __shared__ float sb[kSmemBorders];
    wait_for_previous_launch();
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
    // bin of one value
    auto bin = [&](float x) -> int {
        if (K <= kSmemBorders) {
            int n = 0;
            for (int j = 0; j < K; ++j) n += !(x <= sb[j]);
            return n;
        }
        int lo = 0, hi = K;
        const int steps = 32 - __clz(K);
        for (int s = 0; s < steps; ++s) {
            const int mid = (lo + hi) >> 1;
            const float b = __ldg(bf + (mid < K ? mid : K - 1));
            const bool active = lo < hi;
            const bool right = !(x <= b);
            lo = (active && right) ? mid + 1 : lo;
            hi = (active && !right) ? mid : hi;
        }
        return lo;
    };
    if (VEC) {
        // four consecutive values per thread and access: one 16-byte load, one 32-byte store (a
        // whole sector per lane; two 16-byte stores per lane would each write half of every sector
        // the warp touches: 0.186 ms against 0.154 ms with dense stores)
        const int64_t B4 = B >> 2;
        const float4* __restrict__ v4 = reinterpret_cast<const float4*>(vf);
        constexpr int kQuads = kIlp / 4;
        for (int64_t i = blockIdx.x * (int64_t)kThreads + threadIdx.x; i < B4; i += kQuads * stride) {
            float x[kIlp];
#pragma unroll
            for (int q = 0; q < kQuads; ++q) {
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                if (i + q * stride < B4) a = __ldcs(v4 + i + q * stride);
                x[4 * q] = a.x;
                x[4 * q + 1] = a.y;
                x[4 * q + 2] = a.z;
                x[4 * q + 3] = a.w;
            }
            int n[kIlp];
            if (K <= kSmemBorders) {
#pragma unroll
                for (int k = 0; k < kIlp; ++k) n[k] = 0;
                for (int j = 0; j < K; ++j) {
                    const float b = sb[j];
#pragma unroll
                    for (int k = 0; k < kIlp; ++k) n[k] += !(x[k] <= b);
                }
            } else {
#pragma unroll
                for (int k = 0; k < kIlp; ++k) n[k] = bin(x[k]);
            }
#pragma unroll
            for (int q = 0; q < kQuads; ++q)
                if (i + q * stride < B4)
                    asm volatile("st.global.cs.v4.b64 [%0], {%1, %2, %3, %4};" ::"l"(of + 4 * (i + q * stride)),
                                 "l"(n[4 * q] + add), "l"(n[4 * q + 1] + add), "l"(n[4 * q + 2] + add),
                                 "l"(n[4 * q + 3] + add)
                                 : "memory");
        }
        return;
    }
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
#pragma unroll
            for (int k = 0; k < kIlp; ++k) n[k] = bin(x[k]);
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
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, mbdt_kernel<true>, kThreads, 0) != cudaSuccess) {
        cudaGetLastError();
        return EBAG_ERR_CUDA;
    }
    int64_t bx = (B + kIlp * kThreads - 1) / (kIlp * kThreads);
    int64_t cap = (int64_t)sms * per_sm / F;
    if (cap < 1) cap = 1;
    if (bx > cap) bx = cap;
    const bool vec = (B & 3) == 0 && !((uintptr_t)values & 15u) && !((uintptr_t)out & 31u);
    cudaLaunchAttribute attr[1];
    cudaLaunchConfig_t cfg = serialized_launch(dim3((unsigned)bx, (unsigned)F), kThreads, (cudaStream_t)stream, attr);
    const cudaError_t err = vec ? cudaLaunchKernelEx(&cfg, mbdt_kernel<true>, values, B, borders, border_offsets,
                                                     out_offsets, out)
                                : cudaLaunchKernelEx(&cfg, mbdt_kernel<false>, values, B, borders, border_offsets,
                                                     out_offsets, out);
    if (err != cudaSuccess) {
        cudaGetLastError();
        return EBAG_ERR_CUDA;
    }
    return EBAG_OK;
}

// ---------------------------------------------------------------------------------------------
// Batch Event Truncate (paper Sec. 5.5): keep the first N events of every user in every feature
// of a nested jagged batch, all features in a constant number of launches.  The kept events of a
// user are a prefix of that user's events, so per feature a user's kept inner lengths and kept
// values are each ONE contiguous range; only user-level prefix sums are needed:
//   1. scan outer lengths            -> first event of every user, before and after (1 CTA per tile)
//   2. per (feature, user) sums      -> values held / kept by the user; the kept inner lengths are
//                                       written out as they are read       (a warp per 8 users)
//   3. scan those per feature        -> first value of every user, before and after (1 CTA per tile)
//   4. copy the kept values per (feature, user)                            (a warp per 8 users)
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

// Exclusive prefix sums of a[0..n) and b[0..n), totals written at index n (negative entries count
// as 0), by a grid of CTAs with no communication between them: the CTA of tile c first ADDS UP
// everything before its tile (a plain reduction with many loads in flight, served by L2 once the
// first CTA has touched the data; redundant, but a few hundred KB), then scans its own tile of
// kScanThreads * kScanItems entries in one round.  CLAMP: b is not read, b[i] = min(a[i], clamp)
// and is also written to b_out.  At 32,768 entries a single CTA walking the tiles one after the
// other took 56-60 us per scan, a fifth of the whole truncation.
constexpr int kScanItems = 4;
constexpr int kScanTile = kScanThreads * kScanItems;
__device__ __forceinline__ int64_t nonneg(int64_t x) { return x < 0 ? 0 : x; }

template <bool CLAMP>
__device__ void tile_exscan2(const int64_t* __restrict__ a, const int64_t* __restrict__ b, int64_t clamp,
                             int64_t n, int64_t tile, int64_t* __restrict__ b_out,
                             int64_t* __restrict__ sa, int64_t* __restrict__ sb) {
    __shared__ int64_t warp_a[32], warp_b[32], base[2];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int64_t t0 = tile * kScanTile;
    auto bval = [&](int64_t av, int64_t i) -> int64_t {
        if (CLAMP) return av < clamp ? av : clamp;
        return nonneg(b[i]);
    };
    // ---- the tile's own entries, kScanItems consecutive ones per thread: requested first, so
    // that they travel while everything before the tile is added up
    const int64_t i0 = t0 + (int64_t)tid * kScanItems;
    int64_t xa[kScanItems], xb[kScanItems];
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
        xa[k] = i0 + k < n ? nonneg(a[i0 + k]) : 0;
        xb[k] = i0 + k < n ? bval(xa[k], i0 + k) : 0;
    }
    // ---- everything before the tile
    int64_t pa = 0, pb = 0;
    for (int64_t j0 = tid; j0 < t0; j0 += (int64_t)kScanThreads * 8) {
        int64_t ya[8], yb[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int64_t i = j0 + (int64_t)k * kScanThreads;
            ya[k] = i < t0 ? nonneg(a[i]) : 0;
            yb[k] = i < t0 ? bval(ya[k], i) : 0;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) { pa += ya[k]; pb += yb[k]; }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        pa += __shfl_xor_sync(0xffffffffu, pa, d);
        pb += __shfl_xor_sync(0xffffffffu, pb, d);
    }
    if (lane == 0) { warp_a[wid] = pa; warp_b[wid] = pb; }
    __syncthreads();
    if (wid == 0) {
        int64_t wa = warp_a[lane], wb = warp_b[lane];
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            wa += __shfl_xor_sync(0xffffffffu, wa, d);
            wb += __shfl_xor_sync(0xffffffffu, wb, d);
        }
        if (lane == 0) { base[0] = wa; base[1] = wb; }
    }
    __syncthreads();
    // ---- the tile itself (its entries were requested before the reduction above)
    int64_t ta = 0, tb = 0;                          // this thread's totals
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
        ta += xa[k];
        tb += xb[k];
    }
    int64_t ia = ta, ib = tb;                        // inclusive over the threads of the warp
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int64_t ya = __shfl_up_sync(0xffffffffu, ia, d), yb = __shfl_up_sync(0xffffffffu, ib, d);
        if (lane >= d) { ia += ya; ib += yb; }
    }
    __syncthreads();                                 // warp_a / warp_b are reused
    if (lane == 31) { warp_a[wid] = ia; warp_b[wid] = ib; }
    __syncthreads();
    if (wid == 0) {
        int64_t wa = warp_a[lane], wb = warp_b[lane];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int64_t ya = __shfl_up_sync(0xffffffffu, wa, d), yb = __shfl_up_sync(0xffffffffu, wb, d);
            if (lane >= d) { wa += ya; wb += yb; }
        }
        warp_a[lane] = wa; warp_b[lane] = wb;          // inclusive over warps
    }
    __syncthreads();
    int64_t ra = base[0] + (wid ? warp_a[wid - 1] : 0) + ia - ta;   // exclusive for this thread
    int64_t rb = base[1] + (wid ? warp_b[wid - 1] : 0) + ib - tb;
#pragma unroll
    for (int k = 0; k < kScanItems; ++k) {
        if (i0 + k < n) {
            sa[i0 + k] = ra;
            sb[i0 + k] = rb;
            if (CLAMP) b_out[i0 + k] = xb[k];
        }
        ra += xa[k];
        rb += xb[k];
    }
    if (t0 + kScanTile >= n && tid == kScanThreads - 1) {           // the last tile also leaves the totals
        sa[n] = base[0] + warp_a[31];
        sb[n] = base[1] + warp_b[31];
    }
}

__global__ void __launch_bounds__(kScanThreads)
bet_scan_outer(const int64_t* __restrict__ outer, int64_t U, int64_t N, int64_t* __restrict__ outer_out,
               BetWorkspace w, int64_t* __restrict__ counts_out) {
    wait_for_previous_launch();
    tile_exscan2<true>(outer, nullptr, N, U, blockIdx.x, outer_out, w.ev_in, w.ev_out);
    if ((int64_t)(blockIdx.x + 1) * kScanTile >= U) {
        __syncthreads();
        if (threadIdx.x == 0) counts_out[0] = w.ev_out[U];
    }
}

constexpr int kCopyBatch = 4;       // 8-byte loads a lane keeps in flight
constexpr int kTaskUsers = 8;       // users per warp task
constexpr int kSumBatch = 6;        // bet_user_sums: loads per lane requested one user ahead (192 inner lengths)

// How many values every user holds in a feature and how many its kept events hold.  A warp takes
// kTaskUsers consecutive users of a feature at a time: a lane each reads the event range of one
// of them, then the warp adds up the users' inner lengths one user after the other.  The grid is
// one wave of resident CTAs and the (feature, users) tasks are dealt round-robin to its warps.
__global__ void __launch_bounds__(256, 4)
bet_user_sums(const int64_t* __restrict__ inner, int64_t E, int64_t U, int F, BetWorkspace w,
              int64_t* __restrict__ inner_out) {
    wait_for_previous_launch();
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t chunks = (U + kTaskUsers - 1) / kTaskUsers;       // per feature
    auto clamp_e = [&](int64_t x) { return x < 0 ? 0 : (x > E ? E : x); };   // never read or write past the arrays
    for (int64_t task = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); task < chunks * F;
         task += warps) {
        const int f = (int)(task / chunks);
        const int64_t u0 = (task - (int64_t)f * chunks) * kTaskUsers;
        const int users = U - u0 < kTaskUsers ? (int)(U - u0) : kTaskUsers;
        // Lane k holds user u0 + k: its event count, how many of them are kept, and where its kept
        // inner lengths go, the latter relative to the task's first user (E < 2^31, so 32 bits
        // hold everything below; the users of a task follow one another in the input, so the
        // read position simply runs on).
        const int64_t a0 = clamp_e(w.ev_in[u0]), o0 = clamp_e(w.ev_out[u0]);
        int c = 0, kp = 0, orel = 0;
        if (lane < users) {
            const int64_t a = clamp_e(w.ev_in[u0 + lane]), b = clamp_e(w.ev_in[u0 + lane + 1]);
            const int64_t oa = clamp_e(w.ev_out[u0 + lane]), ob = clamp_e(w.ev_out[u0 + lane + 1]);
            c = (int)(b - a);
            kp = (int)(ob - oa < b - a ? ob - oa : b - a);
            orel = (int)(oa - o0);
        }
        const long long* __restrict__ src = reinterpret_cast<const long long*>(inner + (int64_t)f * E + a0) + lane;
        long long* __restrict__ dst0 = reinterpret_cast<long long*>(inner_out + (int64_t)f * E + o0) + lane;
        int64_t my_all = 0, my_kept = 0;              // results of user u0 + lane
        // the first kSumBatch * 32 inner lengths of the NEXT user are requested before the
        // current user's are added up, so that a warp always has a user's worth of loads in flight
        long long cur[kSumBatch], nxt[kSumBatch];
        int cnt = __shfl_sync(0xffffffffu, c, 0);
#pragma unroll
        for (int q = 0; q < kSumBatch; ++q) cur[q] = lane + 32 * q < cnt ? __ldcs(src + 32 * q) : 0;
        for (int k = 0; k < users; ++k) {
            const int keep = __shfl_sync(0xffffffffu, kp, k);
            long long* __restrict__ dst = dst0 + __shfl_sync(0xffffffffu, orel, k);
            const int cnt_n = __shfl_sync(0xffffffffu, c, (k + 1) & 31);     // 0 behind the task's last user
            const long long* __restrict__ src_n = src + cnt;
#pragma unroll
            for (int q = 0; q < kSumBatch; ++q) nxt[q] = lane + 32 * q < cnt_n ? __ldcs(src_n + 32 * q) : 0;
            // the kept inner lengths go to the output as they pass through (they are a prefix of
            // the user's, so this is the whole copy of that array: the copy kernel moves values only)
            int64_t all = 0, kept = 0;
#pragma unroll
            for (int q = 0; q < kSumBatch; ++q) {
                const int64_t n = nonneg(cur[q]);
                all += n;
                if (lane + 32 * q < keep) {
                    kept += n;
                    __stcs(dst + 32 * q, n);
                }
            }
            for (int j0 = 32 * kSumBatch; j0 < cnt; j0 += 32 * kCopyBatch) {       // the rest, if any
                long long x[kCopyBatch];
#pragma unroll
                for (int q = 0; q < kCopyBatch; ++q) x[q] = lane + j0 + 32 * q < cnt ? __ldcs(src + j0 + 32 * q) : 0;
#pragma unroll
                for (int q = 0; q < kCopyBatch; ++q) {
                    const int64_t n = nonneg(x[q]);
                    all += n;
                    if (lane + j0 + 32 * q < keep) {
                        kept += n;
                        __stcs(dst + j0 + 32 * q, n);
                    }
                }
            }
            // the lanes' sums added up: one warp reduction each while every lane's sum is below
            // 2^26 (then the total fits 32 bits), else five 64-bit shuffle steps
            if (!__any_sync(0xffffffffu, all >= (1ll << 26))) {
                all = (int64_t)__reduce_add_sync(0xffffffffu, (unsigned)all);
                kept = (int64_t)__reduce_add_sync(0xffffffffu, (unsigned)kept);
            } else {
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) {
                    all += __shfl_xor_sync(0xffffffffu, all, d);
                    kept += __shfl_xor_sync(0xffffffffu, kept, d);
                }
            }
            if (lane == k) { my_all = all; my_kept = kept; }
            src = src_n;
            cnt = cnt_n;
#pragma unroll
            for (int q = 0; q < kSumBatch; ++q) cur[q] = nxt[q];
        }
        if (lane < users) {                            // coalesced
            w.v_all[(int64_t)f * U + u0 + lane] = my_all;
            w.v_keep[(int64_t)f * U + u0 + lane] = my_kept;
        }
    }
}

__global__ void __launch_bounds__(kScanThreads)
bet_scan_values(int64_t U, BetWorkspace w, int64_t* __restrict__ counts_out) {
    wait_for_previous_launch();
    const int f = blockIdx.y;
    tile_exscan2<false>(w.v_all + (int64_t)f * U, w.v_keep + (int64_t)f * U, 0, U, blockIdx.x, nullptr,
                        w.v_in + (int64_t)f * (U + 1), w.v_out + (int64_t)f * (U + 1));
    if ((int64_t)(blockIdx.x + 1) * kScanTile >= U) {
        __syncthreads();
        if (threadIdx.x == 0) counts_out[1 + f] = w.v_out[(int64_t)f * (U + 1) + U];
    }
}

// Copies `n` 8-byte words src -> dst with a warp, kCopyBatch loads in flight per lane.
template <bool CLAMP, int BATCH = kCopyBatch>
__device__ __forceinline__ void warp_copy64(const int64_t* __restrict__ src, int64_t* __restrict__ dst,
                                            int64_t n, int lane) {
    for (int64_t j0 = lane; j0 < n; j0 += 32 * BATCH) {
        long long x[BATCH];
#pragma unroll
        for (int k = 0; k < BATCH; ++k) {
            const int64_t j = j0 + 32 * k;
            x[k] = j < n ? __ldcs(reinterpret_cast<const long long*>(src + j)) : 0;
        }
#pragma unroll
        for (int k = 0; k < BATCH; ++k) {
            const int64_t j = j0 + 32 * k;
            if (j < n) __stcs(reinterpret_cast<long long*>(dst + j), CLAMP && x[k] < 0 ? 0 : x[k]);
        }
    }
}

// A warp takes kTaskUsers consecutive users of a feature at a time: a lane each reads the range
// of one of them, then the warp copies the users' kept values, contiguous per user, one user
// after the other.  Same task dealing as bet_user_sums.
__global__ void __launch_bounds__(256, 4)
bet_copy(const int64_t* __restrict__ values, const int64_t* __restrict__ value_offsets, int64_t U, int F,
         BetWorkspace w, int64_t* __restrict__ values_out) {
    wait_for_previous_launch();
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t chunks = (U + kTaskUsers - 1) / kTaskUsers;       // per feature
    for (int64_t task = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); task < chunks * F;
         task += warps) {
        const int f = (int)(task / chunks);
        const int64_t u0 = (task - (int64_t)f * chunks) * kTaskUsers;
        const int64_t vbase = value_offsets[f], vend = value_offsets[f + 1];
        const int64_t u = u0 + lane;
        int64_t v_in = 0, v_out = 0, nv = 0;
        if (lane < kTaskUsers && u < U) {
            v_in = vbase + w.v_in[(int64_t)f * (U + 1) + u];
            v_out = vbase + w.v_out[(int64_t)f * (U + 1) + u];
            nv = w.v_keep[(int64_t)f * U + u];
            if (v_in + nv > vend) nv = vend > v_in ? vend - v_in : 0;   // stay inside the feature's values
        }
        const int users = U - u0 < kTaskUsers ? (int)(U - u0) : kTaskUsers;
        for (int k = 0; k < users; ++k) {
            const int64_t kv_in = __shfl_sync(0xffffffffu, v_in, k), kv_out = __shfl_sync(0xffffffffu, v_out, k);
            const int64_t knv = __shfl_sync(0xffffffffu, nv, k);
            warp_copy64<false, 8>(values + kv_in, values_out + kv_out, knv, lane);   // 8 loads in flight
        }
    }
}

// One wave of resident 256-thread CTAs, or fewer when there are fewer tasks than warps.
template <typename K>
unsigned bet_grid(K kernel, int F, int64_t U) {
    int dev = 0, sms = 148, per_sm = 4;
    if (cudaGetDevice(&dev) == cudaSuccess) {
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, 256, 0) != cudaSuccess || per_sm < 1)
            per_sm = 4;
    }
    cudaGetLastError();
    const int64_t tasks = ((U + kTaskUsers - 1) / kTaskUsers) * F;
    const int64_t need = (tasks + 7) / 8;
    const int64_t wave = (int64_t)sms * per_sm;
    return (unsigned)(need < wave ? (need > 0 ? need : 1) : wave);
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
    if (E >= (1ll << 31)) return EBAG_ERR_UNSUPPORTED;     // positions inside a feature travel in 32 bits
    if (!counts_out) return EBAG_ERR_INVALID_ARG;
    if (U > 0 && (!outer_lengths || !outer_out)) return EBAG_ERR_INVALID_ARG;
    if (F > 0 && (!value_offsets || (E > 0 && (!inner_lengths || !inner_out)))) return EBAG_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < ebag_bet_workspace_bytes(F, U) || ((uintptr_t)workspace & 7u))
        return EBAG_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    const BetWorkspace w = carve(workspace, F, U);
    const unsigned tiles = (unsigned)(U > 0 ? (U + kScanTile - 1) / kScanTile : 1);
    cudaLaunchAttribute attr[1];
    auto config = [&](dim3 grid, unsigned threads) { return serialized_launch(grid, threads, s, attr); };
    cudaError_t err;
    {
        cudaLaunchConfig_t cfg = config(dim3(tiles), kScanThreads);
        err = cudaLaunchKernelEx(&cfg, bet_scan_outer, outer_lengths, U, N, outer_out, w, counts_out);
    }
    if (err == cudaSuccess && F > 0 && U > 0) {
        cudaLaunchConfig_t cfg = config(dim3(bet_grid(bet_user_sums, F, U)), 256);
        err = cudaLaunchKernelEx(&cfg, bet_user_sums, inner_lengths, E, U, (int)F, w, inner_out);
    }
    if (err == cudaSuccess && F > 0) {
        cudaLaunchConfig_t cfg = config(dim3(tiles, (unsigned)F), kScanThreads);
        err = cudaLaunchKernelEx(&cfg, bet_scan_values, U, w, counts_out);
    }
    if (err == cudaSuccess && F > 0 && U > 0) {
        cudaLaunchConfig_t cfg = config(dim3(bet_grid(bet_copy, F, U)), 256);
        err = cudaLaunchKernelEx(&cfg, bet_copy, values, value_offsets, U, (int)F, w, values_out);
    }
    if (err != cudaSuccess) {
        cudaGetLastError();
        return EBAG_ERR_CUDA;
    }
    if (cudaGetLastError() != cudaSuccess) return EBAG_ERR_CUDA;
    return EBAG_OK;
}
