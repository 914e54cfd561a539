// Reproducible backward of the pooled embedding-bag forward (sm_100a): no floating-point atomics.
//
//     grad_t[indices[i], d] += w_i * grad_out[b, Doff[t] + d] * (1/L in mean mode)
//
// The other backward kernel (ebag_bwd.cu) sends every lookup's contribution to its row with a
// vector reduction, so the order of the additions, and with it the last bits of the result,
// depends on timing, and the hot rows of a skewed table queue up in L2.  Here the lookups of
// every table are first SORTED BY ROW, stably, so that the contributions to one row sit next to
// each other in the order of the lookups, and then every run of equal rows is added up by one
// warp in that order and added into its gradient row ONCE (one vector reduction per row and call:
// a single addend per element, so there is no order to depend on).  Two runs of the same call
// give the same bits.
//
//   1. check     offsets non-decreasing inside [0, n]?  If not, this pipeline steps aside (every
//                kernel below returns at once) and the reduction kernel runs instead: with
//                overlapping bags a lookup no longer has one place in the sorted list.
//   2. plan      first lookup and first sorting tile of every table
//   3. expand    per lookup: key = row (rows[t] for a skipped id, which sorts to the end of the
//                table and is ignored), bag, weight / bag length
//   4. sort      least-significant-digit radix sort, 8 bits a pass, as many passes as the largest
//                table's row ids need, tables sorted side by side: per pass a histogram per tile
//                (2048 lookups), running sums per (table, digit) over the tiles, and a stable
//                scatter (ranks inside a tile by warp-wide matching, in lookup order)
//   5. run sums  a warp per unit (table, column tile of 128 columns, 1024 sorted lookups): walks
//                it in order, eight grad_out slices in flight, adds w * grad_out[bag] into
//                registers (lanes tile the columns), and at every change of row adds the sum into
//                the gradient row.  A run cut by the unit's start or end leaves its partial sum
//                in scratch instead.
//   6. join      a warp per cut run: counts its pieces, adds them in order and adds the sum into
//                the row.
#include <cuda_runtime.h>
#include <stdint.h>

#include "ebag_bwd_sorted.cuh"

namespace ebag {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr uint32_t kNoRow = 0xffffffffu;

// table of sorting tile `tile`: last t with tile_base[t] <= tile
__device__ __forceinline__ int table_of_tile(const uint32_t* __restrict__ tile_base, int T, uint32_t tile) {
    int lo = 0, hi = T;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (tile_base[mid] <= tile) lo = mid; else hi = mid;
    }
    return lo;
}

// ---- 1. offsets non-decreasing inside [0, n]?
__global__ void __launch_bounds__(256) bwds_check_kernel(const BwdSortedParams p) {
    const int64_t n_off = (int64_t)p.T * p.B;
    bool bad = false;
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < n_off; g += (int64_t)gridDim.x * blockDim.x) {
        const int64_t a = p.offsets[g], b = p.offsets[g + 1];
        bad = bad || a < 0 || b < a || b > p.n_indices;
    }
    if (__any_sync(kFull, bad) && (threadIdx.x & 31) == 0) p.ctl[0] = 1;
}

// ---- 2. first lookup and first tile of every table (one CTA)
__global__ void __launch_bounds__(256) bwds_plan_kernel(const BwdSortedParams p) {
    if (p.ctl[0]) return;
    for (int t = threadIdx.x; t <= p.T; t += blockDim.x) p.seg[t] = (uint32_t)p.offsets[(int64_t)t * p.B];
    for (int i = threadIdx.x; i < p.T * 256; i += blockDim.x) p.totals[i] = 0;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t run = 0;
        for (int t = 0; t < p.T; ++t) {
            p.tile_base[t] = run;
            run += (p.seg[t + 1] - p.seg[t] + kSortTile - 1) / kSortTile;
        }
        p.tile_base[p.T] = run;
        // units of the run sums: column tiles of 128 columns x sub-chunks
        uint32_t units = 0;
        for (int t = 0; t < p.T; ++t) {
            p.unit_base[t] = units;
            units += (uint32_t)((p.meta[t].nvec + 31) / 32) * ((p.seg[t + 1] - p.seg[t] + kSubChunk - 1) / kSubChunk);
        }
        p.unit_base[p.T] = units;
    }
}

// ---- 3. one key, bag and weight per lookup.  A warp takes 32 consecutive bags; their lookups
// are one contiguous range, walked 128 at a time (the four loads of a step are issued together), and each lookup finds its bag among the 32 by
// a five-step search over the lanes' end offsets.
constexpr int kExpandUnroll = 4;
__global__ void __launch_bounds__(256) bwds_expand_kernel(const BwdSortedParams p) {
    if (p.ctl[0]) return;
    const int lane = threadIdx.x & 31;
    const int64_t n_bags = (int64_t)p.T * p.B;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    unsigned n_oob = 0;
    for (int64_t g0 = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 32; g0 < n_bags; g0 += warps * 32) {
        const int64_t g = g0 + lane < n_bags ? g0 + lane : n_bags - 1;
        const uint32_t lo = (uint32_t)p.offsets[g], hi = g0 + lane < n_bags ? (uint32_t)p.offsets[g + 1] : 0xffffffffu;
        const int t_l = (int)(g / p.B);
        const uint32_t b_l = (uint32_t)(g - (int64_t)t_l * p.B);
        const uint32_t rows_l = (uint32_t)p.meta[t_l].rows;
        const uint32_t len_l = g0 + lane < n_bags ? hi - lo : 0u;
        const int last = n_bags - g0 < 32 ? (int)(n_bags - g0) - 1 : 31;
        const uint32_t p0 = __shfl_sync(kFull, lo, 0);
        const uint32_t p1 = __shfl_sync(kFull, (uint32_t)p.offsets[g + 1], last);
        for (uint32_t base = p0; base < p1; base += 32 * kExpandUnroll) {
            int64_t id[kExpandUnroll];
            float w[kExpandUnroll];
#pragma unroll
            for (int u = 0; u < kExpandUnroll; ++u) {        // every load of the step before any use
                const uint32_t pos = base + 32 * u + lane;
                id[u] = 0;
                w[u] = 1.0f;
                if (pos < p1) {
                    id[u] = p.idx32 ? (int64_t)__ldcs(reinterpret_cast<const int*>(p.indices) + pos)
                                    : (int64_t)__ldcs(reinterpret_cast<const long long*>(p.indices) + pos);
                    if (p.wts[0] && p.weights) w[u] = __ldcs(p.weights + pos);
                }
            }
#pragma unroll
            for (int u = 0; u < kExpandUnroll; ++u) {
                const uint32_t pos = base + 32 * u + lane;
                if (base + 32 * u >= p1) break;              // the whole warp
                const bool have = pos < p1;
                const uint32_t q = have ? pos : p1 - 1;
                int j = 0;                                   // first lane whose bag ends after q
#pragma unroll
                for (int step = 16; step > 0; step >>= 1) {
                    const uint32_t hc = __shfl_sync(kFull, hi, j + step - 1);
                    if (hc <= q) j += step;
                }
                const uint32_t rows = __shfl_sync(kFull, rows_l, j);
                const uint32_t b = __shfl_sync(kFull, b_l, j);
                const uint32_t len = __shfl_sync(kFull, len_l, j);
                if (have) {
                    const bool ok = (uint64_t)id[u] < (uint64_t)rows;
                    if (!ok) ++n_oob;
                    p.kb[0][pos] = make_uint2(ok ? (uint32_t)id[u] : rows, b);
                    if (p.wts[0]) p.wts[0][pos] = p.mean ? __fdiv_rn(w[u], (float)len) : w[u];
                }
            }
        }
    }
    n_oob = __reduce_add_sync(kFull, n_oob);
    if (lane == 0 && n_oob) atomicAdd(&p.status->n_oob, (unsigned long long)n_oob);
}

// ---- 4a. digit counts of every tile
__global__ void __launch_bounds__(256) bwds_hist_kernel(const BwdSortedParams p, int side, int shift) {
    if (p.ctl[0]) return;
    const uint32_t tile = blockIdx.x;
    if (tile >= p.tile_base[p.T]) return;
    __shared__ uint32_t cnt[256];
    cnt[threadIdx.x] = 0;
    __syncthreads();
    const int t = table_of_tile(p.tile_base, p.T, tile);
    const uint32_t k = tile - p.tile_base[t], nt = p.tile_base[t + 1] - p.tile_base[t];
    const uint32_t s0 = p.seg[t] + k * kSortTile;
    const uint32_t s1 = min(p.seg[t + 1], s0 + (uint32_t)kSortTile);
    const uint2* __restrict__ kb = p.kb[side];
    for (uint32_t pos = s0 + threadIdx.x; pos < s1; pos += 256) atomicAdd(&cnt[(kb[pos].x >> shift) & 255u], 1u);
    __syncthreads();
    p.hist[(size_t)256 * p.tile_base[t] + (size_t)threadIdx.x * nt + k] = cnt[threadIdx.x];
}

// ---- 4b. per (digit, table): running sums of the tiles' counts (in place), the total beside them.
// A thread takes a run of consecutive tiles (all its loads in flight at once), the runs' totals
// are scanned across the CTA once; tables of more than 256 * kScanRun tiles go round again.
constexpr int kScanRun = 8;
__global__ void __launch_bounds__(256) bwds_scan_kernel(const BwdSortedParams p) {
    if (p.ctl[0]) return;
    const int d = blockIdx.x, t = blockIdx.y;
    const uint32_t nt = p.tile_base[t + 1] - p.tile_base[t];
    uint32_t* __restrict__ a = p.hist + (size_t)256 * p.tile_base[t] + (size_t)d * nt;
    __shared__ uint32_t warp_sum[8];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t carry = 0;                                   // the same in every thread
    for (uint32_t i0 = 0; i0 < nt; i0 += 256 * kScanRun) {
        const uint32_t first = i0 + threadIdx.x * kScanRun;
        uint32_t x[kScanRun];
#pragma unroll
        for (int k = 0; k < kScanRun; ++k) x[k] = first + k < nt ? a[first + k] : 0u;
        uint32_t mine = 0;
#pragma unroll
        for (int k = 0; k < kScanRun; ++k) mine += x[k];
        uint32_t inc = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(kFull, inc, o);
            if (lane >= o) inc += y;
        }
        __syncthreads();                                  // (warp_sum of the round before has been read)
        if (lane == 31) warp_sum[wid] = inc;
        __syncthreads();
        uint32_t before = carry, all = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            if (w < wid) before += warp_sum[w];
            all += warp_sum[w];
        }
        uint32_t run = before + inc - mine;
#pragma unroll
        for (int k = 0; k < kScanRun; ++k) {
            if (first + k < nt) a[first + k] = run;
            run += x[k];
        }
        carry += all;
    }
    if (threadIdx.x == 0) p.totals[t * 256 + d] = carry;
}

// ---- 4c. stable scatter of a tile.  Warp w owns an eighth of the tile's lookups, consecutive ones,
// 32 per round, so "earlier in the tile" is: a lower warp, an earlier round, a
// lower lane.  The tile is first put in order in shared memory and then written out, so that
// every run of equal digits leaves as one contiguous, coalesced piece.
template <bool WEIGHTS>
__global__ void __launch_bounds__(256, 4) bwds_scatter_kernel(const BwdSortedParams p, int side, int shift) {
    if (p.ctl[0]) return;
    const uint32_t tile = blockIdx.x;
    if (tile >= p.tile_base[p.T]) return;
    __shared__ uint32_t wcnt[8][256];
    __shared__ uint32_t warp_sum[8];
    __shared__ uint32_t gstart[256];                      // where the tile's lookups with digit d go in the output
    __shared__ uint32_t lstart[256];                      // where they sit in the ordered tile
    extern __shared__ __align__(16) unsigned char tile_smem[];   // the ordered tile: (row, bag) pairs, then weights
    uint2* s_kb = reinterpret_cast<uint2*>(tile_smem);
    float* s_w = reinterpret_cast<float*>(tile_smem + (size_t)kSortTile * sizeof(uint2));
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int t = table_of_tile(p.tile_base, p.T, tile);
    const uint32_t k = tile - p.tile_base[t], nt = p.tile_base[t + 1] - p.tile_base[t];
    const uint32_t s0 = p.seg[t] + k * kSortTile;
    const uint32_t s1 = min(p.seg[t + 1], s0 + (uint32_t)kSortTile);
    // the tile's lookups are requested first: they travel while the digits' places are worked out
    const uint2* __restrict__ kb = p.kb[side];
    const float* __restrict__ wts = WEIGHTS ? p.wts[side] : nullptr;
    constexpr int kRounds = kSortTile / 256;              // a warp owns kRounds * 32 consecutive lookups of the tile
    uint2 e[kRounds];
    float wt[kRounds];
#pragma unroll
    for (int r = 0; r < kRounds; ++r) {
        const uint32_t pos = s0 + (wid * kRounds + r) * 32 + lane;
        e[r] = pos < s1 ? __ldcs(kb + pos) : make_uint2(0u, 0u);
        wt[r] = (WEIGHTS && pos < s1) ? __ldcs(wts + pos) : 0.0f;
    }
#pragma unroll
    for (int w = 0; w < 8; ++w) wcnt[w][tid] = 0;
    // where digit `tid` of this tile starts in the output: the table's start, the lookups of the
    // table with a smaller digit, the lookups of earlier tiles with this digit
    const uint32_t tot = p.totals[t * 256 + tid];
    uint32_t inc = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += y;
    }
    if (lane == 31) warp_sum[wid] = inc;
    __syncthreads();
    uint32_t start = p.seg[t] + inc - tot + p.hist[(size_t)256 * p.tile_base[t] + (size_t)tid * nt + k];
    for (int w = 0; w < wid; ++w) start += warp_sum[w];
    gstart[tid] = start;

    uint32_t where[kRounds];                              // digit << 16 | rank among the warp's earlier lookups of that digit
    unsigned peers[kRounds];                              // the lanes of the round with the same digit
#pragma unroll
    for (int r = 0; r < kRounds; ++r) {                   // the matches of all rounds first: they do not depend on one another
        const uint32_t pos = s0 + (wid * kRounds + r) * 32 + lane;
        const uint32_t d = pos < s1 ? (e[r].x >> shift) & 255u : 256u + lane;     // an absent lookup matches nobody
        // The lanes with the same digit.  match.any takes longer the more different values a warp
        // holds: on the lowest digit (32 lookups, close to 32 different values) eight votes, one
        // per bit, are faster (0.64 -> 0.55 ms on the benchmark's first pass); on the higher digits,
        // where sorted neighbours share them, match.any is (0.39-0.50 ms against 0.54).
        if (shift == 0) {
            unsigned same = __ballot_sync(kFull, d < 256u);
#pragma unroll
            for (int bit = 0; bit < 8; ++bit) {
                const unsigned v = __ballot_sync(kFull, (d >> bit) & 1u);
                same &= ((d >> bit) & 1u) ? v : ~v;
            }
            peers[r] = d < 256u ? same : (1u << lane);
        } else {
            peers[r] = __match_any_sync(kFull, d);
        }
        where[r] = d << 16;
    }
#pragma unroll
    for (int r = 0; r < kRounds; ++r) {                   // then the counts, round after round
        const uint32_t d = where[r] >> 16;
        const int leader = __ffs(peers[r]) - 1;
        uint32_t old = 0;
        if (lane == leader && d < 256u) {
            old = wcnt[wid][d];
            wcnt[wid][d] = old + __popc(peers[r]);
        }
        old = __shfl_sync(kFull, old, leader);
        where[r] |= old + __popc(peers[r] & ((1u << lane) - 1u));
        __syncwarp();
    }
    __syncthreads();
    {   // digit `tid`: the warps' counts become their offsets inside the digit's run; the runs' starts in the ordered tile
        uint32_t run = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const uint32_t c = wcnt[w][tid];
            wcnt[w][tid] = run;
            run += c;
        }
        uint32_t inc2 = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t y = __shfl_up_sync(kFull, inc2, o);
            if (lane >= o) inc2 += y;
        }
        __syncthreads();                                  // (warp_sum is reused)
        if (lane == 31) warp_sum[wid] = inc2;
        __syncthreads();
        uint32_t ls = inc2 - run;
        for (int w = 0; w < wid; ++w) ls += warp_sum[w];
        lstart[tid] = ls;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kRounds; ++r) {
        const uint32_t pos = s0 + (wid * kRounds + r) * 32 + lane;
        if (pos < s1) {
            const uint32_t d = where[r] >> 16;
            const uint32_t l = lstart[d] + wcnt[wid][d] + (where[r] & 0xffffu);
            s_kb[l] = e[r];
            if (WEIGHTS) s_w[l] = wt[r];
        }
    }
    __syncthreads();
    uint2* __restrict__ kb_o = p.kb[side ^ 1];
    float* __restrict__ wts_o = WEIGHTS ? p.wts[side ^ 1] : nullptr;
    const uint32_t count = s1 - s0;
    for (uint32_t i = tid; i < count; i += 256) {
        const uint2 x = s_kb[i];
        const uint32_t d = (x.x >> shift) & 255u;
        const uint32_t dst = gstart[d] + (i - lstart[d]);
        kb_o[dst] = x;
        if (WEIGHTS) wts_o[dst] = s_w[i];
    }
}

// ---- 5. run sums.  A unit of work is (table, column tile of 128 columns, sub-chunk of 1024
// sorted lookups), units in that order, so that at any time the grid reads grad_out slices of
// one column tile of one table (65,536 bags x 512 bytes = 32 MB stay in L2; a 256-column table
// read whole does not fit beside the gradient rows being written).
__device__ __forceinline__ int table_of_unit(const uint32_t* __restrict__ unit_base, int T, uint32_t unit) {
    int lo = 0, hi = T;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (unit_base[mid] <= unit) lo = mid; else hi = mid;
    }
    return lo;
}

// Adds a run's sum into its gradient row.  Every element is written once per call (a run is all
// the lookups of its row), so a reduction without a return value does it: nothing to wait for,
// and with a single addend per element the result does not depend on any order.
__device__ __forceinline__ void add_into_row(float* __restrict__ dst, const float4& acc) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(acc.x), "f"(acc.y), "f"(acc.z),
                 "f"(acc.w)
                 : "memory");
}

#ifndef EBAG_RUNSUM_BLOCKS
#define EBAG_RUNSUM_BLOCKS 3
#endif
#ifndef EBAG_RUNSUM_INFLIGHT
#define EBAG_RUNSUM_INFLIGHT 8
#endif
#ifndef EBAG_RUNSUM_INFLIGHT_W
#define EBAG_RUNSUM_INFLIGHT_W 4
#endif
template <bool WEIGHTS>
__global__ void __launch_bounds__(256, EBAG_RUNSUM_BLOCKS) bwds_run_sums_kernel(const BwdSortedParams p, int side) {
    if (p.ctl[0]) return;
    constexpr int kInFlight = WEIGHTS ? EBAG_RUNSUM_INFLIGHT_W : EBAG_RUNSUM_INFLIGHT;                          // lookups whose grad_out slices are in flight together
    const int lane = threadIdx.x & 31;
    // the tables' first units and first lookups, in shared memory: a unit's start-up is then one
    // round of independent loads instead of a chain of them
    extern __shared__ uint32_t runsum_smem[];
    uint32_t* unit_base_s = runsum_smem;                  // [T + 1]
    uint32_t* seg_s = runsum_smem + p.T + 1;              // [T + 1]
    for (int i = threadIdx.x; i <= p.T; i += blockDim.x) {
        unit_base_s[i] = p.unit_base[i];
        seg_s[i] = p.seg[i];
    }
    __syncthreads();
    const uint32_t n_units = unit_base_s[p.T];
    const uint32_t warps = gridDim.x * (blockDim.x >> 5);
    const uint2* __restrict__ kb = p.kb[side];
    const float* __restrict__ wts = WEIGHTS ? p.wts[side] : nullptr;
    for (uint32_t unit = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); unit < n_units; unit += warps) {
        const int t = table_of_unit(unit_base_s, p.T, unit);
        const BwdTableMeta m = p.meta[t];
        const uint32_t seg0 = seg_s[t], seg1 = seg_s[t + 1];
        const uint32_t n_sub = (seg1 - seg0 + kSubChunk - 1) / kSubChunk;
        const uint32_t local = unit - unit_base_s[t];
        const uint32_t c = local / n_sub, sub = local - c * n_sub;
        const uint32_t s0 = seg0 + sub * kSubChunk;
        const uint32_t s1 = min(seg1, s0 + (uint32_t)kSubChunk);
        const int vec = (int)c * 32 + lane;               // this lane's 16-byte vector of the gradient row
        const bool col_on = vec < m.nvec;
        const int vec_ld = col_on ? vec : (int)c * 32;    // lanes past the row's end re-read the tile's first vector; never written
        const uint32_t rows = (uint32_t)m.rows;
        const uint32_t sumD = (uint32_t)p.sumD, D = (uint32_t)m.D;
        float* __restrict__ gcol = p.grad_tables[t] + 4 * vec;
        const float* __restrict__ go = p.grad_out + m.D_off + 4 * vec_ld;
        const uint32_t prev_row = s0 > seg0 ? kb[s0 - 1].x : kNoRow;
        const uint32_t next_row = s1 < seg1 ? kb[s1].x : kNoRow;
        float* __restrict__ head = p.partial + (size_t)unit * 128 + 4 * lane;
        float* __restrict__ tail = p.partial + ((size_t)p.max_units + unit) * 128 + 4 * lane;
        int32_t tail_row = -1, head_flags = 0;

        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        uint32_t cur = kNoRow;
        bool inner = false;                               // the run under way began inside this sub-chunk
        // The run `cur` ends inside the sub-chunk.  (The lookups of skipped ids carry the key
        // rows[t]: they sort to the table's end, are summed like any run and never written.)
        auto close_run = [&]() {
            if (inner) {
                if (col_on && cur < rows) add_into_row(gcol + (uint64_t)cur * D, acc);
            } else if (cur != kNoRow && cur < rows) {
                if (cur == prev_row) {                      // it began before the sub-chunk: a piece for the join
                    if (col_on) *reinterpret_cast<float4*>(head) = acc;
                    head_flags = 1;
                } else if (col_on) {
                    add_into_row(gcol + (uint64_t)cur * D, acc);
                }
            }
            inner = inner || cur != kNoRow;                 // the next run begins inside the sub-chunk unless it is the first
            acc = make_float4(0.f, 0.f, 0.f, 0.f);
        };
        auto add = [&](float w, const float4& g) {
            if (WEIGHTS) {
                acc.x = fmaf(w, g.x, acc.x);
                acc.y = fmaf(w, g.y, acc.y);
                acc.z = fmaf(w, g.z, acc.z);
                acc.w = fmaf(w, g.w, acc.w);
            } else {
                acc.x += g.x;
                acc.y += g.y;
                acc.z += g.z;
                acc.w += g.w;
            }
        };
        // the keys, bags and weights of the next 32 lookups are requested before the current 32 are worked on
        auto fetch = [&](uint32_t base, uint32_t& kk, uint32_t& bb, float& ww) {
            const bool have = base + lane < s1;
            const uint2 x = have ? __ldcs(kb + base + lane) : make_uint2(kNoRow, 0u);
            kk = x.x;
            bb = x.y;
            ww = (WEIGHTS && have) ? __ldcs(wts + base + lane) : 1.0f;
        };
        uint32_t kk, bb, kk_n, bb_n;
        float ww, ww_n;
        fetch(s0, kk, bb, ww);
        for (uint32_t base = s0; base < s1; base += 32) {
            fetch(base + 32, kk_n, bb_n, ww_n);
            const int n = s1 - base < 32 ? (int)(s1 - base) : 32;
            int j0 = 0;
            for (; j0 + kInFlight <= n; j0 += kInFlight) {  // whole groups: nothing to check
                float4 g[kInFlight];
                uint32_t row[kInFlight];
                float w[kInFlight];
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {      // the loads of the group's lookups, together
                    row[u] = __shfl_sync(kFull, kk, j0 + u);
                    const uint32_t b = __shfl_sync(kFull, bb, j0 + u);
                    w[u] = WEIGHTS ? __shfl_sync(kFull, ww, j0 + u) : 1.0f;
                    g[u] = __ldg(reinterpret_cast<const float4*>(go + (uint64_t)b * sumD));
                }
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {      // added in the order of the lookups
                    if (row[u] != cur) {
                        close_run();
                        cur = row[u];
                    }
                    add(w[u], g[u]);
                }
            }
            for (; j0 < n; ++j0) {                          // the ragged end of the sub-chunk
                const uint32_t row = __shfl_sync(kFull, kk, j0);
                const uint32_t b = __shfl_sync(kFull, bb, j0);
                const float w = WEIGHTS ? __shfl_sync(kFull, ww, j0) : 1.0f;
                const float4 g = __ldg(reinterpret_cast<const float4*>(go + (uint64_t)b * sumD));
                if (row != cur) {
                    close_run();
                    cur = row;
                }
                add(w, g);
            }
            kk = kk_n;
            bb = bb_n;
            ww = ww_n;
        }
        // the last run of the sub-chunk
        if (cur != kNoRow && cur < rows) {
            const bool from_before = !inner && cur == prev_row;
            const bool goes_on = cur == next_row;
            if (from_before) {
                if (col_on) *reinterpret_cast<float4*>(head) = acc;
                head_flags = goes_on ? 3 : 1;
            } else if (goes_on) {
                if (col_on) *reinterpret_cast<float4*>(tail) = acc;
                tail_row = (int32_t)cur;
            } else if (col_on) {
                add_into_row(gcol + (uint64_t)cur * D, acc);
            }
        }
        if (lane == 0) {
            p.rec[2 * unit] = tail_row;
            p.rec[2 * unit + 1] = head_flags;
        }
    }
}

// ---- 6. the runs that unit borders cut: a warp per run, from the unit where it starts.  The
// warp first finds how many pieces follow (32 records at a time), then adds them in order with
// eight loads in flight: the hottest rows of a table are cut into hundreds of pieces.
__global__ void __launch_bounds__(256) bwds_join_kernel(const BwdSortedParams p) {
    if (p.ctl[0]) return;
    const int lane = threadIdx.x & 31;
    const uint32_t n_units = p.unit_base[p.T];
    const uint32_t warps = gridDim.x * (blockDim.x >> 5);
    for (uint32_t unit = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); unit < n_units; unit += warps) {
        const int32_t row = p.rec[2 * unit];
        if (row < 0) continue;
        const int t = table_of_unit(p.unit_base, p.T, unit);
        const BwdTableMeta m = p.meta[t];
        const uint32_t n_sub = (p.seg[t + 1] - p.seg[t] + kSubChunk - 1) / kSubChunk;
        const uint32_t c = (unit - p.unit_base[t]) / n_sub;
        const int vec = (int)c * 32 + lane;
        // pieces: units unit + 1 .. unit + count hold a head piece of this run; all but the last say "goes on"
        uint32_t count = 0;
        for (uint32_t k0 = unit + 1; k0 < n_units; k0 += 32) {
            const uint32_t k = k0 + lane;
            const int32_t flags = k < n_units ? p.rec[2 * k + 1] : 0;
            // the chain ends at the first unit that has no piece, or after the first piece that does not go on
            const unsigned none = __ballot_sync(kFull, !(flags & 1));
            const unsigned last = __ballot_sync(kFull, (flags & 1) && !(flags & 2));
            const int first_none = none ? __ffs(none) - 1 : 32;
            const int first_last = last ? __ffs(last) - 1 : 32;
            if (first_last < first_none) {
                count += first_last + 1;
                break;
            }
            count += first_none;
            if (first_none < 32) break;
        }
        if (vec >= m.nvec) continue;
        float4 acc = *reinterpret_cast<const float4*>(p.partial + ((size_t)p.max_units + unit) * 128 + 4 * lane);
        const float* __restrict__ pieces = p.partial + (size_t)(unit + 1) * 128 + 4 * lane;
        for (uint32_t i0 = 0; i0 < count; i0 += 8) {
            float4 x[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                x[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (i0 + i < count) x[i] = *reinterpret_cast<const float4*>(pieces + (size_t)(i0 + i) * 128);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (i0 + i < count) {                       // in order
                    acc.x += x[i].x; acc.y += x[i].y; acc.z += x[i].z; acc.w += x[i].w;
                }
        }
        add_into_row(p.grad_tables[t] + (size_t)row * m.D + 4 * vec, acc);
    }
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace

size_t bwd_sorted_scratch_bytes(int64_t n, int T, int Dmax, bool weighted) {
    const size_t tiles = (size_t)(n / kSortTile) + T + 1;
    size_t b = 0;
    b += 2 * align256((size_t)n * 8);                        // (row, bag) pairs: the two sides of the sort
    if (weighted) b += 2 * align256((size_t)n * 4);
    b += align256(tiles * 256 * 4);                          // hist
    b += align256((size_t)T * 256 * 4);                      // totals
    b += 2 * align256((size_t)(T + 1) * 4);                  // seg, tile_base
    b += align256(256);                                      // ctl
    const size_t units = (size_t)((Dmax + 127) / 128) * ((size_t)(n / kSubChunk) + T + 1);
    b += align256((size_t)(T + 1) * 4);                      // unit_base
    b += align256(2 * units * 128 * 4);                      // partial: a head and a tail piece per unit
    b += align256(2 * units * 4);                            // rec
    return b;
}

void bwd_sorted_carve(BwdSortedParams& p, void* scratch, int64_t n, int T, int Dmax, bool weighted) {
    const size_t tiles = (size_t)(n / kSortTile) + T + 1;
    char* c = static_cast<char*>(scratch);
    auto take = [&](size_t bytes) {
        void* r = c;
        c += align256(bytes);
        return r;
    };
    for (int s = 0; s < 2; ++s) p.kb[s] = static_cast<uint2*>(take((size_t)n * 8));
    for (int s = 0; s < 2; ++s) p.wts[s] = weighted ? static_cast<float*>(take((size_t)n * 4)) : nullptr;
    p.hist = static_cast<uint32_t*>(take(tiles * 256 * 4));
    p.totals = static_cast<uint32_t*>(take((size_t)T * 256 * 4));
    p.seg = static_cast<uint32_t*>(take((size_t)(T + 1) * 4));
    p.tile_base = static_cast<uint32_t*>(take((size_t)(T + 1) * 4));
    p.ctl = static_cast<int32_t*>(take(256));
    const size_t units = (size_t)((Dmax + 127) / 128) * ((size_t)(n / kSubChunk) + T + 1);
    p.unit_base = static_cast<uint32_t*>(take((size_t)(T + 1) * 4));
    p.partial = static_cast<float*>(take(2 * units * 128 * 4));
    p.rec = static_cast<int32_t*>(take(2 * units * 4));
    p.max_tiles = (uint32_t)tiles;
    p.max_units = (uint32_t)units;
    p.Dmax = Dmax;
}

cudaError_t launch_bwd_sorted(const BwdSortedParams& p, int num_sms, cudaStream_t s, int* launches) {
    int count = 0;
    cudaError_t e = cudaFuncSetAttribute(reinterpret_cast<const void*>(bwds_scatter_kernel<true>),
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kSortTile * 12);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(reinterpret_cast<const void*>(bwds_scatter_kernel<false>),
                             cudaFuncAttributeMaxDynamicSharedMemorySize, kSortTile * 8);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(p.ctl, 0, 256, s);
    if (e != cudaSuccess) return e;
    const int wave = num_sms * 8;
    bwds_check_kernel<<<wave, 256, 0, s>>>(p);
    bwds_plan_kernel<<<1, 256, 0, s>>>(p);
    bwds_expand_kernel<<<wave, 256, 0, s>>>(p);
    count += 3;
    int side = 0;
    for (int pass = 0; pass < p.passes; ++pass) {
        bwds_hist_kernel<<<p.max_tiles, 256, 0, s>>>(p, side, 8 * pass);
        bwds_scan_kernel<<<dim3(256, (unsigned)p.T), 256, 0, s>>>(p);
        if (p.wts[0]) bwds_scatter_kernel<true><<<p.max_tiles, 256, kSortTile * 12, s>>>(p, side, 8 * pass);
        else bwds_scatter_kernel<false><<<p.max_tiles, 256, kSortTile * 8, s>>>(p, side, 8 * pass);
        side ^= 1;
        count += 3;
    }
    const size_t tables_smem = 2 * (size_t)(p.T + 1) * sizeof(uint32_t);
    const int resident = num_sms * EBAG_RUNSUM_BLOCKS;    // one wave: units are dealt round-robin, all tables in step
    if (p.wts[0]) bwds_run_sums_kernel<true><<<resident, 256, tables_smem, s>>>(p, side);
    else bwds_run_sums_kernel<false><<<resident, 256, tables_smem, s>>>(p, side);
    bwds_join_kernel<<<wave, 256, 0, s>>>(p);
    count += 2;
    if (launches) *launches = count;
    return cudaGetLastError();
}

}  // namespace ebag
