// Parameters of the reproducible backward (ebag_bwd_sorted.cu): lookups sorted by row, then
// summed run by run.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ebag_bwd.cuh"

namespace ebag {

constexpr int kSortTile = 2048;          // lookups per sorting tile (one CTA; 1024 and 4096 measured: 8.46 and 9.57 ms against 8.15 ms)
constexpr int kSubChunk = 1024;          // lookups a warp sums in one go (512 and 2048 measured: 8.79 and 8.18 ms against 8.15 ms)
constexpr int kSortedMaxD = 8192;        // widest gradient row (the run sums walk it in column tiles of 128; the cut-run scratch grows with it)

struct BwdSortedParams {
    float* const* grad_tables;   // device [T]
    const BwdTableMeta* meta;    // device [T]
    const void* indices;         // int64 ids, or int32 when idx32
    const int64_t* offsets;
    const float* weights;        // or null
    const float* grad_out;       // [B, sumD]
    Status* status;
    int64_t n_indices;           // < 2^32
    int64_t B;
    int32_t T;
    int32_t sumD;
    int32_t mean;
    int32_t idx32;
    // ---- scratch owned by the handle
    uint2* kb[2];                // [n] (row, bag) of every lookup (row = rows[t] for a skipped id): the two sides of the sort
    float* wts[2];               // [n] weight / bag length of every lookup; null when both are 1
    uint32_t* hist;              // [256 * max_tiles] per table: [digit][tile] counts, then their running sums
    uint32_t* totals;            // [T * 256] lookups of table t with digit d
    uint32_t* seg;               // [T + 1] first lookup of every table
    uint32_t* tile_base;         // [T + 1] first tile of every table
    int32_t* ctl;                // [0] = 1: the offsets are not non-decreasing inside [0, n]; the other kernel runs
    uint32_t* unit_base;         // [T + 1] first unit (column tile x sub-chunk) of every table's run sums
    float* partial;              // [2][max_units][128]: sums of runs cut by a unit's start / end
    int32_t* rec;                // [max_units][2]: row of the run cut by the end (-1: none), flags of the one cut by the start
    int32_t passes;              // 8-bit digits the row ids need
    int32_t Dmax;                // widest table, floats
    uint32_t max_tiles;          // n / kSortTile + T + 1
    uint32_t max_units;          // ceil(Dmax / 128) * (n / kSubChunk + T + 1)
};

// bytes of scratch for n lookups in T tables of at most Dmax columns (weighted: with the weight arrays)
size_t bwd_sorted_scratch_bytes(int64_t n, int T, int Dmax, bool weighted);
// carve `scratch` (256-byte aligned) into the arrays of p (n, T, Dmax as given to the size function)
void bwd_sorted_carve(BwdSortedParams& p, void* scratch, int64_t n, int T, int Dmax, bool weighted);
// enqueue the whole pipeline; *launches receives the number of kernels launched
cudaError_t launch_bwd_sorted(const BwdSortedParams& p, int num_sms, cudaStream_t s, int* launches);

}  // namespace ebag
