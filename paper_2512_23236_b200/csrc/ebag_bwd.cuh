// Parameters of the backward kernel (see ebag_bwd.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ebag_fwd.cuh"     // Status

namespace ebag {

struct BwdTableMeta {        // per table; gradient tables are dense fp32 [rows, D]
    int64_t rows;
    int32_t D;
    int32_t D_off;           // first column of this table in grad_out
    int32_t nvec;            // 16-byte vectors per gradient row (D / 4)
    int32_t g_log2;          // log2 of the lanes that cover a row (or one column tile of it)
};

constexpr int kHotSlots = 32;        // hot-row slots per table (a table of width D uses the first K = min(32, 2048 / D))
constexpr int kCacheFloats = 2048;   // floats of shared memory per warp for the sums of hot rows (8 KB)

// the two slots row r may sit in among K slots (K a power of two)
__host__ __device__ inline int hot_slot(uint32_t r, int K) { return (int)((r * 2654435761u) >> 27) & (K - 1); }
__host__ __device__ inline int hot_slot2(uint32_t r, int K) { return (int)((r * 0x85EBCA6Bu) >> 27) & (K - 1); }

struct BwdParams {
    float* const* grad_tables;   // device [T]
    const BwdTableMeta* meta;    // device [T]
    const void* indices;         // int64 ids, or int32 when idx32
    const int64_t* offsets;
    const float* weights;
    const float* grad_out;       // [B, sumD]
    Status* status;
    int64_t n_indices;
    int64_t B;
    int32_t T;
    int32_t sumD;
    int32_t mean;
    int32_t idx32;
    int32_t* hot;                // [T, kHotSlots] frequent rows of every table by a sample, at their hash slot (-1: none)
    int32_t use_cache;           // 0: hot rows are not looked for
    const int32_t* only_if;      // null, or a device word: both kernels return at once while it is 0
};

size_t bwd_smem_bytes(int T);
cudaError_t launch_bwd(const BwdParams& p, bool weighted, int grid, cudaStream_t s);
cudaError_t occupancy_bwd(bool weighted, int T, int* ctas_per_sm);

}  // namespace ebag
