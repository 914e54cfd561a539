// Parameters of the kernel that computes the gradient of the per-sample weights (ebag_bwd_weights.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ebag_fwd.cuh"     // TableMeta, Status, Elem

namespace ebag {

struct BwdWeightsParams {
    const void* const* tables;   // device [T]
    const TableMeta* meta;       // device [T]
    const void* indices;         // int64 ids, or int32 when idx32
    const int64_t* offsets;
    const float* grad_out;       // [B, sumD]
    float* grad_w;               // [n_indices]
    Status* status;
    int64_t n_indices;
    int64_t B;
    int32_t T;
    int32_t sumD;
    int32_t mean;
    int32_t idx32;
    float code_zero;             // rowwise 8-bit tables: the stored byte that means code 0
};

size_t bwd_weights_smem_bytes(int dtype, int T);
// one persistent launch (as many CTAs as fit on num_sms multiprocessors) per width class present:
// bit g of `classes` is set when some table has g_log2 == g (2..5); *launches receives their number
cudaError_t launch_bwd_weights(int dtype, const BwdWeightsParams& p, unsigned classes, int num_sms, cudaStream_t s,
                               int* launches);

}  // namespace ebag
