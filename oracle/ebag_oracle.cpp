// CPU oracle for the jagged pooled embedding-bag forward ("TBE" = table-batched embedding).
//
// THIS FILE IS TEST INFRASTRUCTURE.  It is the slow, plain definition that the CUDA library is
// checked against.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may call
// it; the product (libebag.so and its Python binding) never does, and the two share no code.
//
// What it computes.  The paper motivates the operator (Sec. 1.1, paragraph "Model Diversity Across
// Ranking Stages": production embedding tables pass 100 GB and need kernels that look rows up and
// pool them under irregular memory access; Sec. 2.1, paragraph "DLRM Architecture": sparse
// features pass through embeddings) and fixes the input types (Sec. 2.2, paragraph "Feature Types and Memory Layout": sparse features are
// jagged lists of int64 ids, weighted sparse features are lists of (int64 id, float32 score)
// pairs) but prints no formula.  The formula is the operator's plain definition:
//
//   for every table t and bag b (bag id g = t*B + b):
//       s = offsets[g], e = offsets[g+1], L = e - s
//       out[b, Doff[t] + d] = pool_{i = s .. e-1} w_i * value(t, indices[i], d)
//   pool = sum, or sum / L (mean; an empty bag stays +0.0f), or max (the largest value among the
//   lookups that were not skipped; +0.0f if there is none; no weights), w_i = weights[i] or 1.  With weights
//   the mean still divides by the lookup count L (not by the sum of the weights).
//   value() widens the stored element to fp32: fp32 as is, fp16/bf16 exactly, rowwise int8 as
//   scale[row] * (float)q + bias[row] (one fp32 multiply, then one fp32 add).
//
// Arithmetic: every bag element is accumulated in fp32, sequentially in ascending i, product and
// sum rounded separately (build with -ffp-contract=off).  Next to it the same element values are
// accumulated in fp64 (out64) together with S = sum |w*x| (fp64), the scale that the parity
// tolerances are relative to.  In mean mode out64 and S are divided by L as well, so that S is on
// the scale of the value that is output.
//
// Indices outside [0, rows[t]) are skipped and counted (once per lookup); a bag whose end offset
// is below its start offset, or that reaches outside [0, n_indices], is treated as empty and
// counted in n_bad_offsets.  Skipped lookups still count in L.
//
// Parallel mode splits BAGS over OpenMP threads; one bag is always summed by one thread in the
// same order, so the result is bit-identical for any thread count.
//
// Parity pins (tests/test_oracle_*.py): hand-worked example, CPU library routine
// (torch.nn.functional.embedding_bag), brute force through a dense one-hot product in fp64,
// closed forms (one-hot table, row-id table, all-ones table), linearity, mean*L = sum, fp64 error
// bound, planted out-of-range indices.  No function here is "parity unpinned".

#include <cstdint>
#include <cstring>
#include <cmath>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

enum { DT_F32 = 0, DT_F16 = 1, DT_BF16 = 2, DT_INT8_ROWWISE = 3, DT_UINT8_ROWWISE = 4 };
enum { MODE_SUM = 0, MODE_MEAN = 1, MODE_MAX = 2 };

inline float bits_to_float(uint32_t u) {
    float f;
    std::memcpy(&f, &u, sizeof f);
    return f;
}

// IEEE binary16 -> binary32, exact (every binary16 value, subnormals included, is a binary32 value).
inline float half_to_float(uint16_t h) {
    const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    const uint32_t expo = (h >> 10) & 0x1Fu;
    const uint32_t mant = h & 0x3FFu;
    if (expo == 0x1Fu) return bits_to_float(sign | 0x7F800000u | (mant << 13));   // inf / nan
    if (expo != 0) return bits_to_float(sign | ((expo + 112u) << 23) | (mant << 13));
    // zero or subnormal: value = mant * 2^-24
    const float v = std::ldexp((float)mant, -24);
    return sign ? -v : v;
}

// bfloat16 is the upper half of a binary32.
inline float bf16_to_float(uint16_t h) { return bits_to_float((uint32_t)h << 16); }

}  // namespace

extern "C" {

int ebag_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

// Returns 0 on success, 1 on an invalid argument.  All pointers are HOST pointers.
//   tables[t]  : dense row-major [rows[t], D[t]] of float (F32), uint16_t bit patterns (F16, BF16)
//                or int8_t codes (INT8_ROWWISE) or uint8_t codes (UINT8_ROWWISE)
//   scales[t], biases[t] : [rows[t]] fp32, the two rowwise types only (else the arrays may be NULL)
//   indices    : [n_indices] int64;  weights : [n_indices] fp32 or NULL
//   offsets    : [T*B + 1] int64
//   out32      : [B, sum(D)] fp32, fully overwritten
//   out64, S   : [B, sum(D)] fp64 or NULL
//   nthreads   : OpenMP threads to use (<= 0: all)
int ebag_oracle_forward(int32_t T, const int64_t* rows, const int32_t* D, int32_t dtype,
                        const void* const* tables, const float* const* scales,
                        const float* const* biases, const int64_t* indices, int64_t n_indices,
                        const int64_t* offsets, const float* weights, int64_t B, int32_t mode,
                        float* out32, double* out64, double* S, int64_t* n_oob,
                        int64_t* n_bad_offsets, int32_t nthreads) {
    if (T <= 0 || B < 0 || !rows || !D || !tables || !offsets || !out32) return 1;
    if (dtype < DT_F32 || dtype > DT_UINT8_ROWWISE) return 1;
    if (mode != MODE_SUM && mode != MODE_MEAN && mode != MODE_MAX) return 1;
    if (mode == MODE_MAX && weights) return 1;
    if ((dtype == DT_INT8_ROWWISE || dtype == DT_UINT8_ROWWISE) && (!scales || !biases)) return 1;
    std::vector<int64_t> Doff(T + 1, 0);
    for (int32_t t = 0; t < T; ++t) {
        if (D[t] <= 0 || rows[t] < 0) return 1;
        Doff[t + 1] = Doff[t] + D[t];
    }
    const int64_t sumD = Doff[T];
    int64_t oob_total = 0, bad_total = 0;
    const int64_t n_bags = (int64_t)T * B;
#ifdef _OPENMP
    const int use_threads = nthreads > 0 ? nthreads : omp_get_max_threads();
#else
    (void)nthreads;
#endif

#pragma omp parallel num_threads(use_threads) reduction(+ : oob_total, bad_total)
    {
        std::vector<float> acc32;
        std::vector<double> acc64, accS;
#pragma omp for schedule(dynamic, 64)
        for (int64_t g = 0; g < n_bags; ++g) {
            const int32_t t = (int32_t)(g / B);
            const int64_t b = g - (int64_t)t * B;
            const int32_t Dt = D[t];
            int64_t s = offsets[g], e = offsets[g + 1];
            if (e < s || s < 0 || e > n_indices) {   // malformed bag: empty, counted
                ++bad_total;
                e = s = 0;
            }
            const int64_t L = e - s;
            acc32.assign(Dt, 0.0f);
            acc64.assign(Dt, 0.0);
            accS.assign(Dt, 0.0);
            int64_t seen = 0;                              // lookups that were not skipped
            for (int64_t i = s; i < e; ++i) {              // ascending, sequential
                const int64_t r = indices[i];
                if (r < 0 || r >= rows[t]) { ++oob_total; continue; }
                const float w = weights ? weights[i] : 1.0f;
                for (int32_t d = 0; d < Dt; ++d) {
                    float x;
                    const int64_t at = r * (int64_t)Dt + d;
                    switch (dtype) {
                        case DT_F32:  x = ((const float*)tables[t])[at]; break;
                        case DT_F16:  x = half_to_float(((const uint16_t*)tables[t])[at]); break;
                        case DT_BF16: x = bf16_to_float(((const uint16_t*)tables[t])[at]); break;
                        default: {
                            const float q = dtype == DT_UINT8_ROWWISE
                                                ? (float)((const uint8_t*)tables[t])[at]
                                                : (float)((const int8_t*)tables[t])[at];
                            const float sq = scales[t][r] * q;      // rounded product
                            x = sq + biases[t][r];                  // rounded sum
                        }
                    }
                    if (mode == MODE_MAX) {
                        // max pooling: the largest value among the bag's (valid) lookups; the
                        // scale the tolerance refers to is the largest magnitude seen
                        if (seen == 0 || x > acc32[d]) acc32[d] = x;
                        if (seen == 0 || (double)x > acc64[d]) acc64[d] = (double)x;
                        accS[d] = std::fmax(accS[d], std::fabs((double)x));
                        continue;
                    }
                    const float p = w * x;                          // rounded product
                    acc32[d] = acc32[d] + p;                        // rounded sum
                    const double pd = (double)w * (double)x;
                    acc64[d] += pd;
                    accS[d] += std::fabs(pd);
                }
                ++seen;
            }
            float* o32 = out32 + b * sumD + Doff[t];
            double* o64 = out64 ? out64 + b * sumD + Doff[t] : nullptr;
            double* oS = S ? S + b * sumD + Doff[t] : nullptr;
            const bool mean = (mode == MODE_MEAN && L > 0);
            for (int32_t d = 0; d < Dt; ++d) {
                o32[d] = mean ? acc32[d] / (float)L : acc32[d];
                if (o64) o64[d] = mean ? acc64[d] / (double)L : acc64[d];
                if (oS) oS[d] = mean ? accS[d] / (double)L : accS[d];
            }
        }
    }
    if (n_oob) *n_oob = oob_total;
    if (n_bad_offsets) *n_bad_offsets = bad_total;
    return 0;
}

}  // extern "C"
