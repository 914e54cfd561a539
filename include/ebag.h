/*
 * ebag.h -- C ABI of libebag.so: jagged, pooled embedding-bag forward over one or many tables
 * ("TBE", table-batched embedding) on one NVIDIA B200 (sm_100a).
 *
 * The operator.  Recommendation models keep categorical features as embedding tables, in
 * production often larger than 100 GB; looking rows up and pooling them touches memory
 * irregularly and is bound by memory capacity and bandwidth, which is why the paper asks for
 * kernels specialised to it (Sec. 1.1, paragraph "Model Diversity Across Ranking Stages";
 * Sec. 2.1, paragraph "DLRM Architecture", has the sparse features go through embeddings).  The ids arrive as jagged lists of int64 and, for weighted
 * features, as (int64 id, float32 score) pairs (Sec. 2.2, paragraph "Feature Types and Memory
 * Layout").  For T tables and B
 * bags per table this library computes, with bag id g = t*B + b,
 *
 *     out[b, Doff[t] + d] = pool_{i = offsets[g] .. offsets[g+1]-1} w_i * value(t, indices[i], d)
 *
 * where pool is a sum or (EBAG_MEAN) the sum divided by the bag length L = offsets[g+1] -
 * offsets[g] (an empty bag gives +0.0f in every mode), w_i = per_sample_weights[i] or 1, and
 * value() widens the stored element to fp32 (fp16 and bf16 exactly; rowwise int8 as
 * scale[row]*q + bias[row]).  Accumulation and output are fp32.  Doff is the running sum of D.
 * Batching every table behind one launch follows the flattened-array-plus-offsets idea the
 * paper uses for its own jagged preprocessing kernels (Sec. 5.4, "Data Preprocessing Kernels on
 * MTIA", MBDT; Sec. 5.5, "Batch Event Truncate").
 *
 * Conventions.  "device" pointers are CUDA global-memory pointers on the handle's device;
 * "host" pointers are ordinary process memory.  Nothing here takes ownership of a caller's
 * buffer.  ebag_stream is a cudaStream_t passed as void* (NULL = the legacy default stream).
 * Unless stated otherwise a call only enqueues work on the stream and returns; the caller keeps
 * every buffer alive until the stream has passed that work.  One forward per handle may be in
 * flight at a time (the handle's work-queue counters and status words are shared).
 * There is no CPU fallback: without a usable CUDA device every call fails with EBAG_ERR_CUDA.
 */
#ifndef EBAG_H_
#define EBAG_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ebag_tbe ebag_tbe; /* opaque, library-owned */
typedef void* ebag_stream;        /* a cudaStream_t */

typedef enum {
    EBAG_OK = 0,
    EBAG_ERR_INVALID_ARG = 1, /* NULL where a pointer is required, T<=0, B<0, bad D, ... */
    EBAG_ERR_UNSUPPORTED = 2, /* sizes beyond the stated limits */
    EBAG_ERR_CUDA = 3,        /* a CUDA runtime call failed (see ebag_last_cuda_error) */
    EBAG_ERR_INDEX_OOB = 4,   /* reported by ebag_last_status: ids outside [0, rows) were skipped */
    EBAG_ERR_BAD_OFFSETS = 5  /* reported by ebag_last_status: malformed bags were treated as empty */
} ebag_status;

typedef enum { EBAG_F32 = 0, EBAG_F16 = 1, EBAG_BF16 = 2, EBAG_INT8_ROWWISE = 3,
               EBAG_UINT8_ROWWISE = 4 } ebag_dtype;

/* weighted sum = EBAG_SUM with per_sample_weights != NULL.  EBAG_MAX: element-wise maximum over
 * the bag's lookups (ids that are skipped take no part; a bag with no valid lookup gives +0.0f);
 * no weights, not for ebag_forward_mapid nor ebag_forward_noalloc (UNSUPPORTED), long bags are
 * not split.  A maximum is exact, so EBAG_MAX results do not depend on the order of the lookups. */
typedef enum { EBAG_SUM = 0, EBAG_MEAN = 1, EBAG_MAX = 2 } ebag_mode;

#define EBAG_MAX_TABLES 2048

/*
 * Bytes from one stored row to the next.  F32/F16/BF16: D * element size.  INT8_ROWWISE and
 * UINT8_ROWWISE (value = scale[row] * code + bias[row], code signed or unsigned 8-bit): the
 * packed row [D codes, one byte each: q + 128 for signed codes, the code itself for unsigned
 * ones][fp32 scale][fp32 bias][8 bytes pad]
 * = D + 16 (one gather fetches codes and dequantisation constants together; build it with
 * ebag_pack_int8_rowwise or ebag_pack_uint8_rowwise).  Returns -1 if D is not allowed for the dtype:
 * D > 0 and D * element size must be a multiple of 16 bytes (D%4==0 for F32, D%8==0 for
 * F16/BF16, D%16==0 for the rowwise types), so that rows can be gathered with 128-bit loads.
 */
int64_t ebag_row_stride(ebag_dtype dtype, int32_t D);

/*
 * Create a handle for T tables of `dtype` with rows[t] rows (0 <= rows[t] < 2^31) of D[t]
 * elements on CUDA device `device`.  rows and D are host arrays [T], copied.  1 <= T <=
 * EBAG_MAX_TABLES.  Allocates a few KB of device memory (per-table metadata, work-queue
 * counters, status words) plus up to 64 MB of scratch for the partial sums of split bags (see
 * "split_bytes" under ebag_set_param), all owned by the handle until ebag_destroy.  Synchronous.
 * Errors: INVALID_ARG, UNSUPPORTED (T or rows too large), CUDA.
 */
ebag_status ebag_create_tbe(int32_t T, const int64_t* rows, const int32_t* D, ebag_dtype dtype,
                            int device, ebag_tbe** out);

/*
 * Pooled forward for all T tables in ONE kernel launch on `stream` (the operator defined at
 * the top of this file), followed on the same stream by a second, short launch that pools the
 * bags too long for one warp in parts (see "split_bytes" under ebag_set_param; the second launch
 * is skipped when the call is too small to hold such a bag or splitting is off).  Both kernels
 * are launched with programmatic stream serialization and begin by waiting for the kernel ahead
 * of them on the stream, so stream order is what the caller sees.
 *   tables   host array [T] of DEVICE pointers; table t is row-major with row pitch
 *            ebag_row_stride(dtype, D[t]) bytes, 16-byte aligned.  The array is read before the
 *            call returns.
 *   D        host [T]; must equal the create-time D (checked).
 *   indices  device int64 [n_indices]: the concatenated id lists, table-major.
 *   n_indices  length of indices (and of per_sample_weights); bags reaching past it are malformed.
 *   offsets  device int64 [T*B + 1], non-decreasing, offsets[0] == 0: bag g = t*B + b owns
 *            indices[offsets[g] .. offsets[g+1]).
 *   per_sample_weights  device fp32 [n_indices] or NULL.  With EBAG_MEAN the weighted sum is
 *            divided by the bag length L (the lookup count), not by the sum of the weights.
 *   B        bags per table, B >= 0, T*B < 2^31.
 *   out      device fp32 [B, sum(D)] row-major, 16-byte aligned; every element is overwritten
 *            exactly once; must not alias an input.
 * No allocation.  The host does not wait for the device, with one exception: the handle keeps
 * four device copies of the `tables` pointer array (re-sent only when the array's contents
 * change); a call that brings a fifth different array while the call that used the oldest copy
 * is still running waits for that call (cudaEventSynchronize).  A call on another stream than
 * the one that sent the copy it reuses is ordered behind that copy on the device
 * (cudaStreamWaitEvent).  Callers that pass the same pointers every time never meet either.
 * Host-detectable problems return an error and launch nothing.  Problems only the device can see never fault: an id outside [0, rows[t]) is
 * skipped (it adds nothing but still counts in the mean's divisor) and a bag with
 * offsets[g+1] < offsets[g], or reaching outside [0, n_indices], is treated as empty; both are
 * counted and reported by ebag_last_status.  B == 0 or n_indices == 0 is fine.
 */
ebag_status ebag_forward(ebag_tbe* h, const void* const* tables, const int32_t* D,
                         const int64_t* indices, int64_t n_indices, const int64_t* offsets,
                         const float* per_sample_weights, int64_t B, ebag_mode mode, float* out,
                         ebag_stream stream);

/*
 * ebag_forward for 32-bit ids: `indices` is device int32 [n_indices] (4-byte aligned); everything
 * else, the offsets included, is as in ebag_forward.  The paper's problem statement allows ids of
 * either width (Sec. 2.2); negative ids are rejected like any id outside the table.
 */
ebag_status ebag_forward_i32(ebag_tbe* h, const void* const* tables, const int32_t* D,
                             const int32_t* indices, int64_t n_indices, const int64_t* offsets,
                             const float* per_sample_weights, int64_t B, ebag_mode mode, float* out,
                             ebag_stream stream);

/*
 * Backward of the pooled forward with respect to the tables (the training half; the operator is
 * linear in the tables, so this is its transpose):
 *     grad_tables[t][indices[i], d] += w_i * grad_out[b, Doff[t] + d]      (EBAG_MEAN: / L)
 * for every lookup i of every bag (t, b).
 *   grad_out     device fp32 [B, sum(D)], 16-byte aligned: gradient of the loss with respect to `out`.
 *   indices      device int64 or int32 ids (index_bits = 64 or 32), as given to the forward.
 *   offsets, per_sample_weights, B, mode   as given to the forward.
 *   grad_tables  host array [T] of DEVICE pointers to dense fp32 [rows[t], D[t]] arrays (whatever
 *                the storage type of the tables), 16-byte aligned, owned and zeroed by the caller:
 *                the call ADDS into them.  Needs D[t] % 4 == 0 (else UNSUPPORTED).
 * By default the lookups of every table are sorted by row (a stable radix sort, in device scratch
 * the handle keeps: about 16 bytes per lookup, 24 with weights or EBAG_MEAN; grown, with a device
 * synchronisation, when a larger call arrives: the only allocation) and every run of equal rows
 * is added up in the order of the lookups and added into its gradient row once.  No
 * floating-point atomics meet on one address, so two runs of the same call give the same bits
 * (3 + 3 * passes + 2 kernel launches on `stream`, passes = the 8-bit digits the largest table's
 * row count needs).  That path needs offsets that do not decrease, which is checked on the
 * device, n_indices < 2^32, D[t] <= 8192 and room for its scratch; otherwise, and with ebag_set_param("bwd_sorted", 0),
 * the call runs the reduction kernel: a short launch that samples the ids of every table for its
 * most frequent rows, whose contributions are then summed in shared memory, and the backward
 * proper, which adds every contribution with a floating-point reduction in memory; their order
 * is not fixed, so two runs then agree up to fp32 rounding, not bit for bit.  (Both kernels are
 * launched either way; the ones that are not needed return at once.)  Ids outside the table and
 * malformed bags are skipped and counted as in the forward
 * (ebag_last_status).  The gradient with respect to per_sample_weights: ebag_backward_weights.
 */
ebag_status ebag_backward(ebag_tbe* h, const float* grad_out, const void* indices, int32_t index_bits,
                          int64_t n_indices, const int64_t* offsets, const float* per_sample_weights,
                          int64_t B, ebag_mode mode, float* const* grad_tables, ebag_stream stream);

/*
 * Backward of the pooled forward with respect to the per-sample weights (the scores of the
 * paper's weighted sparse features, Sec. 2.2 "Feature Types and Memory Layout"; the forward is
 * linear in them):
 *     grad_weights[i] = sum_d grad_out[b, Doff[t] + d] * value(t, indices[i], d)     (EBAG_MEAN: / L)
 * for lookup i of bag (t, b), value() as in the forward (16-bit storage widened, rowwise 8-bit
 * codes dequantised).  It does not depend on the weights themselves.
 *   tables, D     as given to the forward (host array [T] of DEVICE pointers; read before the call returns).
 *   grad_out      device fp32 [B, sum(D)], 16-byte aligned.
 *   indices       device int64 or int32 ids (index_bits = 64 or 32); offsets, B, mode as given to the forward.
 *   grad_weights  device fp32 [n_indices]; entry i is written for every lookup of a well-formed
 *                 bag (0 for an id outside its table, which is counted); entries that no
 *                 well-formed bag covers are left as they are, and an entry that malformed
 *                 offsets put into several bags receives the value of one of them.
 * One to four kernels on `stream` (one per width class of the tables: rows covered by 4, 8, 16
 * or 32 lanes), no allocation; the sums over a row are added in a fixed order, so two runs give
 * the same bits.  A rowwise 8-bit row contributes scale * sum_d g_d * code_d + bias * sum_d g_d
 * (the value() of the forward rounds scale * code + bias per element first; the two differ by a
 * few roundings of the terms).  D[t] must be a multiple of 4.  A bag is walked by one group of lanes,
 * so a single very long bag is slow (it is not split as in the forward).  Counts of skipped ids
 * and malformed bags go to ebag_last_status.
 */
ebag_status ebag_backward_weights(ebag_tbe* h, const void* const* tables, const int32_t* D,
                                  const float* grad_out, const void* indices, int32_t index_bits,
                                  int64_t n_indices, const int64_t* offsets, int64_t B, ebag_mode mode,
                                  float* grad_weights, ebag_stream stream);

/*
 * The same forward for callers whose per-step data lives in HOST memory: indices, offsets,
 * per_sample_weights and out are host pointers (pinned memory makes the copies asynchronous);
 * tables stay device pointers (they are model state, loaded once).  The call copies the inputs
 * to device staging buffers owned by the handle, runs the forward, and copies the result back;
 * when it returns, everything is enqueued and `stream` is ordered after the last copy: the
 * caller synchronises `stream` before reading `out`.  Large calls are cut into a few ranges (up to 16)
 * of bags so that the inputs of one range, the kernel of the previous and the result of the one
 * before travel at the same time (two copy streams owned by the handle; kernels stay on
 * `stream`, one launch per range).  offsets is read on the host during the call; if it is not
 * non-decreasing within [0, n_indices] the call falls back to one piece and the device reports
 * the malformed bags as usual.  The staging buffers are (re)allocated inside this call whenever
 * n_indices or B exceed what they hold, so the first call, and any call with larger inputs,
 * allocates and synchronises.  `out` holds elements of the handle's "out_dtype" (fp32 unless
 * changed with ebag_set_param; 16-bit output halves the bytes that travel back, which is the
 * longest leg of this call).
 */
ebag_status ebag_forward_host(ebag_tbe* h, const void* const* tables, const int32_t* D,
                              const int64_t* indices, int64_t n_indices, const int64_t* offsets,
                              const float* per_sample_weights, int64_t B, ebag_mode mode,
                              float* out, ebag_stream stream);

/* ebag_forward_host for 32-bit ids: `indices` is host int32 [n_indices]; the rest as above. */
ebag_status ebag_forward_host_i32(ebag_tbe* h, const void* const* tables, const int32_t* D,
                                  const int32_t* indices, int64_t n_indices, const int64_t* offsets,
                                  const float* per_sample_weights, int64_t B, ebag_mode mode,
                                  float* out, ebag_stream stream);

/*
 * Wait for `stream`, then report and clear what the device counted since the last call:
 * *n_oob = ids skipped as out of range, *n_bad_offsets = malformed bags (either pointer may be
 * NULL).  Returns EBAG_ERR_BAD_OFFSETS, else EBAG_ERR_INDEX_OOB, else EBAG_OK.  The only call
 * that synchronises besides create/destroy.
 */
ebag_status ebag_last_status(ebag_tbe* h, ebag_stream stream, int64_t* n_oob,
                             int64_t* n_bad_offsets);

/*
 * Load-time helper: build the packed INT8_ROWWISE table (see ebag_row_stride) from separate
 * device arrays q [rows, D] int8, scale [rows] fp32, bias [rows] fp32 into device buffer dst
 * (rows * ebag_row_stride bytes, 16-byte aligned).  Enqueued on `stream`.
 */
ebag_status ebag_pack_int8_rowwise(const int8_t* q, const float* scale, const float* bias,
                                   int64_t rows, int32_t D, void* dst, ebag_stream stream);

/* The same for UINT8_ROWWISE tables: q [rows, D] holds unsigned codes. */
ebag_status ebag_pack_uint8_rowwise(const uint8_t* q, const float* scale, const float* bias,
                                    int64_t rows, int32_t D, void* dst, ebag_stream stream);

/*
 * MapId transform (paper Sec. 5.4.1 "MapId Transform"): `mapping` is a sorted (strictly
 * increasing) list of the m known ids; every value becomes its 1-based position in it, 0 if it
 * is not in it: insertion index by binary search, clamp to m-1, compare.
 *   values, out  device int64 [n] (out may not alias values);  mapping  device int64 [m], m < 2^31
 * m == 0 maps everything to 0.  One kernel on `stream`, no allocation.
 */
ebag_status ebag_mapid(const int64_t* values, int64_t n, const int64_t* mapping, int64_t m,
                       int64_t* out, ebag_stream stream);

/*
 * MapId for every table of a TBE call in ONE launch: values is the jagged raw-id list of
 * ebag_forward_mapid (device int64 [n_values]), offsets the device array [T*B + 1] that cuts it
 * into tables, mappings / mapping_len as for ebag_forward_mapid; out (device int64 [n_values])
 * receives the row ids, ready for ebag_forward.  The table slices are read from offsets on the
 * device, so there is no host synchronisation.  Followed by ebag_forward this was measured
 * faster than the fused call for mappings of 1 k - 100 k ids (the fused search stalls the gather).
 * When the call has at least as many values as the hash tables of its mappings have slots (per
 * table the power of two at or above four times its length, 16 bytes a slot, 2^24 slots in all
 * at most), those tables are first built in a scratch buffer the handle keeps (grown, with a device
 * synchronisation, when a larger call arrives) and every value is then found with one or two
 * loads: three operations on the stream (clear, build, look up; two kernel launches) instead of
 * one binary-search launch.  Both give the same ids for a sorted mapping, with equal keys mapped
 * to the first of their run.  ebag_set_param("mapid_hash", 0) keeps to the binary search.
 * Table t's values are the range [offsets[t*B], offsets[(t+1)*B]) of the list (clipped to
 * [0, n_values]), which is the union of its bags whenever offsets do not decrease.  With
 * malformed offsets a bag may lie outside its table's range: its values are then mapped by the
 * list of whichever table's range covers them, or not written at all.
 */
ebag_status ebag_mapid_tbe(ebag_tbe* h, const int64_t* values, int64_t n_values,
                           const int64_t* offsets, const int64_t* const* mappings,
                           const int64_t* mapping_len, int64_t B, int64_t* out, ebag_stream stream);

/*
 * The pooled forward with the MapId transform fused into the id fetch: `values` holds RAW ids
 * (same jagged layout as `indices` of ebag_forward); table t looks every one up in mappings[t]
 * (host array [T] of device pointers to sorted int64 lists, mapping_len[t] entries each, host
 * array [T]) and pools row 0 for unknown ids, row k for the k-th known id.  Table t therefore
 * has mapping_len[t] + 1 rows (create the handle with those row counts); a mapped id beyond the
 * table's rows is skipped and counted like any out-of-range id.  Everything else as
 * ebag_forward; the mapping arrays are read before the call returns.  By default the transform
 * runs for all tables in one launch into a buffer of n_values ids that the handle keeps (it is
 * grown, with a device synchronisation, when a larger call arrives: the only allocation), and
 * the plain forward follows on the same stream.  With ebag_set_param("mapid_fused", 1) the
 * look-up runs inside the forward kernel instead, directly in front of the gather, so that the
 * mapped ids never travel through memory: less traffic, but measured slower at the mapping sizes
 * tried (the look-ups stall the row pipeline).  Either way the ids are found through hash tables
 * of the mappings when the call is large enough (see ebag_mapid_tbe), else by binary search.  This is the
 * producer of embedding ids the paper's preprocessing section describes.
 * The two ways agree bit for bit when offsets do not decrease.  Offsets that do decrease can
 * leave a bag that is well-formed by itself outside its table's range of the value list; the
 * fused way still maps such a bag with its own table's list (the per-bag definition), the
 * default way pools whatever ebag_mapid_tbe left at those positions (see there), still without a
 * fault since every id is range-checked.  Callers that cannot vouch for their offsets and need
 * the per-bag definition use the fused way.
 */
ebag_status ebag_forward_mapid(ebag_tbe* h, const void* const* tables, const int32_t* D,
                               const int64_t* values, int64_t n_values, const int64_t* offsets,
                               const float* per_sample_weights, const int64_t* const* mappings,
                               const int64_t* mapping_len, int64_t B, ebag_mode mode, float* out,
                               ebag_stream stream);

/*
 * MergeBucketizedDense transform (paper Sec. 5.4.2): continuous features become embedding ids.
 *   values   device fp32 [F, B] feature-major
 *   borders  device fp32: the sorted border lists of the F features back to back
 *   border_offsets  device int64 [F+1]: feature f owns borders[border_offsets[f] .. [f+1])
 *   out_offsets     device int64 [F]: added to the bins of feature f (the paper's `offsets`,
 *                   which make the bins of different features distinct ids)
 *   out      device int64 [F, B]:  out[f,i] = #borders of f strictly below values[f,i] + out_offsets[f]
 * A value equal to a border falls in the bin on its left (the reading of the paper's worked
 * example and pseudocode, i.e. torch.bucketize's default); NaN falls in the last bin.
 * F <= 65535.  One kernel on `stream`, no allocation.  Borders must be sorted (not checked).
 */
ebag_status ebag_mbdt(const float* values, int32_t F, int64_t B, const float* borders,
                      const int64_t* border_offsets, const int64_t* out_offsets, int64_t* out,
                      ebag_stream stream);

/*
 * Batch Event Truncate (paper Sec. 5.5 "Sequence Learning: Batch Event Truncate"): a nested
 * jagged batch of event features keeps only the first N events of every user, in all F features
 * at once, in four launches whatever F is.
 *   outer_lengths  device int64 [U]: events per user (shared by all features)
 *   inner_lengths  device int64 [F, E] row-major: attributes per event, E = sum(outer_lengths) < 2^31
 *                  (more returns EBAG_ERR_UNSUPPORTED)
 *   values         device int64: the attribute values of feature 0, then feature 1, ...;
 *   value_offsets  device int64 [F+1]: feature f owns values[value_offsets[f] .. [f+1])
 *   outer_out      device int64 [U]: min(outer_lengths[u], N)
 *   inner_out      device int64 [F, E] (same pitch as the input): row f holds the inner lengths
 *                  of the kept events, counts_out[0] = sum(outer_out) of them
 *   values_out     device int64, same size and feature offsets as `values`: feature f holds the
 *                  values of the kept events, counts_out[1 + f] of them, from value_offsets[f] on
 *   counts_out     device int64 [1 + F]
 *   workspace      device, ebag_bet_workspace_bytes(F, U) bytes, 8-byte aligned, caller-owned
 * Order is preserved everywhere.  Negative lengths count as 0; ranges that would leave the
 * caller's arrays (E or a feature's value range too small for the lengths) are cut short
 * instead of read.  No allocation, no synchronisation; outputs must not alias inputs.
 */
int64_t ebag_bet_workspace_bytes(int32_t F, int64_t U);
ebag_status ebag_batch_event_truncate(const int64_t* outer_lengths, int64_t U,
                                      const int64_t* inner_lengths, int64_t E,
                                      const int64_t* values, const int64_t* value_offsets,
                                      int32_t F, int64_t N, int64_t* outer_out, int64_t* inner_out,
                                      int64_t* values_out, int64_t* counts_out, void* workspace,
                                      int64_t workspace_bytes, ebag_stream stream);

/*
 * The same forward without a handle and without any allocation (the paper has no counterpart;
 * this exists for deployment).  Some callers cannot allocate device memory when they need a
 * forward: code that runs inside a memory pool whose owner forbids side allocations, a plugin in
 * a host application that has already given all device memory to its own allocator, a serving
 * thread that may not pay for an allocation and the synchronisation it can imply.
 * ebag_create_tbe allocates, so such callers cannot use a handle.  Here the few KB of device
 * scratch the forward kernel needs (work-queue counters, status words, the table-pointer array
 * and per-table metadata) live in a static device array of EBAG_NOALLOC_SCRATCH_BYTES that the
 * loaded library holds on every GPU until the process exits.
 *   T, rows, D, dtype   as for ebag_create_tbe, host arrays, read before the call returns;
 *                       T <= EBAG_NOALLOC_MAX_TABLES (more: EBAG_ERR_UNSUPPORTED, nothing runs)
 *   tables ... out      as for ebag_forward (device pointers; tables is a host array)
 *   status_counts       device unsigned long long [2] or NULL.  If given, the kernel ADDS the
 *                       number of skipped out-of-range ids to [0] and of malformed bags to [1]
 *                       (the caller zeroes and reads it); if NULL those counts are dropped.
 * Runs on the CURRENT device of the calling thread, on `stream`: one small set-up kernel and the
 * forward kernel.  It calls no cudaMalloc/cudaFree and no allocating library routine.  The
 * first call on each device also looks up the device address of the static array; make that
 * first call before any stream capture.  All calls on one device share the array, which keeps
 * the previous call's contents (each call rewrites what it uses and clears the counters that
 * must start at zero): two calls that overlap on the GPU -- different streams, or the handle-free
 * path from two threads -- race on it; run them one after another.
 */
#define EBAG_NOALLOC_MAX_TABLES 64
#define EBAG_NOALLOC_SCRATCH_BYTES 4096
ebag_status ebag_forward_noalloc(int32_t T, const int64_t* rows, const int32_t* D,
                                 ebag_dtype dtype, const void* const* tables,
                                 const int64_t* indices, int64_t n_indices, const int64_t* offsets,
                                 const float* per_sample_weights, int64_t B, ebag_mode mode,
                                 float* out, unsigned long long* status_counts,
                                 ebag_stream stream);

/*
 * Tuning knobs, for experiments; defaults are chosen at create.  Names:
 *   "item_bytes"   target bytes of gathered rows per work item (default 32768)
 *   "ctas_per_sm"  resident CTAs per SM of the persistent grid (default: occupancy limit)
 *   "host_chunks"  bag ranges per ebag_forward_host call, 1..16 (default 0: from the size)
 *   "mapid_fused"  ebag_forward_mapid: 1 = search inside the forward kernel, 0 (default) = the
 *                  transform in a launch of its own, then the plain forward
 *   "mapid_hash"   ebag_mapid_tbe (and with it the default ebag_forward_mapid): 1 (default) =
 *                  look values up through hash tables of the mappings when the call is large
 *                  enough to pay for building them, 0 = always binary search
 *   "out_dtype"    element type of `out` in ebag_forward, ebag_forward_i32 and
 *                  ebag_forward_mapid: EBAG_F32 (default), EBAG_F16 or EBAG_BF16.  Sums are still
 *                  accumulated in fp32 and rounded to nearest-even once, when the bag is written;
 *                  `out` then points at [B, sum(D)] 16-bit elements (same alignment rule).
 *                  ebag_forward_host and ebag_forward_host_i32 return 16-bit elements too.
 *   "bwd_sorted"   ebag_backward: 1 (default) = the reproducible path (lookups sorted by row),
 *                  0 = floating-point reductions in memory (see ebag_backward)
 *   "split_bytes"  a bag whose rows add up to this many bytes or more (rows narrower than 256
 *                  bytes count as 256) is pooled in parts by many warps instead of by one, the
 *                  partial sums added in lookup order by a second, short kernel launched after
 *                  the forward kernel on the same stream (default 65536; 0: never split, one
 *                  launch per forward; otherwise 1024 .. 2^31-1).  The library raises the
 *                  threshold for very large calls so that the bookkeeping always fits, which
 *                  makes the choice of bags to split, and so the result, independent of timing.
 *                  A call whose lookups could not add up to one such bag skips the second launch.
 * Returns INVALID_ARG for an unknown name or a value out of range.
 */
ebag_status ebag_set_param(ebag_tbe* h, const char* name, int64_t value);

/* Number of kernels this handle has launched so far (forward and host-forward; a forward whose
 * call is large enough to hold a bag that would be split counts two, see "split_bytes"). */
int64_t ebag_launch_count(const ebag_tbe* h);

/* Text of the last CUDA error seen by this handle ("" if none). */
const char* ebag_last_cuda_error(const ebag_tbe* h);

/* Frees the handle and its device memory.  Synchronises the device.  NULL is allowed. */
void ebag_destroy(ebag_tbe* h);

const char* ebag_status_string(ebag_status s);

#ifdef __cplusplus
}
#endif
#endif /* EBAG_H_ */
