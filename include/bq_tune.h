/*
 * bq_tune.h -- C ABI of the block-size selection of libbq's dynamic blockwise quantization.
 *
 * Source of the operation: the paper's section "Compression techniques", item 1 ("Dynamic
 * Quantization") compresses the exchanged hidden states blockwise and fixes no block size.  The
 * block size trades payload (4 / block bytes of scale per element) against error (one outlier
 * stretches the scale of its whole block); these calls measure that trade on a tensor and pick.
 * The paper has no counterpart of the selection rule; it is stated in full below.
 *
 * Conventions are those of bq.h: device pointers owned by the caller unless marked HOST, work
 * enqueued on `cuda_stream` without synchronising, integer status codes of bq.h, nothing
 * allocated per call.
 */
#ifndef BQ_TUNE_H
#define BQ_TUNE_H

#include <stddef.h>
#include <stdint.h>

#include "bq.h"

#ifdef __cplusplus
extern "C" {
#endif

#define BQT_MAX_CANDIDATES 16

/* Bytes of device scratch bqt_block_errors needs for a tensor of n elements of type xdt: one
 * reconstructed copy of the tensor plus 16 KiB of partial sums.  0 for an unknown type. */
size_t bqt_workspace_bytes(bq_dtype xdt, size_t n);

/*
 * bqt_block_errors -- for every candidate block size blocks[c] (HOST array, n_blocks entries,
 * 1 <= n_blocks <= BQT_MAX_CANDIDATES, each >= 1): y = bq_roundtrip(x, blocks[c]) with the output
 * type equal to xdt, and
 *     sums_out[c]        = sum_i (x_i - y_i)^2
 *     sums_out[n_blocks] = sum_i x_i^2
 * the difference of the widened elements formed exactly in fp64, its square accumulated in fp64
 * by fused multiply-adds in a fixed order (the same call on the same tensor returns the same
 * bits; the order is not the element order, so the result agrees with an exactly rounded sum to
 * about 1e-13 relative).  sums_out: DEVICE, n_blocks + 1 doubles.  workspace: DEVICE, 256-byte aligned, at
 * least bqt_workspace_bytes(xdt, n) bytes (BQ_ERR_SIZE otherwise).  n = 0 writes zeros.
 * Errors: BQ_ERR_NULL, BQ_ERR_DTYPE, BQ_ERR_BLOCK (a candidate < 1 or n_blocks out of range),
 * BQ_ERR_SIZE, BQ_ERR_CODEBOOK, BQ_ERR_CUDA -- all argument errors before any launch.
 */
int bqt_block_errors(const void* x, bq_dtype xdt, size_t n, const bq_codebook* cb, const int* blocks, int n_blocks,
                     void* workspace, size_t workspace_bytes, double* sums_out, void* cuda_stream);

/*
 * bqt_pick_block -- host arithmetic only (all pointers HOST).  sums = the n_blocks + 1 doubles of
 * bqt_block_errors copied to the host.  A candidate is admissible when its relative rms error is
 * within the bound, decided in fp64 as sums[c] <= max_rel_rms^2 * sums[n_blocks].  *block_out =
 * the largest admissible block (the smallest payload); if none is admissible, the candidate with
 * the smallest sums[c] (the larger block on equal sums).  max_rel_rms must be >= 0 and finite
 * (BQ_ERR_SIZE otherwise).
 */
int bqt_pick_block(const int* blocks, const double* sums, int n_blocks, double max_rel_rms, int* block_out);

#ifdef __cplusplus
}
#endif
#endif
