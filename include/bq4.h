/*
 * bq4.h -- C ABI of the 4-bit variant of libbq's dynamic blockwise quantization: the same
 * method as bq.h with a 16-entry codebook and two codes per byte, so that a 16-bit hidden
 * state crosses a shard boundary in a quarter of its bytes (plus one fp32 absmax per block).
 *
 * Source of the operation: the paper's section "Compression techniques", item 1 ("Dynamic
 * Quantization") names dynamic blockwise quantization of the exchanged hidden states; the
 * 8-bit form of bq.h is the one it reports (halved bandwidth).  The bit width is a parameter
 * of the technique the paper leaves open; this header is the 4-bit point of it.
 *
 * Conventions are those of bq.h (device pointers owned by the caller, flattened row-major
 * tensor cut into blocks of `block` elements, last block may be short, work enqueued on
 * `cuda_stream`, status codes of bq.h, nothing allocated per call) with these differences:
 *   - codes: element 2i sits in the low nibble of byte i, element 2i + 1 in the high nibble;
 *     `packed` has ceil(n / 2) bytes; the unused high nibble of an odd n is written as 0.
 *   - Power-of-two blocks of 8 to 65536 elements on 16-byte aligned x / y (4-byte aligned
 *     packed) take vectorised kernels; everything else takes slower general kernels with
 *     identical results.
 */
#ifndef BQ4_H
#define BQ4_H

#include <stddef.h>
#include <stdint.h>

#include "bq.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque: the 16 code values and the 15 search thresholds derived from them (host memory only). */
typedef struct bq4_codebook bq4_codebook;

/*
 * bq4_make_codebook -- kind = BQ_CODEBOOK_DYNAMIC_TREE: the dynamic-tree map with 4 bits: a sign
 * bit; in the other 3 bits the first set bit picks decade k = 0..2 (scale 10^(k-2)) and leaves k
 * bits of linear fraction, m(k, j) = 10^(k-2) (0.1 + 0.9 (2j + 1) / 2^(k+1)); plus 0 and 1.
 * Ascending, the code is the index, 0.0 is code 7, +1.0 is code 15, the lowest value is -0.8875.
 * kind = BQ_CODEBOOK_USER: user_values16 (HOST, 16 floats) finite, strictly ascending, within
 * [-1, 1], no non-zero magnitude below 2^-24; else BQ_ERR_CODEBOOK.
 * host_values_out16 (HOST, may be NULL) receives the values.  No device memory is involved.
 */
int bq4_make_codebook(int kind, const float* user_values16, float* host_values_out16, bq4_codebook** out);

/* Frees the handle.  NULL is allowed. */
int bq4_free_codebook(bq4_codebook* cb);

/*
 * bq4_quantize -- per block b: absmax_out[b] = max |x_i| (fp32); xhat_i = x_i / absmax_out[b] as
 * one IEEE fp32 division (divisor 1 for an all-zero block); code_i = index of the nearest codebook
 * value, equal distances to the smaller index; codes packed two per byte.
 *   x: n elements of type xdt.  packed_out: ceil(n / 2) bytes.  absmax_out: ceil(n / block) floats.
 */
int bq4_quantize(const void* x, bq_dtype xdt, size_t n, int block, const bq4_codebook* cb,
                 uint8_t* packed_out, float* absmax_out, void* cuda_stream);

/*
 * bq4_dequantize -- y_out[i] = round-to-nearest-even to ydt of the fp32 product
 * value[code_i] * absmax[i / block].
 */
int bq4_dequantize(const uint8_t* packed, const float* absmax, size_t n, int block, const bq4_codebook* cb,
                   void* y_out, bq_dtype ydt, void* cuda_stream);

/*
 * bq4_quantize_s16 / bq4_dequantize_s16 -- the same codec with the block scale stored in two
 * bytes instead of four (at block 64 the fp32 absmax is 11 % of the 4-bit payload, the 16-bit
 * scale 6 %).  The paper fixes no format for the scale; this is a variant of its "Dynamic
 * Quantization" item.
 *   scale_b = the block's absmax rounded toward +infinity to a bf16 (1 sign, 8 exponent, 7
 *   fraction bits), so that no |x_i| / scale_b exceeds 1; never above the largest finite bf16
 *   (inputs above it are outside the contract); 0 for an all-zero block.  scale_out[b] holds the
 *   bf16's 16 bits.  xhat_i = x_i / scale_b as one IEEE fp32 division (divisor 1 for a zero
 *   block); codes and packing as in bq4_quantize.  Dequantize: y_i = round-to-nearest-even to
 *   ydt of the fp32 product value[code_i] * scale_b.
 *   scale_out / scale: ceil(n / block) 16-bit words, device memory, 2-byte aligned.
 * Arguments, errors and kernels otherwise as bq4_quantize / bq4_dequantize.
 */
int bq4_quantize_s16(const void* x, bq_dtype xdt, size_t n, int block, const bq4_codebook* cb,
                     uint8_t* packed_out, uint16_t* scale_out, void* cuda_stream);
int bq4_dequantize_s16(const uint8_t* packed, const uint16_t* scale, size_t n, int block, const bq4_codebook* cb,
                       void* y_out, bq_dtype ydt, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif
