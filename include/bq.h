/*
 * bq.h -- C ABI of libbq: dynamic blockwise 8-bit quantization of the hidden state that
 * crosses a shard boundary, and its inverse, as CUDA kernels for sm_100a.
 *
 * Source of the operation: the paper's section "Compression techniques", item 1
 * ("Dynamic Quantization"): hidden states exchanged between nodes are compressed by
 * dynamic blockwise quantization (8 bits per element, halving a 16-bit payload) before
 * they are sent and expanded on the receiving node.
 *
 * Conventions for every data call
 *   - Pointers named x, y_out, codes, codes_out, absmax, absmax_out are DEVICE pointers to
 *     contiguous memory owned by the caller: n elements of the stated type, n bytes of
 *     codes, ceil(n / block) floats of absmax.  The library never allocates per call.
 *   - The tensor is taken flattened in row-major order and cut into consecutive blocks of
 *     `block` elements; the last block may be short and uses only its real elements.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t; NULL = legacy default stream) and
 *     the call returns without synchronising.
 *   - The codebook handle belongs to the device that was current when it was made; data calls
 *     must be made with that device current (BQ_ERR_CODEBOOK otherwise).
 *   - Return value: a bq_status.  Argument errors are found on the host before anything is
 *     launched; nothing throws, aborts or exits.  n == 0 returns BQ_OK without a launch.
 *   - Any block >= 1 and any pointer alignment is accepted.  Blocks of 64, 128, 256, 512,
 *     1024, 2048 or 4096 elements on 16-byte aligned pointers take the tuned kernels; all
 *     other cases take a slower general kernel with identical results.
 *   - NaN / Inf inputs are outside the contract: the affected block's results are
 *     unspecified (every code is still a valid byte, no access is out of bounds, other
 *     blocks are unaffected).
 */
#ifndef BQ_H
#define BQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { BQ_F32 = 0, BQ_F16 = 1, BQ_BF16 = 2 } bq_dtype;

typedef enum {
    BQ_OK = 0,
    BQ_ERR_NULL = 1,      /* a required pointer is NULL                         */
    BQ_ERR_DTYPE = 2,     /* element type is not one of bq_dtype                */
    BQ_ERR_BLOCK = 3,     /* block < 1                                          */
    BQ_ERR_SIZE = 4,      /* n does not fit the launch limits (n >= 2^40)       */
    BQ_ERR_CODEBOOK = 5,  /* unknown kind, bad user values, NULL handle or wrong device */
    BQ_ERR_CUDA = 6       /* a CUDA runtime call or a launch failed             */
} bq_status;

enum { BQ_CODEBOOK_DYNAMIC_TREE = 0, BQ_CODEBOOK_USER = 1 };

/* Opaque.  Owns the device copies of the code values and of the search tables derived
 * from them, on the device that was current when it was made. */
typedef struct bq_codebook bq_codebook;

/*
 * bq_make_codebook -- build the 256-entry codebook and its device tables (step "codebook"
 * of the method; the paper says "dynamic" and does not define the map).
 *   kind = BQ_CODEBOOK_DYNAMIC_TREE: the 8-bit dynamic-tree map over [-1, 1]: sign bit,
 *          an exponent field whose length picks one of 7 decades 10^(k-6), a linear
 *          fraction of k bits giving the midpoints of 2^k equal bins of [0.1, 1], plus the
 *          end values 0 and 1.  Ascending; the code byte is the index; 0.0 is code 127.
 *          user_values256 must be NULL.
 *   kind = BQ_CODEBOOK_USER: user_values256 (HOST pointer, 256 floats) must be finite,
 *          strictly ascending, within [-1, 1], contain 0.0, and have no non-zero magnitude
 *          below 2^-24; otherwise BQ_ERR_CODEBOOK.
 *   host_values_out256: HOST pointer, may be NULL; receives the 256 values.
 *   out: receives the handle (HOST pointer to a pointer).  Allocates device memory on the
 *          current device and synchronises that device once.  Free with bq_free_codebook.
 */
int bq_make_codebook(int kind, const float* user_values256, float* host_values_out256, bq_codebook** out);

/* Frees the handle and its device memory.  NULL is allowed. */
int bq_free_codebook(bq_codebook* cb);

/*
 * bq_quantize -- the sending side (absmax, normalise, nearest code, pack).
 * For every block b: absmax_out[b] = max |x_i| in fp32 (0.0 for an all-zero block);
 * xhat_i = x_i / absmax_out[b] as one IEEE fp32 division (divisor 1 when the absmax is 0);
 * codes_out[i] = index of the codebook value nearest to xhat_i, equal distances going to
 * the smaller index.
 *   x: n elements of type xdt (device).  codes_out: n bytes (device).
 *   absmax_out: ceil(n / block) floats (device).
 */
int bq_quantize(const void* x, bq_dtype xdt, size_t n, int block, const bq_codebook* cb,
                uint8_t* codes_out, float* absmax_out, void* cuda_stream);

/*
 * bq_dequantize -- the receiving side (lookup, scale, narrow).
 * y_out[i] = round-to-nearest-even to ydt of the fp32 product value[codes[i]] * absmax[i / block].
 *   codes: n bytes, absmax: ceil(n / block) floats, y_out: n elements of type ydt (all device).
 */
int bq_dequantize(const uint8_t* codes, const float* absmax, size_t n, int block, const bq_codebook* cb,
                  void* y_out, bq_dtype ydt, void* cuda_stream);

/*
 * bq_roundtrip -- bq_quantize followed by bq_dequantize in one kernel, for the loop that
 * simulates a boundary crossing: the codes stay in registers.  y_out is bit-identical to
 * the two separate calls.  codes_out and absmax_out are optional side outputs (both NULL,
 * or both non-NULL).  y_out may be the same pointer as x when xdt == ydt.
 */
int bq_roundtrip(const void* x, bq_dtype xdt, size_t n, int block, const bq_codebook* cb,
                 void* y_out, bq_dtype ydt, uint8_t* codes_out, float* absmax_out, void* cuda_stream);

/* 1 when the codebook mirrors around zero (value[j] == -value[254 - j], zero at 127) and its
 * midpoints are spaced so that the tuned kernels' folded search applies; 0 when every call
 * with this codebook takes the general kernels.  The dynamic-tree codebook gives 1. */
int bq_codebook_is_folded(const bq_codebook* cb);

/* A fixed English description of a status code (never NULL). */
const char* bq_status_string(int status);

/* The message of the last CUDA error seen by this library on the calling thread ("" if none). */
const char* bq_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif
