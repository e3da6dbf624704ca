/*
 * bq_oracle.h -- CPU oracle for dynamic blockwise 8-bit quantization of hidden states.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, single-threaded restatement of the
 * method, written so that a reader can check it against the definition by eye.  It is
 * what the CUDA library is compared with and what the CPU baseline times; it is not a
 * fallback and no product code may call it.  It shares no code with the CUDA library.
 *
 * The method (paper, section "Compression techniques", item 1 "Dynamic Quantization"):
 * the hidden state sent from one shard to the next is compressed by dynamic blockwise
 * quantization to 8 bits per element (which halves the bytes of a 16-bit tensor) and is
 * expanded again on the receiving shard.  The paper names the technique and nothing
 * more; every numeric choice below (codebook, rounding, ties, zero blocks) is a stated
 * reading, listed next to each function.
 *
 * Pins: every function here is pinned by closed forms, exact-rational brute force,
 * invariants and library cross-checks in the CPU test-suite.  Agreement with any outside
 * library's "dynamic" 8-bit map: parity unpinned (no such code is available or used).
 *
 * All pointers are HOST pointers.  Element types: 0 = fp32, 1 = fp16, 2 = bf16
 * (16-bit types are passed as their raw little-endian bit patterns).
 */
#ifndef BQ_ORACLE_H
#define BQ_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { BQ_ORACLE_F32 = 0, BQ_ORACLE_F16 = 1, BQ_ORACLE_BF16 = 2 };

/* Dynamic-tree codebook: 256 ascending fp32 values in [-1, 1]; the code is the index.
 * Returns 0. */
int bq_oracle_make_codebook(float values_out[256]);

/* Per block of `block` consecutive elements (the last block may be short):
 * absmax in fp32, divide, nearest code by linear scan.  Returns 0, or 1 on a bad
 * argument (null pointer, block < 1, unknown dtype). */
int bq_oracle_quantize(const void* x, int xdt, size_t n, int block, const float codebook[256],
                       uint8_t* codes_out, float* absmax_out);

/* y[i] = round_to_dtype( codebook[codes[i]] * absmax[i / block] ). */
int bq_oracle_dequantize(const uint8_t* codes, const float* absmax, size_t n, int block,
                         const float codebook[256], void* y_out, int ydt);

/* dequantize(quantize(x)); codes_out / absmax_out may be NULL. */
int bq_oracle_roundtrip(const void* x, int xdt, size_t n, int block, const float codebook[256],
                        void* y_out, int ydt, uint8_t* codes_out, float* absmax_out);

/* The two element conversions the oracle uses, exported so that tests can pin them. */
float    bq_oracle_widen(uint16_t bits, int dt);      /* fp16 / bf16 bits -> fp32, exact   */
uint16_t bq_oracle_narrow(float v, int dt);           /* fp32 -> fp16 / bf16 bits, RNE     */

/* Nearest code of one already-normalised value (the linear scan alone). */
int bq_oracle_nearest(float xhat, const float codebook[256]);

#ifdef __cplusplus
}
#endif
#endif
