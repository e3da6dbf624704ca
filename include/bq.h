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
    BQ_ERR_CUDA = 6,      /* a CUDA runtime call or a launch failed             */
    BQ_ERR_ASSERT = 11    /* a debug build's assertion failed (bq_debug_build); the condition is the last error text */
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

/* 1 if this library was built with its host-side assertions (overlapping buffers, the split of
 * a tensor between kernels; they return BQ_ERR_ASSERT before anything is launched), else 0. */
int bq_debug_build(void);

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

/* ------------------------------------------------------------------------------------------
 * Host-buffer calls.  The paper's receiving node gets the compressed hidden state from the
 * network, i.e. in host memory, and the sending node hands it to the network from host memory
 * (section "Compression techniques", item 1: the hidden states "exchanged between nodes").
 * These calls take HOST pointers and stream the tensor through the GPU in chunks: upload of
 * chunk i+1, the kernel on chunk i and the download of chunk i-1 overlap on three streams of
 * the pipe's own (PCIe is full duplex, the copy engines run beside the SMs).  Every step of
 * the method still runs in the kernels of bq_quantize / bq_dequantize / bq_roundtrip.
 *
 * A pipe owns its device staging buffers, streams and events; all of them are made by
 * bq_host_pipe_create and nothing is allocated per call.  One cudaMemcpyAsync per chunk and
 * direction.  Host buffers should be page-locked (cudaHostAlloc / cudaHostRegister): pageable
 * memory still gives the right bytes, but the copies then block the calling thread and do
 * not overlap.
 */
typedef struct bq_host_pipe bq_host_pipe;

/*
 * bq_host_pipe_create -- on the codebook's device (which must be current).
 *   chunk_elems: elements per piece (> 0); a call uses the largest multiple of its block size that
 *                fits, so block <= chunk_elems is required of every call.
 *   min_block:   the smallest block size calls will use (sizes the absmax staging: chunk_elems /
 *                min_block + 1 floats per slot); calls with a smaller block get BQ_ERR_BLOCK.
 *   widest:      the widest element type calls will use (BQ_F32, or BQ_F16 / BQ_BF16 for 2-byte
 *                staging); calls with a wider type get BQ_ERR_DTYPE.
 *   slots:       pieces in flight, 2..8 (3 keeps upload, kernel and download of different pieces busy).
 * Device memory held: slots * chunk_elems * (2 * element bytes + 1) + the absmax staging.
 * The codebook must outlive the pipe.
 */
int bq_host_pipe_create(const bq_codebook* cb, size_t chunk_elems, int min_block, bq_dtype widest, int slots,
                        bq_host_pipe** out);

/* Waits for the pipe's work, then frees its streams, events and device memory.  NULL is allowed. */
int bq_host_pipe_destroy(bq_host_pipe* pipe);

/*
 * The three data calls, host to host.  Same results, bit for bit, as the device-pointer calls
 * on the whole tensor (pieces are whole numbers of blocks, and blocks are independent).
 *   x_host, y_host: n elements; codes_host: n bytes; absmax_host: ceil(n / block) floats.
 * Each call ENQUEUES its copies and kernels and returns; calls on one pipe take effect in the
 * order they were made, and a later call may read host memory that an earlier one writes (the
 * pipe sees the overlap and holds the later call's uploads back until the earlier call has
 * finished; calls without such an overlap run into each other: the uploads of one under the
 * downloads of the one before).  The host buffers belong to the pipe until bq_host_pipe_wait
 * returns.  Errors as for the device calls, plus
 * BQ_ERR_BLOCK for block < min_block or block > chunk_elems and BQ_ERR_DTYPE for a type wider
 * than `widest`.  y_host may be x_host in bq_roundtrip_host when the types agree.
 */
int bq_quantize_host(bq_host_pipe* pipe, const void* x_host, bq_dtype xdt, size_t n, int block,
                     uint8_t* codes_host, float* absmax_host);
int bq_dequantize_host(bq_host_pipe* pipe, const uint8_t* codes_host, const float* absmax_host, size_t n, int block,
                       void* y_host, bq_dtype ydt);
int bq_roundtrip_host(bq_host_pipe* pipe, const void* x_host, bq_dtype xdt, size_t n, int block,
                      void* y_host, bq_dtype ydt);

/* Blocks the calling thread until everything enqueued on the pipe has finished (results are then in
 * the host buffers); returns BQ_ERR_CUDA if any of that work failed. */
int bq_host_pipe_wait(bq_host_pipe* pipe);

/* Makes `cuda_stream` wait (on the device, without blocking the host) for everything enqueued on
 * the pipe so far. */
int bq_host_pipe_wait_on_stream(bq_host_pipe* pipe, void* cuda_stream);

/* 1 when the codebook mirrors around zero (value[j] == -value[254 - j], zero at 127) and its
 * midpoints are spaced so that the tuned kernels' folded search applies; 0 when every call
 * with this codebook takes the general kernels.  The dynamic-tree codebook gives 1. */
int bq_codebook_is_folded(const bq_codebook* cb);

/*
 * bq_set_staging -- chooses, for the whole process, how bq_quantize and bq_roundtrip bring blocks of
 * 2048 and 4096 elements on chip: 0 (the default) = every thread loads its part of a tile into
 * registers; non-zero = whole blocks are staged through shared memory by bulk asynchronous copies
 * (cp.async.bulk onto an mbarrier ring; this GPU's memory only).  Same results, bit for bit.
 * Returns the previous setting.  Shapes without a staged kernel (other block sizes, fp32 blocks of
 * 4096, unaligned pointers) are unaffected.
 */
int bq_set_staging(int on);

/*
 * bq_kernel_status -- 0, or non-zero when a kernel launched with this codebook gave up on a wait
 * that is bounded for safety (the staged kernels wait for their copies for about two seconds at
 * most): the outputs of that call are then incomplete.  Synchronises the device, reads the word and
 * clears it.  status_out: HOST.
 */
int bq_kernel_status(const bq_codebook* cb, int* status_out);

/* A fixed English description of a status code (never NULL). */
const char* bq_status_string(int status);

/* The message of the last CUDA error seen by this library on the calling thread ("" if none). */
const char* bq_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif
