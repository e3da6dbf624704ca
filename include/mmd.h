/*
 * mmd.h -- C ABI of the mixed matrix decomposition in libbq: 16-bit weight matrices stored as
 * 8-bit integers plus a small 16-bit part, and the linear layer computed from that form on
 * the sm_100a tensor cores.
 *
 * Source of the operation: the paper's section "Compression techniques", item 2 ("Mixed
 * matrix decomposition"): weights go from 16-bit to 8-bit values while a small fraction of
 * critical weights is kept at 16-bit precision.  The paper gives no arithmetic; the reading
 * implemented here is the vector-wise int8 decomposition with a 16-bit side matrix over a
 * fixed, ascending set O of critical input features (columns):
 *
 *   rowquant of a [R, K] 16-bit matrix v, row by row:
 *       a_r      = max over k not in O of |v[r,k]|           (fp32, exact)
 *       q[r,k]   = 0 for k in O, else rint(RN32(RN32(127 v[r,k]) / d_r)), d_r = a_r or 1 if a_r == 0
 *       scale[r] = RN32(a_r / 127)
 *       side[r,j] = v[r, O_j] for j < |O|, and 0 for the padding columns j up to mmd_side_columns(|O|)
 *   linear layer Y = X W^T from rowquant(X) (per call) and rowquant(W) (once, mmd_decompose):
 *       acc[m,n]  = sum_k qx[m,k] qw[n,k]                    (int32, exact)
 *       part[m,n] = sum_j sidex[m,j] sidew[n,j]              (fp32 accumulation)
 *       Y[m,n]    = narrow( fma( fp32(acc[m,n]), RN32(scalex[m] scalew[n]), part[m,n] ) )
 *
 * Conventions
 *   - Pointers are DEVICE pointers to contiguous row-major memory owned by the caller unless
 *     a comment says HOST.  Status codes and element types are those of bq.h.
 *   - Element types: BQ_F16 or BQ_BF16 for v, X, W; Y is the same type or BQ_F32.
 *   - K must be a multiple of 16 and at most 262144; |O| at most 1024; rows at most 2^31 - 1.
 *     Inputs must be finite with magnitudes below 2^120 (127 v must not overflow).
 *   - Work is enqueued on `cuda_stream` and the call returns without synchronising; nothing
 *     is allocated per call (mmd_decompose allocates the handle's device memory once).
 *   - A handle belongs to the device that was current when it was made.
 */
#ifndef MMD_H
#define MMD_H

#include <stddef.h>
#include <stdint.h>

#include "bq.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Additional status codes (continuing bq_status). */
enum {
    MMD_ERR_WORKSPACE = 7, /* workspace missing, misaligned (256 bytes) or too small   */
    MMD_ERR_FEATURES = 8,  /* feature list not ascending, out of range or too long      */
    MMD_ERR_PATH = 9,      /* the requested kernel path cannot take this shape          */
    MMD_ERR_STATIC_LIMIT = 10 /* mmd_linear_static: the call needs more scratch than MMD_STATIC_SCRATCH_BYTES */
};

/* Size of the scratch array built into the library for mmd_linear_static. */
#define MMD_STATIC_SCRATCH_BYTES (4u << 20)

/* Kernel choice of mmd_linear. */
enum {
    MMD_PATH_AUTO = 0,     /* tensor-core kernel when the shape allows, else the general one */
    MMD_PATH_GENERAL = 1,  /* integer dot-product kernel, any M and N                       */
    MMD_PATH_TENSOR = 2,   /* a tcgen05 kernel; needs N % 8 == 0 and 16-byte aligned Y: the persistent CTA-pair
                              kernel for large products with at most 16 critical features, else one tile per CTA */
    MMD_PATH_TENSOR_TILE = 3, /* the one-tile-per-CTA tcgen05 kernel, whatever the size                */
    MMD_PATH_TENSOR_SOLO = 4, /* the persistent kernel without CTA pairs (same limits as the pair kernel; MMD_ERR_PATH
                                 when the product is too small or has more than 16 critical features) */
    MMD_PATH_TENSOR_STREAMK = 5 /* the decode-step kernel that deals the K steps of all tiles out over one CTA per SM: at most 64
                                 rows, K a multiple of 128 and at least 2048, N >= 1024, fewer 128-column tiles than SMs
                                 (MMD_ERR_PATH otherwise) and a workspace of mmd_workspace_bytes_streamk bytes
                                 (MMD_ERR_WORKSPACE otherwise).  Only on request: measured slower than the cluster split that
                                 AUTO uses for such calls (the partial sums cross global memory instead of shared memory). */
};

/* Opaque: the decomposed weights of one linear layer (int8 rows, row scales, 16-bit side
 * columns, the feature list) on the device that was current when it was made. */
typedef struct mmd_weights mmd_weights;

/* Width of the side matrices for n_features critical features: the next multiple of 64
 * (0 for 0). */
int mmd_side_columns(int n_features);

/*
 * mmd_select_features -- the critical input features of a layer: those whose calibration
 * magnitude reaches tau.  Host only.
 *   feature_absmax: HOST, K floats (largest |activation| seen per input feature).
 *   idx_out: HOST, room for K ints; receives the ascending indices.  count_out: HOST.
 */
int mmd_select_features(const float* feature_absmax, int K, float tau, int32_t* idx_out, int* count_out);

/*
 * mmd_rowquant -- the row operation defined at the top of this file.
 *   v: [R, K] of type dt.  idx: n_features ascending ints on the DEVICE (may be NULL when 0).
 *   q_out: [R, K] int8.  scale_out: [R] floats.  side_out: [R, mmd_side_columns(n_features)]
 *   of type dt (may be NULL when n_features == 0).  v and q_out need 16-byte alignment.
 */
int mmd_rowquant(const void* v, bq_dtype dt, int R, int K, const int32_t* idx, int n_features,
                 int8_t* q_out, float* scale_out, void* side_out, void* cuda_stream);

/*
 * mmd_decompose -- rowquant of a weight matrix W [N, K] into a new handle (the offline step).
 *   idx_host: HOST, n_features ascending ints in [0, K).  Allocates device memory, enqueues
 *   the row kernel on cuda_stream; the handle may be used by later calls on the same stream
 *   (or after synchronising).  W may be freed once that work has run.  Free with mmd_free.
 */
int mmd_decompose(const void* W, bq_dtype dt, int N, int K, const int32_t* idx_host, int n_features,
                  void* cuda_stream, mmd_weights** out);

/* Frees the handle and its device memory.  NULL is allowed. */
int mmd_free(mmd_weights* w);

/* Device pointers and sizes of a handle's parts, for inspection (any out pointer may be NULL). */
int mmd_weights_view(const mmd_weights* w, const int8_t** q, const float** scale, const void** side,
                     const int32_t** idx, int* N, int* K, int* n_features, int* dtype);

/*
 * mmd_workspace_layout -- the scratch memory mmd_linear needs for M rows of activations:
 * byte offsets of qx [M, K] int8, scalex [M] floats and sidex [M, side columns] inside the
 * workspace, and its total size.  Host only.  offsets3 may be NULL.
 */
int mmd_workspace_layout(const mmd_weights* w, int M, size_t* offsets3, size_t* total_bytes);

/*
 * mmd_workspace_bytes_streamk -- the size of a workspace that also lets mmd_linear take its decode-step kernel for
 * M rows (MMD_PATH_TENSOR_STREAMK): mmd_workspace_layout's total plus, behind it, one counter per 128-column tile and the
 * slots through which CTAs that share a tile hand over their partial sums (a few MB for an 8192 x 8192 layer).  Equal to
 * mmd_workspace_layout's total for shapes that kernel does not take.  Host only.
 */
int mmd_workspace_bytes_streamk(const mmd_weights* w, int M, size_t* total_bytes);

/*
 * mmd_linear -- Y = X W^T through the decomposition: one row kernel over X into the
 * workspace, then the product kernel (two launches of it for one row of tiles that does not
 * fill whole waves of the device: the whole waves, then the tiles left over).  Consecutive
 * calls on one stream are ordered as usual; the kernels of a call and of the next may become
 * resident early (programmatic stream serialization) but wait for the kernels before them
 * before they touch global memory.
 *   X: [M, K] of the handle's element type (16-byte aligned).  Y: [M, N] of type ydt.
 *   workspace: at least mmd_workspace_layout's total, 256-byte aligned; its contents after
 *   the call are the decomposition of X (tests read them back).  Calls that share a
 *   workspace must not overlap on the device (different streams): order them.
 *   path: MMD_PATH_*.  The two kernels give identical integer sums; their fp32 side sums may
 *   differ in the order of the additions.
 */
int mmd_linear(const mmd_weights* w, const void* X, int M, void* Y, bq_dtype ydt,
               void* workspace, size_t workspace_bytes, int path, void* cuda_stream);

/*
 * mmd_linear_static -- mmd_linear without a workspace argument, for callers that cannot get
 * device memory at the moment of the call: a serving process whose own pool already holds all
 * of the GPU's memory, or a loop that cannot afford the device-wide synchronisation an
 * allocation may cause.  (The paper has no counterpart of this call; it is a convenience of
 * this library.)  The scratch is an array of MMD_STATIC_SCRATCH_BYTES (4 MiB) that is part of
 * the library: every GPU that loads the library holds it until the process exits.  The call
 * allocates and frees nothing.
 *   Limit: the sizes must satisfy mmd_workspace_layout(w, M) <= MMD_STATIC_SCRATCH_BYTES --
 *   about M (K + 4 + 2 side columns) bytes, e.g. 64 rows of 8192 features, a decode step;
 *   otherwise MMD_ERR_STATIC_LIMIT is returned before anything is launched and
 *   bq_last_cuda_error() names both sizes.
 *   The first call on a device looks up the array's device address (one runtime call, no
 *   allocation); make that first call before any stream capture is begun.
 *   All calls on a device share the one array and it keeps what the last call wrote; no call
 *   depends on its previous contents.  Two calls that overlap on the device (different
 *   streams, or this call and an mmd_linear given the same memory) race on it: order them.
 *   Arguments, results and the other error codes are those of mmd_linear.
 */
int mmd_linear_static(const mmd_weights* w, const void* X, int M, void* Y, bq_dtype ydt, int path, void* cuda_stream);

/*
 * mmd_kernel_status -- synchronises the device and returns, through status_out (HOST), 0 or
 * the code a tensor-core kernel left when one of its bounded waits ran out (it then stores
 * nothing more and returns; the context stays usable).  Clears the code.
 */
int mmd_kernel_status(const mmd_weights* w, int* status_out);

/*
 * mmd_selftest_bounded_wait -- a diagnostic with no counterpart in the paper: runs, on the
 * handle's device, one CTA that has the roles of a tensor-core product kernel (tensor memory
 * allocated, an "MMA thread", epilogue warps) and lets the MMA thread wait, through the kernels'
 * own bounded wait, for a barrier that nothing ever arms, with a limit of limit_us microseconds
 * (1 .. 100000) instead of the kernels' two seconds.  The wait runs out, the thread records
 * MMD_SELFTEST_CODE in the handle's status word and raises the CTA's give-up flag, the other
 * waiters leave on seeing it, the tensor memory is freed and the kernel returns: the same path a
 * product kernel takes when a copy never lands.  Nothing traps, faults or waits without a limit.
 * threads_left_out (HOST) receives how many threads left through that path (160 of the CTA's 192:
 * warp 1 waits for nothing).  Synchronises the stream.  Afterwards mmd_kernel_status returns
 * MMD_SELFTEST_CODE once, and the handle works as before.
 */
enum { MMD_SELFTEST_CODE = 77 };
int mmd_selftest_bounded_wait(const mmd_weights* w, unsigned limit_us, int* threads_left_out, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif
