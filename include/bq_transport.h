/*
 * bq_transport.h -- C ABI of the boundary transport: the compressed hidden state on its way
 * from one sequential shard to the next.
 *
 * Source of the operation: the paper's section "Compression techniques", item 1 (the hidden
 * states are quantized to be SENT between nodes and expanded by the node that receives them),
 * its section "Sequential sharding" and the caption of its Fig. 2 (the chain orchestrator ->
 * block 1 -> ... -> block p, each block handing its hidden state to the next).  The paper's
 * nodes talk over a WAN; here both shards are B200s of one machine and the hand-off crosses
 * NVLink: the sender's quantize kernel stores `codes || absmax` straight into a mailbox that
 * lives in the RECEIVER's memory (a peer mapping), piece by piece, while the receiver expands
 * the piece before it from its own memory.  n + 4 ceil(n / block) bytes cross the link instead
 * of the 2 n bytes of a 16-bit tensor.
 *
 * Roles.  The receiver owns the mailbox (`bqx_rx`): `slots` pieces of `chunk_elems` codes plus
 * their absmax, and per slot two events, "filled" and "drained".  The sender (`bqx_tx`) is opened
 * from the receiver's exported description, in the same process (any two devices with peer
 * access, or one device: loop-back) or in another process (CUDA IPC handles).  Per piece
 *     sender:    wait drained[slot] (if it filled the slot before) -> bq_quantize into the mailbox
 *                -> record filled[slot]
 *     receiver:  wait filled[slot] -> bq_dequantize from the mailbox -> record drained[slot]
 * all stream-ordered: no kernel ever waits on another kernel, and the host never blocks.
 * A stream wait on an event takes the event's most recent record AT THE TIME OF THE CALL, so the
 * host must call bqx_rx_recv_piece for a piece after bqx_tx_send_piece for that piece has returned
 * (and bqx_tx_send_piece for a reused slot after the bqx_rx_recv_piece that drains it has returned).
 * bqx_transfer does this for a sender and a receiver driven by one thread; two processes pass one
 * small host message per piece and direction (see the Python module `transport`).
 *
 * Pointers named x, y_out are DEVICE pointers owned by the caller; status codes are bq_status
 * (include/bq.h); argument errors are found on the host before anything is launched; nothing is
 * allocated per call.
 */
#ifndef BQ_TRANSPORT_H
#define BQ_TRANSPORT_H

#include <stddef.h>
#include <stdint.h>

#include "bq.h"

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bqx_rx bqx_rx;      /* the receiving shard's end: owns the mailbox */
typedef struct bqx_tx bqx_tx;      /* the sending shard's end */

enum {
    BQX_STORE = 0,   /* the quantize kernel's stores go straight into the receiver's mailbox        */
    BQX_COPY = 1     /* quantize into a staging buffer of the sender's, then two async peer copies */
};

enum { BQX_EXPORT_BYTES = 2048 };   /* size of the description bqx_rx_export writes */

/* Bytes of device memory a mailbox of this geometry takes (host arithmetic; 0 for bad arguments). */
size_t bqx_mailbox_bytes(size_t chunk_elems, int min_block, int slots);

/*
 * The piece schedule both ends derive from (n, block, chunk_elems, slots): piece p covers
 * elements [first, first + count) (whole blocks of `block` elements except at the tensor's end),
 * uses slot p mod slots, and there are ceil(n / piece_elems) pieces with piece_elems the largest
 * multiple of block within chunk_elems.  Host arithmetic.  Returns BQ_ERR_SIZE when p is past the
 * last piece (with *pieces still set), BQ_ERR_BLOCK for block < 1 or block > chunk_elems.
 */
int bqx_plan(size_t n, int block, size_t chunk_elems, int slots, size_t p, size_t* pieces, int* slot, size_t* first, size_t* count);

/*
 * bqx_rx_create -- on the current device, which must be the codebook's.  Allocates the mailbox
 * (bqx_mailbox_bytes) and 2 * slots events, once.  chunk_elems > 0; min_block >= 1 is the smallest
 * block size transfers will use (sizes the absmax part of a slot); slots 2..8.
 */
int bqx_rx_create(const bq_codebook* cb, size_t chunk_elems, int min_block, int slots, bqx_rx** out);
int bqx_rx_destroy(bqx_rx* rx);

/* Writes the mailbox's description (geometry, owning process and device, pointers, IPC handles of
 * the memory and of the events) into `out` (HOST, BQX_EXPORT_BYTES bytes), for bqx_tx_open. */
int bqx_rx_export(const bqx_rx* rx, void* out);

/*
 * bqx_tx_open -- on the current device (the sender's; must be the codebook's).  `description` is
 * what bqx_rx_export wrote (HOST).  Same process: the mailbox is used through its own pointer; when
 * the two devices differ, cudaDeviceCanAccessPeer is asked first and peer access is enabled
 * (BQ_ERR_CUDA with a message when the devices cannot reach each other).  Another process: the
 * memory and the events are opened through their IPC handles.  mode: BQX_STORE or BQX_COPY (the
 * latter allocates one slot-sized staging buffer per slot on the sender).
 */
int bqx_tx_open(const bq_codebook* cb, const void* description, int mode, bqx_tx** out);
int bqx_tx_close(bqx_tx* tx);

/*
 * One piece, sender side: on `cuda_stream` (the sender device's): waits for drained[slot] when this
 * sender has filled the slot before (in this tensor or an earlier one), quantizes `count` elements
 * at x_piece (blocks of `block`) into the slot, records filled[slot].  count <= chunk_elems, block >=
 * the mailbox's min_block.
 */
int bqx_tx_send_piece(bqx_tx* tx, const void* x_piece, bq_dtype xdt, size_t count, int block, int slot, void* cuda_stream);

/*
 * One piece, receiver side: on `cuda_stream` (the receiver device's): waits for filled[slot],
 * dequantizes the slot into y_piece (count elements of ydt), records drained[slot].
 */
int bqx_rx_recv_piece(bqx_rx* rx, size_t count, int block, int slot, void* y_piece, bq_dtype ydt, void* cuda_stream);

/*
 * bqx_transfer -- the whole tensor across the boundary, for a sender and a receiver driven by one
 * host thread (two devices of one process, or loop-back on one device): y_out = dequantize(
 * quantize(x)), bit-identical to bq_roundtrip, with the pieces pipelined over the two streams
 * (the receiver expands piece p while the sender compresses piece p + 1).  x on the sender's
 * device, y_out on the receiver's; send_stream / recv_stream belong to those devices and must
 * differ from each other for the overlap (they may be the same stream: the pieces then run in
 * turn).  Enqueues and returns.
 */
int bqx_transfer(bqx_tx* tx, bqx_rx* rx, const void* x, bq_dtype xdt, size_t n, int block, void* y_out, bq_dtype ydt,
                 void* send_stream, void* recv_stream);

/* Bytes that cross the boundary for a tensor of n elements in blocks of `block`: n + 4 ceil(n / block). */
size_t bqx_payload_bytes(size_t n, int block);

#ifdef __cplusplus
}
#endif
#endif
