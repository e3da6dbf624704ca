"""Boundary transport: the compressed hidden state on its way from one shard to the next.

``Receiver`` / ``Sender`` / ``transfer`` are the calls of ``include/bq_transport.h`` taking torch
tensors (argument marshalling only).  ``ChainEndpoint`` is the host-side plumbing of the
paper's chain of sequential shards (block 1 -> ... -> block p) with one process per shard: which
rank hands its hidden state to which, the exchange of the mailbox descriptions, and the one small
host message per piece and direction that keeps the two processes' event calls in order.  The
plumbing knows nothing of CUDA: it drives any pair of objects with ``send_piece`` / ``recv_piece``
and any messenger with ``post`` / ``wait``, which is how it is tested on CPU ranks.
"""
from __future__ import annotations

import ctypes

import torch

from .binding import _DT, BqError, Codebook, _check, lib

STORE, COPY = 0, 1
EXPORT_BYTES = 2048
SYMBOLS = ("bqx_mailbox_bytes", "bqx_plan", "bqx_rx_create", "bqx_rx_destroy", "bqx_rx_export", "bqx_tx_open", "bqx_tx_close",
           "bqx_tx_send_piece", "bqx_rx_recv_piece", "bqx_transfer", "bqx_payload_bytes")
_ready = False


def _lib():
    global _ready
    L = lib()
    if not _ready:
        vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        L.bqx_mailbox_bytes.argtypes = [sz, i32, i32]
        L.bqx_mailbox_bytes.restype = sz
        L.bqx_payload_bytes.argtypes = [sz, i32]
        L.bqx_payload_bytes.restype = sz
        L.bqx_plan.argtypes = [sz, i32, sz, i32, sz, ctypes.POINTER(sz), ctypes.POINTER(i32), ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.bqx_rx_create.argtypes = [vp, sz, i32, i32, ctypes.POINTER(vp)]
        L.bqx_rx_destroy.argtypes = [vp]
        L.bqx_rx_export.argtypes = [vp, vp]
        L.bqx_tx_open.argtypes = [vp, vp, i32, ctypes.POINTER(vp)]
        L.bqx_tx_close.argtypes = [vp]
        L.bqx_tx_send_piece.argtypes = [vp, vp, i32, sz, i32, i32, vp]
        L.bqx_rx_recv_piece.argtypes = [vp, sz, i32, i32, vp, i32, vp]
        L.bqx_transfer.argtypes = [vp, vp, vp, i32, sz, i32, vp, i32, vp, vp]
        _ready = True
    return L


def plan(n: int, block: int, chunk: int, slots: int):
    """The piece schedule (``bqx_plan``): a list of (slot, first element, count)."""
    L = _lib()
    pieces, slot, first, count = ctypes.c_size_t(), ctypes.c_int(), ctypes.c_size_t(), ctypes.c_size_t()
    out = []
    p = 0
    while True:
        rc = L.bqx_plan(n, block, chunk, slots, p, ctypes.byref(pieces), ctypes.byref(slot), ctypes.byref(first), ctypes.byref(count))
        if rc == 4 and p >= pieces.value:
            return out
        _check(rc, "bqx_plan")
        out.append((slot.value, first.value, count.value))
        p += 1


def payload_bytes(n: int, block: int) -> int:
    return int(_lib().bqx_payload_bytes(n, block))


def mailbox_bytes(chunk: int, min_block: int, slots: int) -> int:
    return int(_lib().bqx_mailbox_bytes(chunk, min_block, slots))


def _stream_ptr(stream, device) -> int:
    return (torch.cuda.current_stream(device) if stream is None else stream).cuda_stream


class Receiver:
    """The receiving shard's end (``bqx_rx_create``): owns the mailbox on the codebook's device."""

    def __init__(self, cb: Codebook, chunk: int, min_block: int = 64, slots: int = 3):
        self.cb, self.chunk, self.min_block, self.slots, self.device = cb, int(chunk), int(min_block), int(slots), cb.device
        self._h = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            _check(_lib().bqx_rx_create(cb.handle, self.chunk, self.min_block, self.slots, ctypes.byref(self._h)), "bqx_rx_create")

    def export(self) -> bytes:
        buf = ctypes.create_string_buffer(EXPORT_BYTES)
        _check(_lib().bqx_rx_export(self._h, buf), "bqx_rx_export")
        return buf.raw

    def recv_piece(self, count: int, block: int, slot: int, y_piece: torch.Tensor, stream=None) -> None:
        with torch.cuda.device(self.device):
            _check(_lib().bqx_rx_recv_piece(self._h, count, block, slot, y_piece.data_ptr(), _DT[y_piece.dtype], _stream_ptr(stream, self.device)),
                   "bqx_rx_recv_piece")

    def close(self) -> None:
        if self._h:
            _lib().bqx_rx_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Sender:
    """The sending shard's end (``bqx_tx_open``), opened from a receiver's exported description."""

    def __init__(self, cb: Codebook, description: bytes, mode: int = STORE):
        if len(description) != EXPORT_BYTES:
            raise BqError("a mailbox description has %d bytes" % EXPORT_BYTES)
        self.cb, self.device, self.mode = cb, cb.device, mode
        self._h = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            _check(_lib().bqx_tx_open(cb.handle, description, mode, ctypes.byref(self._h)), "bqx_tx_open")

    def send_piece(self, x_piece: torch.Tensor, block: int, slot: int, stream=None) -> None:
        with torch.cuda.device(self.device):
            _check(_lib().bqx_tx_send_piece(self._h, x_piece.data_ptr(), _DT[x_piece.dtype], x_piece.numel(), block, slot,
                                            _stream_ptr(stream, self.device)), "bqx_tx_send_piece")

    def close(self) -> None:
        if self._h:
            _lib().bqx_tx_close(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def transfer(tx: Sender, rx: Receiver, x: torch.Tensor, block: int, y_out: torch.Tensor, send_stream=None, recv_stream=None) -> torch.Tensor:
    """``bqx_transfer``: x (on the sender's device) -> y_out (on the receiver's), one host thread."""
    if not (x.is_cuda and y_out.is_cuda and x.is_contiguous() and y_out.is_contiguous()) or x.numel() != y_out.numel():
        raise BqError("x and y_out must be contiguous CUDA tensors of the same length")
    _check(_lib().bqx_transfer(tx._h, rx._h, x.data_ptr(), _DT[x.dtype], x.numel(), block, y_out.data_ptr(), _DT[y_out.dtype],
                               _stream_ptr(send_stream, tx.device), _stream_ptr(recv_stream, rx.device)), "bqx_transfer")
    return y_out


# ------------------------------------------------------------------------------------------ one process per shard

class DistMessenger:
    """Small host messages between neighbouring ranks over a CPU (gloo) process group: post() sends
    one int64, wait() receives one and checks that it is the expected one."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self._pending = []          # (work, tensor) of posts still on their way: a post must not block, because the
                                    # neighbour may itself be in a post to us (it takes our message only later)

    def post(self, dst: int, tag: int, value: int) -> None:
        t = torch.tensor([tag, value], dtype=torch.int64)
        self._pending.append((self.dist.isend(t, dst, group=self.group), t))
        self._pending = [(w, b) for w, b in self._pending if not w.is_completed()]

    def flush(self) -> None:
        for w, _ in self._pending:
            w.wait()
        self._pending = []

    def wait(self, src: int, tag: int, value: int) -> None:
        t = torch.zeros(2, dtype=torch.int64)
        self.dist.recv(t, src, group=self.group)
        if int(t[0]) != tag or int(t[1]) != value:
            raise BqError(f"out-of-order boundary message from rank {src}: got {(int(t[0]), int(t[1]))}, expected {(tag, value)}")

    def exchange(self, payload: bytes | None, src: int | None, dst: int | None, size: int) -> bytes | None:
        """Sends `payload` to dst (if any) and receives `size` bytes from src (if any)."""
        out = None
        if dst is not None:
            self.dist.send(torch.frombuffer(bytearray(payload), dtype=torch.uint8), dst, group=self.group)
        if src is not None:
            t = torch.zeros(size, dtype=torch.uint8)
            self.dist.recv(t, src, group=self.group)
            out = bytes(t.numpy().tobytes())
        return out


FILLED, DRAINED = 1, 2


class ChainEndpoint:
    """Rank r of a chain of p sequential shards: receives its hidden state from rank r - 1 and hands
    its own to rank r + 1.

    ``make_receiver(chunk, min_block, slots)`` builds this rank's mailbox end (an object with
    ``export()`` and ``recv_piece(count, block, slot, y_piece)``); ``make_sender(description)``
    opens the next rank's mailbox (an object with ``send_piece(x_piece, block, slot)``).  The descriptions travel once, at set-up, from each rank to the rank before
    it.  Per piece the sender posts FILLED after its ``send_piece`` call has returned and the
    receiver posts DRAINED after its ``recv_piece`` call has returned; a sender waits for DRAINED of
    the piece that used the slot before, a receiver for FILLED of the piece it is about to take.
    The messages only order the HOST calls (an event wait takes the event's latest record at the
    time of the call); the data dependencies themselves are the events, on the device.
    """

    def __init__(self, rank: int, world: int, messenger, make_receiver, make_sender, chunk: int, min_block: int, slots: int,
                 description_bytes: int = EXPORT_BYTES):
        self.rank, self.world, self.msg = rank, world, messenger
        self.chunk, self.min_block, self.slots = chunk, min_block, slots
        self.prev = rank - 1 if rank > 0 else None
        self.next = rank + 1 if rank + 1 < world else None
        self.rx = make_receiver(chunk, min_block, slots) if self.prev is not None else None
        mine = self.rx.export() if self.rx is not None else None
        # descriptions flow against the data: rank r sends its own to r - 1 and gets r + 1's.  Even ranks
        # send first and odd ranks receive first, so that blocking sends never face each other.
        theirs = None
        if rank % 2 == 0:
            if self.prev is not None:
                messenger.exchange(mine, None, self.prev, description_bytes)
            if self.next is not None:
                theirs = messenger.exchange(None, self.next, None, description_bytes)
        else:
            if self.next is not None:
                theirs = messenger.exchange(None, self.next, None, description_bytes)
            if self.prev is not None:
                messenger.exchange(mine, None, self.prev, description_bytes)
        self.tx = make_sender(theirs) if self.next is not None else None
        self.sent = 0          # pieces sent over this endpoint's life: slot use carries over from tensor to tensor
        self.received = 0

    def _pieces(self, n: int, block: int):
        if block < self.min_block or block > self.chunk:
            raise BqError("block outside the range the mailbox was made for")
        piece = (self.chunk // block) * block
        return [(lo, min(piece, n - lo)) for lo in range(0, n, piece)]

    def send(self, x_flat, block: int) -> None:
        """Hands x (a flat tensor or array on this rank's device) to the next rank."""
        if self.tx is None:
            raise BqError("the last shard of the chain has nobody to send to")
        for lo, cnt in self._pieces(len(x_flat), block):
            p = self.sent
            slot = p % self.slots
            if p >= self.slots:
                self.msg.wait(self.next, DRAINED, p - self.slots)
            self.tx.send_piece(x_flat[lo:lo + cnt], block, slot)
            self.msg.post(self.next, FILLED, p)
            self.sent += 1

    def recv(self, y_flat, block: int) -> None:
        """Receives len(y_flat) elements from the rank before this one into y_flat."""
        if self.rx is None:
            raise BqError("the first shard of the chain has nobody to receive from")
        pieces = self._pieces(len(y_flat), block)
        for i, (lo, cnt) in enumerate(pieces):
            p = self.received
            slot = p % self.slots
            self.msg.wait(self.prev, FILLED, p)
            self.rx.recv_piece(cnt, block, slot, y_flat[lo:lo + cnt])
            # the sender only waits for DRAINED of pieces whose slot it reuses: the last `slots` pieces of a
            # chain's life are never asked for, but tensors follow each other, so every piece is answered
            self.msg.post(self.prev, DRAINED, p)
            self.received += 1

    def drain_acks(self) -> None:
        """Takes the DRAINED messages the next rank posted for this rank's last pieces (at most `slots`), so that
        no message is left in flight when the group shuts down."""
        if self.tx is None:
            return
        for p in range(max(0, self.sent - self.slots), self.sent):
            self.msg.wait(self.next, DRAINED, p)

    def close(self) -> None:
        """End of the chain's life: outstanding acknowledgements are taken and posts completed."""
        self.drain_acks()
        if hasattr(self.msg, "flush"):
            self.msg.flush()
