"""The chain plumbing of the boundary transport on CPU ranks (gloo): which rank hands its hidden
state to which, the exchange of the mailbox descriptions against the direction of the data, and
the per-piece FILLED / DRAINED messages that keep a slot from being read before it is written or
overwritten before it is read.

The ranks' CUDA ends are replaced by stand-ins with the same two calls: the "mailbox" is a file
both processes map, `send_piece` writes the oracle's codes and absmax of the piece into its slot and
`recv_piece` expands the slot with the oracle.  The stand-ins act at call time, so a host call made
out of order shows as wrong data: a receiver that ran ahead of its sender reads a slot's old
contents, a sender that ran ahead of its receiver overwrites a slot that was not read yet.
"""
import os
import socket
import sys
import time

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

CHUNK, BLOCK, SLOTS = 64 * 50, 64, 2
NB = CHUNK // BLOCK + 1
SLOT_BYTES = CHUNK + 4 * NB
DESC = 256


def _free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


class FileReceiver:
    def __init__(self, path, rng):
        self.path, self.rng = path, rng
        self.mem = np.memmap(path, dtype=np.uint8, mode="w+", shape=(SLOTS * SLOT_BYTES,))
        self.mem[:] = 0xEE
        self.mem.flush()

    def export(self) -> bytes:
        return self.path.encode().ljust(DESC, b"\0")

    def recv_piece(self, count, block, slot, y_piece):
        import oracle
        time.sleep(float(self.rng.uniform(0, 0.004)))                       # uneven ranks: whoever may run ahead will
        base = slot * SLOT_BYTES
        nb = (count + block - 1) // block
        codes = np.array(self.mem[base:base + count])
        absmax = np.array(self.mem[base + CHUNK:base + CHUNK + 4 * nb]).view(np.float32)
        y_piece[:] = oracle.dequantize(codes, absmax, block, oracle.make_codebook(), oracle.BF16)
        self.mem[base:base + SLOT_BYTES] = 0xEE                              # a slot read twice, or too early, gives junk


class FileSender:
    def __init__(self, description, rng):
        self.rng = rng
        self.mem = np.memmap(description.rstrip(b"\0").decode(), dtype=np.uint8, mode="r+", shape=(SLOTS * SLOT_BYTES,))

    def send_piece(self, x_piece, block, slot):
        import oracle
        time.sleep(float(self.rng.uniform(0, 0.004)))
        codes, absmax = oracle.quantize(np.ascontiguousarray(x_piece), oracle.BF16, block, oracle.make_codebook())
        base = slot * SLOT_BYTES
        self.mem[base:base + codes.size] = codes
        self.mem[base + CHUNK:base + CHUNK + 4 * absmax.size] = absmax.view(np.uint8)


def _tensor(seed, n):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal(n).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)      # bf16 bit patterns


def _rank_main(rank, world, port, tmp):
    import torch.distributed as dist
    import oracle
    from paper_2407_19775_b200 import transport
    dist.init_process_group("gloo", rank=rank, world_size=world, init_method=f"tcp://127.0.0.1:{port}")
    rng = np.random.default_rng(100 + rank)
    end = transport.ChainEndpoint(rank, world, transport.DistMessenger(),
                                  lambda c, b, s: FileReceiver(os.path.join(tmp, f"mailbox{rank}"), rng),
                                  lambda d: FileSender(d, rng), CHUNK, BLOCK, SLOTS, description_bytes=DESC)
    assert (end.prev, end.next) == (rank - 1 if rank else None, rank + 1 if rank + 1 < world else None)
    cb = oracle.make_codebook()
    sizes = [CHUNK * 7 + 64 * 3 + 5, 64, CHUNK * 2, CHUNK * 5 + 1]           # tensors follow each other through the slots
    ok = True
    for i, n in enumerate(sizes):
        # every shard applies "its layers" (here: one more quantize-dequantize crossing) to what it received
        expected = _tensor(i, n)
        for _ in range(rank):
            expected = oracle.roundtrip(expected, oracle.BF16, BLOCK, cb, oracle.BF16)
        if rank == 0:
            mine = expected
        else:
            mine = np.zeros(n, np.uint16)
            end.recv(mine, BLOCK)
            ok = ok and np.array_equal(mine, expected)
        if end.next is not None:
            end.send(mine, BLOCK)
    end.close()
    with open(os.path.join(tmp, f"ok{rank}"), "w") as f:
        f.write("ok" if ok else "mismatch")
    dist.barrier()
    dist.destroy_process_group()


def _run(world, tmp_path):
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for rank in range(world):
        assert open(tmp_path / f"ok{rank}").read() == "ok", rank


def test_two_shards(tmp_path):
    _run(2, tmp_path)


def test_chain_of_three_shards(tmp_path):
    """The middle rank receives and sends: descriptions flow 2 -> 1 -> 0, data 0 -> 1 -> 2."""
    _run(3, tmp_path)


def test_messenger_refuses_a_message_out_of_order():
    from paper_2407_19775_b200 import transport

    class OneMessage(transport.DistMessenger):
        def __init__(self):
            self._pending = []

            class FakeDist:
                @staticmethod
                def recv(t, src, group=None):
                    t[0], t[1] = transport.FILLED, 4

            self.dist, self.group = FakeDist, None

    m = OneMessage()
    m.wait(0, transport.FILLED, 4)
    try:
        m.wait(0, transport.FILLED, 5)
        raise AssertionError("an unexpected piece number must be refused")
    except transport.BqError:
        pass
