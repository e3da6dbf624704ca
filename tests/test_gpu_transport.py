"""Boundary transport, loop-back on one device: the sending shard's quantize kernel fills a mailbox,
the receiving shard's dequantize kernel drains it, piece by piece over two streams; what arrives
must be the oracle's dequantize(quantize(x)) bit for bit, for ragged piece counts, reused slots,
both transport modes and tensors that follow each other through one mailbox."""
import numpy as np
import pytest
import torch

import oracle
from paper_2407_19775_b200 import transport, workloads

pytestmark = pytest.mark.gpu
ODT = {torch.float32: oracle.F32, torch.float16: oracle.F16, torch.bfloat16: oracle.BF16}


def _bits(t):
    return workloads.as_numpy_bits(t)


@pytest.mark.parametrize("mode", [transport.STORE, transport.COPY])
@pytest.mark.parametrize("dtype,block,chunk,slots,n", [
    (torch.bfloat16, 256, 256 * 64, 3, 256 * 64 * 7 + 256 * 3 + 11),      # 8 pieces, the last one short with a short block
    (torch.float16, 64, 5000, 2, 64 * 78 * 5),                           # the piece is rounded down to 78 blocks; exactly 5 pieces
    (torch.float32, 4096, 4096 * 2, 4, 4096 * 2 * 3 + 1),                # one element in the last piece
    (torch.bfloat16, 2048, 1 << 22, 3, (1 << 23) + (1 << 22) + 2048 * 5),  # pieces above the small-tensor switch of the kernels
    (torch.bfloat16, 100, 1000, 2, 777),                                 # a block size that takes the general kernels; one piece
])
def test_loop_back_transfer_equals_the_oracle(bq, cb, mode, dtype, block, chunk, slots, n):
    dev = torch.device("cuda:0")
    gcb = bq.Codebook(device=dev)
    g = torch.Generator().manual_seed(n % 1000 + block)
    x = (torch.randn(n, generator=g) * (1.0 + 20.0 * (torch.rand(n, generator=g) < 0.003))).to(dtype)
    rx = transport.Receiver(gcb, chunk, min_block=block, slots=slots)
    tx = transport.Sender(gcb, rx.export(), mode)
    xd = x.to(dev)
    xd_flipped = xd.flip(0).contiguous()
    s_send, s_recv = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ys = [torch.full((n + 16,), 7.0, dtype=dtype, device=dev) for _ in range(3)]
    torch.cuda.synchronize()                                             # inputs and outputs exist before the two streams start
    for rep, y in enumerate(ys):                                         # tensors follow each other through the same slots
        transport.transfer(tx, rx, xd if rep != 1 else xd_flipped, block, y[:n], s_send, s_recv)
    s_recv.synchronize()
    s_send.synchronize()
    ref = oracle.roundtrip(_bits(x), ODT[dtype], block, cb, ODT[dtype])
    ref_flipped = oracle.roundtrip(_bits(x.flip(0).contiguous()), ODT[dtype], block, cb, ODT[dtype])
    for rep, y in enumerate(ys):
        assert np.array_equal(_bits(y[:n].cpu()), ref_flipped if rep == 1 else ref), f"tensor {rep}"
        assert bool((y[n:] == 7.0).all())
    assert len(transport.plan(n, block, chunk, slots)) == (n + (chunk // block) * block - 1) // ((chunk // block) * block)
    tx.close()
    rx.close()


def test_piece_calls_through_the_chain_plumbing(bq, cb):
    """The per-piece calls driven by ChainEndpoint in one process (both roles, messages kept in a list):
    the same call order two processes would make, on one device."""
    dev = torch.device("cuda:0")
    gcb = bq.Codebook(device=dev)
    n, block, chunk, slots = 64 * 1000 + 17, 64, 64 * 90, 2
    x = workloads.make("decode70b", rows=8).view(-1)[:n].contiguous()
    xd = x.to(dev)

    class Mailroom:                                                      # in-process stand-in for the two ranks' messages
        def __init__(self):
            self.box = []

        def post(self, dst, tag, value):
            self.box.append((dst, tag, value))

        def wait(self, src, tag, value):
            assert any(m[1] == tag and m[2] == value for m in self.box), (tag, value)

        def exchange(self, payload, src, dst, size):
            if dst is not None:
                self.desc = payload
            return self.desc if src is not None else None

    room = Mailroom()
    recv_end = transport.ChainEndpoint(1, 2, room, lambda c, b, s: transport.Receiver(gcb, c, b, s), None, chunk, block, slots)
    send_end = transport.ChainEndpoint(0, 2, room, None, lambda d: transport.Sender(gcb, d, transport.STORE), chunk, block, slots)
    y = torch.empty(n, dtype=x.dtype, device=dev)
    s_send, s_recv = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    # one thread plays both ranks piece by piece, in the order the messages allow
    pieces = transport.plan(n, block, chunk, slots)
    for p, (slot, first, count) in enumerate(pieces):
        with torch.cuda.stream(s_send):
            send_end.tx.send_piece(xd[first:first + count], block, slot)
        room.post(1, transport.FILLED, p)
        with torch.cuda.stream(s_recv):
            recv_end.rx.recv_piece(count, block, slot, y[first:first + count])
        room.post(0, transport.DRAINED, p)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(y.cpu()), oracle.roundtrip(_bits(x), oracle.F16, block, cb, oracle.F16))


def test_transport_refuses_what_the_mailbox_was_not_made_for(bq):
    dev = torch.device("cuda:0")
    gcb = bq.Codebook(device=dev)
    rx = transport.Receiver(gcb, 1 << 16, min_block=256, slots=2)
    tx = transport.Sender(gcb, rx.export())
    x = torch.zeros(1 << 17, dtype=torch.bfloat16, device=dev)
    y = torch.empty_like(x)
    with pytest.raises(bq.BqError):
        transport.transfer(tx, rx, x, 64, y)                             # below min_block
    with pytest.raises(bq.BqError):
        transport.transfer(tx, rx, x, 1 << 17, y)                        # a block larger than a piece
    with pytest.raises(bq.BqError):
        tx.send_piece(x, 256, 0)                                  # more elements than a slot holds
    with pytest.raises(bq.BqError):
        tx.send_piece(x[:256], 256, 5)                            # no such slot
    bad = bytearray(rx.export()); bad[0] ^= 0xFF
    with pytest.raises(bq.BqError):
        transport.Sender(gcb, bytes(bad))
    tx.close()
    rx.close()


def _shard_process(rank, world, port, tmp):
    """One process per shard, both on device 0: rank 0 sends through the mailbox that rank 1 owns and exported (CUDA IPC
    handles of the memory and of the events); the FILLED / DRAINED messages travel over a gloo group."""
    import torch.distributed as dist
    import paper_2407_19775_b200 as bq
    dist.init_process_group("gloo", rank=rank, world_size=world, init_method=f"tcp://127.0.0.1:{port}")
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    gcb = bq.Codebook(device=dev)
    n, block, chunk, slots = 256 * 64 * 9 + 256 * 2 + 5, 256, 256 * 64, 3
    end = transport.ChainEndpoint(rank, world, transport.DistMessenger(),
                                  lambda c, b, s: transport.Receiver(gcb, c, b, s), lambda d: transport.Sender(gcb, d, transport.STORE),
                                  chunk, block, slots)
    ok = True
    for i in range(3):                                                   # tensors follow each other through the same slots
        x = workloads.make("prefill7b", rows=40).view(-1)[: n].contiguous().roll(i * 1000)
        if rank == 0:
            end.send(x.to(dev), block)
        else:
            y = torch.empty(n, dtype=torch.bfloat16, device=dev)
            end.recv(y, block)
            torch.cuda.synchronize()
            ok = ok and np.array_equal(_bits(y.cpu()), oracle.roundtrip(_bits(x), oracle.BF16, block, oracle.make_codebook(), oracle.BF16))
    end.close()
    torch.cuda.synchronize()
    with open(f"{tmp}/ok{rank}", "w") as f:
        f.write("ok" if ok else "mismatch")
    dist.barrier()
    dist.destroy_process_group()


def test_two_processes_share_the_mailbox_through_ipc_handles(bq, tmp_path):
    """The form a deployment uses (one process per GPU), with both processes on the one GPU there is: the sender opens the
    receiver's mailbox and events through their IPC handles.  Nothing here waits on the device for the other process: the
    order of the two processes' event calls is kept by host messages, the data dependencies by the events."""
    import socket
    import torch.multiprocessing as mp
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_shard_process, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert open(tmp_path / "ok0").read() == "ok" and open(tmp_path / "ok1").read() == "ok"
