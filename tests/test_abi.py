"""The C-ABI library loads and exports every function include/*.h declares; argument
errors come back as status codes before anything touches a device (CPU only)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared(header="bq.h", prefix="bq_"):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(" + prefix + r"[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(bq):
    from paper_2407_19775_b200 import binding
    L = binding.lib()
    names = _declared()
    assert {"bq_make_codebook", "bq_free_codebook", "bq_quantize", "bq_dequantize", "bq_roundtrip"} <= set(names)
    for name in names:
        assert hasattr(L, name), name
    assert set(binding.SYMBOLS) == set(names)


def test_every_header_is_covered():
    assert sorted(os.listdir(os.path.join(ROOT, "include"))) == ["bq.h", "bq4.h", "bq_transport.h", "bq_tune.h", "mmd.h", "mtpp.h"]


def test_every_declared_bq4_symbol_is_exported(bq):
    from paper_2407_19775_b200 import binding, bq4
    L = binding.lib()
    names = _declared("bq4.h", "bq4_")
    assert {"bq4_make_codebook", "bq4_free_codebook", "bq4_quantize", "bq4_dequantize", "bq4_quantize_s16", "bq4_dequantize_s16"} == set(names)
    for name in names:
        assert hasattr(L, name), name
    assert set(bq4.SYMBOLS) == set(names)


def test_bq4_argument_errors_and_host_codebook(bq):
    import numpy as np
    from paper_2407_19775_b200 import bq4
    from oracle import bq4_oracle
    L = bq4._lib()
    one = ctypes.c_void_p(64)        # never dereferenced: every call below fails a check first
    assert L.bq4_quantize(one, 9, 4, 64, one, one, one, None) == 2
    assert L.bq4_quantize(one, 0, 4, 0, one, one, one, None) == 3
    assert L.bq4_quantize(one, 0, 1 << 41, 64, one, one, one, None) == 4
    assert L.bq4_quantize(one, 0, 4, 64, None, one, one, None) == 5
    assert L.bq4_quantize(None, 0, 0, 64, one, None, None, None) == 0
    assert L.bq4_quantize(None, 0, 4, 64, one, one, one, None) == 1
    assert L.bq4_dequantize(one, one, 4, 64, one, None, 0, None) == 1
    assert L.bq4_dequantize(one, one, 4, 64, one, one, 7, None) == 2
    assert L.bq4_quantize_s16(one, 9, 4, 64, one, one, one, None) == 2
    assert L.bq4_quantize_s16(one, 0, 4, 0, one, one, one, None) == 3
    assert L.bq4_quantize_s16(one, 0, 4, 64, None, one, one, None) == 5
    assert L.bq4_quantize_s16(one, 0, 4, 64, one, one, None, None) == 1
    assert L.bq4_quantize_s16(None, 0, 0, 64, one, None, None, None) == 0
    assert L.bq4_dequantize_s16(one, None, 4, 64, one, one, 0, None) == 1
    assert L.bq4_dequantize_s16(one, one, 4, 64, one, one, 7, None) == 2
    out = ctypes.c_void_p()
    assert L.bq4_make_codebook(5, None, None, ctypes.byref(out)) == 5
    assert L.bq4_make_codebook(0, None, None, None) == 1
    assert L.bq4_free_codebook(None) == 0
    cb = bq4.Codebook4()             # host only: no device is touched
    assert np.array_equal(cb.values.view(np.uint32), bq4_oracle.make_codebook().view(np.uint32))
    bad = cb.values.copy(); bad[3] = bad[4]
    assert L.bq4_make_codebook(1, bad.ctypes.data, None, ctypes.byref(out)) == 5


def test_every_declared_tune_symbol_is_exported_and_host_rule(bq):
    import numpy as np
    from paper_2407_19775_b200 import binding, tune
    L = binding.lib()
    names = _declared("bq_tune.h", "bqt_")
    assert {"bqt_workspace_bytes", "bqt_block_errors", "bqt_pick_block"} == set(names)
    for name in names:
        assert hasattr(L, name), name
    assert set(tune.SYMBOLS) == set(names)
    T = tune._lib()
    assert T.bqt_workspace_bytes(2, 1000) == 2048 + 16384 and T.bqt_workspace_bytes(0, 64) == 256 + 16384 and T.bqt_workspace_bytes(7, 64) == 0
    one = ctypes.c_void_p(256)       # never dereferenced: every call below fails a check first
    blocks = np.array([64, 256], np.int32)
    bad = np.array([64, 0], np.int32)
    assert T.bqt_block_errors(one, 9, 4, one, blocks.ctypes.data, 2, one, 1 << 20, one, None) == 2
    assert T.bqt_block_errors(one, 0, 4, one, None, 2, one, 1 << 20, one, None) == 1
    assert T.bqt_block_errors(one, 0, 4, one, blocks.ctypes.data, 0, one, 1 << 20, one, None) == 3
    assert T.bqt_block_errors(one, 0, 4, one, blocks.ctypes.data, 17, one, 1 << 20, one, None) == 3
    assert T.bqt_block_errors(one, 0, 4, one, bad.ctypes.data, 2, one, 1 << 20, one, None) == 3
    assert T.bqt_block_errors(one, 0, 4, None, blocks.ctypes.data, 2, one, 1 << 20, one, None) == 5
    assert T.bqt_block_errors(None, 0, 4, one, blocks.ctypes.data, 2, one, 1 << 20, one, None) == 1
    assert T.bqt_block_errors(one, 0, 4, one, blocks.ctypes.data, 2, one, 100, one, None) == 4
    assert T.bqt_block_errors(one, 0, 4, one, blocks.ctypes.data, 2, ctypes.c_void_p(264), 1 << 20, one, None) == 4
    # the host rule against the oracle's statement of it, every branch
    from oracle import tune_oracle
    cases = [([64, 256, 1024], [1.0, 2.0, 5.0], 100.0, 0.15), ([64, 256, 1024], [1.0, 2.0, 5.0], 100.0, 0.3), ([64, 256, 1024], [1.0, 2.0, 5.0], 100.0, 0.05),
             ([1024, 64, 256], [5.0, 1.0, 2.0], 100.0, 0.15), ([64, 256], [3.0, 3.0], 100.0, 0.01), ([64, 256], [0.0, 0.0], 0.0, 0.0),
             ([256, 64], [4.0, 4.0], 100.0, 0.2), ([32], [7.0], 1.0, 0.0)]
    for cand, err2, norm2, tol in cases:
        assert tune.pick_block(cand, err2 + [norm2], tol) == tune_oracle.pick_block(cand, err2, norm2, tol), (cand, err2, tol)
    out = ctypes.c_int()
    sums = np.array([1.0, 2.0, 9.0])
    assert T.bqt_pick_block(blocks.ctypes.data, sums.ctypes.data, 2, -1.0, ctypes.byref(out)) == 4
    assert T.bqt_pick_block(blocks.ctypes.data, sums.ctypes.data, 2, float("nan"), ctypes.byref(out)) == 4
    assert T.bqt_pick_block(None, sums.ctypes.data, 2, 0.1, ctypes.byref(out)) == 1


def test_every_declared_mmd_symbol_is_exported(bq):
    from paper_2407_19775_b200 import binding, mmd
    L = binding.lib()
    names = _declared("mmd.h", "mmd_")
    assert {"mmd_rowquant", "mmd_decompose", "mmd_linear", "mmd_free"} <= set(names)
    for name in names:
        assert hasattr(L, name), name
    assert set(mmd.SYMBOLS) == set(names)


def test_mmd_argument_errors_need_no_device(bq):
    import numpy as np
    from paper_2407_19775_b200 import mmd
    L = mmd._lib()
    one = ctypes.c_void_p(256)       # never dereferenced: every call below fails a check first
    assert L.mmd_rowquant(one, 0, 4, 64, None, 0, one, one, None, None) == 2          # fp32 rows are not taken
    assert L.mmd_rowquant(one, 2, 4, 40, None, 0, one, one, None, None) == 4          # K not a multiple of 16
    assert L.mmd_rowquant(one, 2, 4, 64, None, 2000, one, one, None, None) == 8       # too many features
    assert L.mmd_rowquant(one, 2, 0, 64, None, 0, None, None, None, None) == 0        # no rows: nothing to do
    assert L.mmd_rowquant(None, 2, 4, 64, None, 0, one, one, None, None) == 1
    assert L.mmd_rowquant(ctypes.c_void_p(8), 2, 4, 64, None, 0, one, one, None, None) == 4   # misaligned rows
    out = ctypes.c_void_p()
    bad = np.array([5, 3], np.int32)
    assert L.mmd_decompose(one, 2, 8, 64, bad.ctypes.data, 2, None, ctypes.byref(out)) == 8   # not ascending
    far = np.array([3, 64], np.int32)
    assert L.mmd_decompose(one, 2, 8, 64, far.ctypes.data, 2, None, ctypes.byref(out)) == 8   # out of range
    assert L.mmd_decompose(one, 2, 8, 64, None, 1, None, ctypes.byref(out)) == 1
    assert L.mmd_decompose(one, 2, 0, 64, None, 0, None, ctypes.byref(out)) == 4
    assert L.mmd_decompose(one, 2, 8, 64, None, 0, None, None) == 1
    assert L.mmd_linear(None, one, 4, one, 0, one, 1 << 20, 0, None) == 1
    assert L.mmd_free(None) == 0
    assert [L.mmd_side_columns(k) for k in (0, 1, 64, 65)] == [0, 64, 64, 128]
    for code in (7, 8, 9):
        assert L.bq_status_string(code) not in (b"unknown status", b"ok")


def test_status_strings(bq):
    from paper_2407_19775_b200 import binding
    L = binding.lib()
    seen = {L.bq_status_string(i).decode() for i in range(12)}
    assert len(seen) == 12 and L.bq_status_string(0) == b"ok" and "unknown status" not in seen
    assert L.bq_status_string(99) == b"unknown status"


def test_release_and_debug_builds_say_which_they_are(bq):
    """The library the package loads is the release build; the debug build links the same kernels behind API units compiled
    with their assertions and says so.  (Its behaviour on a GPU: tests/test_gpu_debug_build.py.)"""
    from paper_2407_19775_b200 import binding, build
    assert binding.lib().bq_debug_build() == 0 and bq.debug_build() is False
    dbg = ctypes.CDLL(build.build_debug())
    assert dbg.bq_debug_build() == 1
    for name in binding.SYMBOLS:
        assert hasattr(dbg, name), name


def test_argument_errors_need_no_device(bq):
    from paper_2407_19775_b200 import binding
    L = binding.lib()
    one = ctypes.c_void_p(16)        # never dereferenced: every call below fails a check first
    assert L.bq_quantize(one, 9, 4, 64, one, one, one, None) == 2          # dtype
    assert L.bq_quantize(one, 0, 4, 0, one, one, one, None) == 3           # block
    assert L.bq_quantize(one, 0, 1 << 41, 64, one, one, one, None) == 4    # size
    assert L.bq_quantize(one, 0, 4, 64, None, one, one, None) == 5         # codebook handle
    assert L.bq_quantize(None, 0, 0, 64, one, None, None, None) == 0       # n == 0: nothing to do
    assert L.bq_quantize(None, 0, 4, 64, one, one, one, None) == 1         # null x
    assert L.bq_dequantize(one, one, 4, 64, one, None, 0, None) == 1
    assert L.bq_dequantize(one, one, 4, 64, one, one, 5, None) == 2
    assert L.bq_roundtrip(one, 0, 4, 64, one, one, 0, one, None, None) == 1   # one side output without the other
    assert L.bq_roundtrip(one, 0, 4, -1, one, one, 0, None, None, None) == 3
    out = ctypes.c_void_p()
    assert L.bq_make_codebook(7, None, None, ctypes.byref(out)) == 5
    assert L.bq_make_codebook(0, None, None, None) == 1
    assert L.bq_free_codebook(None) == 0


def test_every_declared_transport_symbol_is_exported_and_host_arithmetic(bq):
    from paper_2407_19775_b200 import binding, transport
    L = binding.lib()
    names = _declared("bq_transport.h", "bqx_")
    assert {"bqx_rx_create", "bqx_tx_open", "bqx_tx_send_piece", "bqx_rx_recv_piece", "bqx_transfer", "bqx_plan"} <= set(names)
    for name in names:
        assert hasattr(L, name), name
    assert set(transport.SYMBOLS) == set(names)
    # what crosses the boundary: n + 4 ceil(n / block) bytes, about half of a 16-bit tensor (the paper's "halve")
    assert transport.payload_bytes(1 << 20, 64) == (1 << 20) + 4 * (1 << 14)
    assert transport.payload_bytes(1000, 64) == 1000 + 4 * 16 and transport.payload_bytes(0, 64) == 0
    assert abs(2 * (1 << 30) / transport.payload_bytes(1 << 30, 256) - 2 * 256 / 260) < 1e-12
    assert transport.mailbox_bytes(1 << 20, 64, 3) == 3 * ((1 << 20) + 65792)      # codes + (2^14 + 1 floats rounded up to 256 bytes)
    assert transport.mailbox_bytes(0, 64, 3) == 0 and transport.mailbox_bytes(1 << 20, 64, 1) == 0 and transport.mailbox_bytes(32, 64, 3) == 0
    # the piece schedule: whole blocks per piece, slots in turn, a short last piece
    assert transport.plan(1000, 64, 300, 3) == [(0, 0, 256), (1, 256, 256), (2, 512, 256), (0, 768, 232)]
    assert transport.plan(256, 64, 300, 2) == [(0, 0, 256)]
    assert transport.plan(0, 64, 300, 2) == []
    assert transport.plan(257, 1, 100, 2) == [(0, 0, 100), (1, 100, 100), (0, 200, 57)]
    T = transport._lib()
    assert T.bqx_plan(1000, 0, 300, 3, 0, None, None, None, None) == 3 and T.bqx_plan(1000, 301, 300, 3, 0, None, None, None, None) == 3
    one = ctypes.c_void_p(256)       # never dereferenced: every call below fails a check first
    out = ctypes.c_void_p()
    assert T.bqx_rx_create(None, 1 << 20, 64, 3, ctypes.byref(out)) == 5
    assert T.bqx_rx_create(one, 1 << 20, 64, 3, None) == 1
    assert T.bqx_rx_create(one, 1 << 20, 0, 3, ctypes.byref(out)) == 3
    assert T.bqx_rx_create(one, 1 << 20, 64, 9, ctypes.byref(out)) == 4
    assert T.bqx_rx_create(one, 0, 64, 3, ctypes.byref(out)) == 4
    assert T.bqx_tx_open(one, None, 0, ctypes.byref(out)) == 1
    assert T.bqx_tx_open(None, one, 0, ctypes.byref(out)) == 5
    junk = ctypes.create_string_buffer(2048)
    assert T.bqx_tx_open(one, junk, 0, ctypes.byref(out)) == 4                    # not a mailbox description
    assert T.bqx_tx_open(one, junk, 7, ctypes.byref(out)) == 4                    # unknown mode
    assert T.bqx_rx_destroy(None) == 0 and T.bqx_tx_close(None) == 0
    assert T.bqx_tx_send_piece(None, one, 2, 64, 64, 0, None) == 1
    assert T.bqx_rx_recv_piece(None, 64, 64, 0, one, 2, None) == 1
    assert T.bqx_transfer(None, None, one, 2, 64, 64, one, 2, None, None) == 1


def test_every_declared_mtpp_symbol_is_exported_and_argument_errors(bq):
    import numpy as np
    from paper_2407_19775_b200 import binding, mtpp
    L = binding.lib()
    names = _declared("mtpp.h", "mtpp_")
    assert set(names) == {"mtpp_graph_create", "mtpp_graph_free", "mtpp_decode_orders", "mtpp_slice_orders"} == set(mtpp.SYMBOLS)
    for name in names:
        assert hasattr(L, name), name
    T = mtpp._lib()
    out = ctypes.c_void_p()
    three = np.array([1, 2, 3], np.int64)

    def create(n, edges, w=three, sp=three, so=three, outp=ctypes.byref(out)):
        e = np.asarray(edges, np.int32).reshape(-1, 2)
        return T.mtpp_graph_create(n, e.shape[0], e.ctypes.data if e.size else None, w.ctypes.data, sp.ctypes.data, so.ctypes.data, outp)

    # every check below fails on the host, before any device is touched
    assert create(3, [(0, 1)], outp=None) == 1
    assert create(0, []) == 4 and create(2000, []) == 4
    assert create(3, [(0, 3)]) == 4 and create(3, [(1, 1)]) == 4 and create(3, [(-1, 2)]) == 4
    assert create(3, [(0, 1), (1, 2), (2, 0)]) == 4                                  # a cycle
    assert create(3, [(0, 1)], w=np.array([1, -2, 3], np.int64)) == 4               # negative work
    assert create(3, [(0, 1)], so=np.array([1, 2, 1 << 41], np.int64)) == 4         # too large
    assert T.mtpp_graph_create(3, 1, None, three.ctypes.data, three.ctypes.data, three.ctypes.data, ctypes.byref(out)) == 1
    assert T.mtpp_graph_free(None) == 0
    one = ctypes.c_void_p(256)
    assert T.mtpp_decode_orders(None, one, 4, one, None) == 1
    assert T.mtpp_slice_orders(None, one, 4, 3, 1, 0, one, one, one, one, None) == 1


def test_host_call_argument_errors_need_no_device(bq):
    from paper_2407_19775_b200 import binding
    L = binding.lib()
    one = ctypes.c_void_p(16)        # never dereferenced: every call below fails a check first
    out = ctypes.c_void_p()
    assert L.bq_host_pipe_create(one, 1 << 20, 64, 2, 3, None) == 1             # nowhere to put the handle
    assert L.bq_host_pipe_create(None, 1 << 20, 64, 2, 3, ctypes.byref(out)) == 5     # no codebook
    assert L.bq_host_pipe_create(one, 1 << 20, 64, 9, 3, ctypes.byref(out)) == 2      # element type
    assert L.bq_host_pipe_create(one, 1 << 20, 0, 2, 3, ctypes.byref(out)) == 3       # smallest block
    assert L.bq_host_pipe_create(one, 32, 64, 2, 3, ctypes.byref(out)) == 3           # a block does not fit a piece
    assert L.bq_host_pipe_create(one, 0, 1, 2, 3, ctypes.byref(out)) == 3
    assert L.bq_host_pipe_create(one, 1 << 20, 64, 2, 1, ctypes.byref(out)) == 4      # slots
    assert L.bq_host_pipe_create(one, 1 << 20, 64, 2, 9, ctypes.byref(out)) == 4
    assert L.bq_host_pipe_create(one, 1 << 35, 64, 2, 3, ctypes.byref(out)) == 4      # piece too large
    assert out.value is None
    assert L.bq_host_pipe_destroy(None) == 0
    assert L.bq_host_pipe_wait(None) == 1
    assert L.bq_host_pipe_wait_on_stream(None, None) == 1
    assert L.bq_quantize_host(None, one, 2, 64, 64, one, one) == 1
    assert L.bq_dequantize_host(None, one, one, 64, 64, one, 2) == 1
    assert L.bq_roundtrip_host(None, one, 2, 64, 64, one, 2) == 1


def test_missing_library_is_an_error(monkeypatch):
    from paper_2407_19775_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libbq.so")
    with pytest.raises(binding.BqError):
        binding.lib()
