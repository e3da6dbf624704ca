"""GPU parity of the mixed matrix decomposition against the CPU oracle, through the C ABI.

Bar: the int8 codes, row scales and side columns are bit-exact; the layer's output is
bit-exact when there are no critical features (integer sums are exact and the output is one
fp32 product); with critical features the fp32 side sum is accumulated on the GPU in an
unspecified order, so the output is compared within
    tol = 2^-23 |y| + (side columns + 2) 2^-22 sum_j |x_j w_j|
(one rounding of the result plus one rounding per accumulated product, with a factor 4 for
tensor-core accumulation that may truncate), and 16-bit outputs must lie between the
narrowings of y - tol and y + tol.
"""
import zlib

import numpy as np
import pytest
import torch

from oracle import mmd_oracle as mo
from paper_2407_19775_b200 import workloads

pytestmark = pytest.mark.gpu
F32, F16, BF16 = 0, 1, 2
DT = {torch.float16: F16, torch.bfloat16: BF16}


def bits(t: torch.Tensor) -> np.ndarray:
    return workloads.bits_2d(t.cpu())


def as_f32(a: np.ndarray, dt: int) -> np.ndarray:
    return a if dt == F32 else mo.widen(a, dt)


def y_bits(y: torch.Tensor) -> np.ndarray:
    return y.cpu().numpy() if y.dtype == torch.float32 else bits(y)


def check_output(y_gpu: torch.Tensor, X, W, idx, dt, exact_expected: bool):
    qw, sw, wo = mo.rowquant(bits(W), dt, idx)
    ydt = F32 if y_gpu.dtype == torch.float32 else dt
    y_ref, acc, side, sabs = mo.linear(bits(X), dt, qw, sw, wo, idx, ydt, parts=True)
    got = y_bits(y_gpu)
    if exact_expected:
        assert np.array_equal(got.view(np.uint32 if ydt == F32 else np.uint16), y_ref.view(np.uint32 if ydt == F32 else np.uint16))
        return
    y32 = mo.linear(bits(X), dt, qw, sw, wo, idx, F32).astype(np.float64)
    tol = 2.0 ** -23 * np.abs(y32) + (wo.shape[1] + 2) * 2.0 ** -22 * sabs
    if ydt == F32:
        assert np.all(np.abs(got.astype(np.float64) - y32) <= tol)
    else:
        lo = as_f32(mo.narrow((y32 - tol).astype(np.float32), ydt), ydt)
        hi = as_f32(mo.narrow((y32 + tol).astype(np.float32), ydt), ydt)
        g = as_f32(got, ydt)
        assert np.all((g >= lo) & (g <= hi))
        assert np.mean(got == y_ref) > 0.99                      # and nearly all are the oracle's own bits


@pytest.mark.parametrize("tdt", [torch.bfloat16, torch.float16])
def test_rowquant_bit_exact(bq, tdt):
    dt = DT[tdt]
    g = torch.Generator().manual_seed(21)
    R, K = 75, 1040                                               # ragged: 130 chunks over 256 threads
    v = (torch.randn(R, K, generator=g) * 1.3).to(tdt)
    idx = np.array([0, 7, 8, 500, 1039], np.int32)
    v[:, idx.tolist()] *= 25
    v[3] = 0                                                      # zero row
    v[4, :] = 0; v[4, 7] = 3.0                                    # only a critical feature is non-zero
    v[5, 11] = -v[5].abs().max() * 2                              # the absmax element is negative
    v[6, :16] = torch.tensor([127.0 / 64] + [h / 64 for h in (0.5, 1.5, 2.5, -4.5, -5.5, 100.5, -126.5)] + [0.0] * 8).to(tdt)
    v[6, 16:] = 0; v[6, idx.tolist()] = 9.0                       # exact ties in the regular part
    if tdt == torch.float16:
        v[7] = v[7] * 1e-6                                        # fp16 subnormals
    q_ref, s_ref, side_ref = mo.rowquant(bits(v), dt, idx)
    q, s, side = bq.mmd_rowquant(v.cuda(), torch.from_numpy(idx).cuda())
    torch.cuda.synchronize()
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(bits(side), side_ref)
    q0, s0, side0 = bq.mmd_rowquant(v.cuda(), None)
    q0_ref, s0_ref, _ = mo.rowquant(bits(v), dt, np.zeros(0, np.int32))
    assert np.array_equal(q0.cpu().numpy(), q0_ref) and np.array_equal(s0.cpu().numpy(), s0_ref) and side0.shape == (R, 0)


@pytest.mark.parametrize("K", [16, 2064, 6144, 8192, 12288, 16384, 16400])
def test_rowquant_row_lengths(bq, K):
    """Rows from one chunk to more chunks than the CTA has threads (several trips of its loops), with ragged last trips;
    rows scaled far down and far up (tiny and huge divisors) and a zero row."""
    g = torch.Generator().manual_seed(K)
    R = 9
    v = torch.randn(R, K, generator=g)
    v[1] *= 1e-25; v[2] *= 1e25; v[3] *= 2.0 ** -64; v[4] *= 2.0 ** 63; v[5] = 0
    v = v.to(torch.bfloat16)
    ko = min(5, K - 1)
    idx = np.sort(torch.randperm(K, generator=g)[:ko].numpy()).astype(np.int32)
    v[:, idx.tolist()] *= 8
    q_ref, s_ref, side_ref = mo.rowquant(bits(v), BF16, idx)
    q, s, side = bq.mmd_rowquant(v.cuda(), torch.from_numpy(idx).cuda())
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(bits(side), side_ref)


def test_rowquant_division_cases(bq):
    """Pairs on which a multiplication by the reciprocal would land on another integer."""
    vals = (np.arange(0x3C00, 0x4300, dtype=np.uint32) << 16).view(np.float32)
    rows = []
    for d in vals[::5]:
        scaled = vals * np.float32(127)
        differ = (np.rint(scaled / d) != np.rint(scaled * (np.float32(1) / d))) & (vals <= d)
        rows += [(float(x), float(d)) for x in vals[differ][:3]]
    assert len(rows) > 40
    v = torch.zeros(len(rows), 16)
    for r, (x, d) in enumerate(rows):
        v[r, 0], v[r, 1], v[r, 2] = d, x, -x
    v = v.to(torch.bfloat16)
    q_ref, _, _ = mo.rowquant(bits(v), BF16, np.zeros(0, np.int32))
    q, _, _ = bq.mmd_rowquant(v.cuda(), None)
    assert np.array_equal(q.cpu().numpy(), q_ref)


def test_decompose_matches_oracle(bq):
    X, W, idx = workloads.make_linear("mmd_tiny")
    lin = bq.DecomposedLinear(W.cuda(), idx)
    q, s, side, didx = lin.view()
    torch.cuda.synchronize()
    q_ref, s_ref, side_ref = mo.rowquant(bits(W), BF16, idx)
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(bits(side), side_ref)
    assert np.array_equal(didx.cpu().numpy(), idx)
    lin.close()


@pytest.mark.parametrize("path", [1, 2])                           # general, tensor
@pytest.mark.parametrize("out", ["f32", "same"])
def test_linear_tiny(bq, path, out):
    X, W, idx = workloads.make_linear("mmd_tiny")                 # M = 37, K = 320, N = 72: ragged in every direction
    lin = bq.DecomposedLinear(W.cuda(), idx)
    y = lin.linear(X.cuda(), torch.float32 if out == "f32" else None, path=path)
    assert lin.kernel_status() == 0
    check_output(y, X, W, idx, BF16, exact_expected=False)
    qx, sx, sd = lin.workspace_parts(X.shape[0])
    q_ref, s_ref, side_ref = mo.rowquant(bits(X), BF16, idx)
    assert np.array_equal(qx.cpu().numpy(), q_ref) and np.array_equal(sx.cpu().numpy(), s_ref) and np.array_equal(bits(sd), side_ref)
    # no critical features: bit-exact
    lin0 = bq.DecomposedLinear(W.cuda(), np.zeros(0, np.int32))
    y0 = lin0.linear(X.cuda(), torch.float32 if out == "f32" else None, path=path)
    assert lin0.kernel_status() == 0
    check_output(y0, X, W, np.zeros(0, np.int32), BF16, exact_expected=True)


# shapes chosen so that each tile width of the tensor-core kernel is taken (the width is picked
# from the number of tiles against the SM count), with ragged last tiles in M, N and K
TC_SHAPES = [
    ("bn64", 300, 400, 520, torch.bfloat16, 5),
    ("bn64_fp16", 129, 144, 72, torch.float16, 2),
    ("bn128", 1300, 272, 2056, torch.bfloat16, 70),              # 11 x 17 tiles of 128; two side steps
    ("bn256", 1300, 400, 4104, torch.float16, 3),                # 11 x 17 tiles of 256: persistent kernel, one or two tiles per CTA
    ("bn256_many", 2560, 144, 6152, torch.bfloat16, 16),         # 20 x 25 tiles: three to four per CTA, fewer K steps than ring stages
    ("bn256_side", 1300, 400, 4104, torch.bfloat16, 17),         # too many features for the persistent kernel
    ("one_row", 1, 128, 8, torch.bfloat16, 1),
]


@pytest.mark.parametrize("name,M,K,N,tdt,ko", TC_SHAPES, ids=[s[0] for s in TC_SHAPES])
def test_linear_tensor_path(bq, name, M, K, N, tdt, ko):
    dt = DT[tdt]
    g = torch.Generator().manual_seed(zlib.crc32(name.encode()) % 1000)
    X = (torch.randn(M, K, generator=g) * 0.7).to(tdt)
    W = (torch.randn(N, K, generator=g) * 0.05).to(tdt)
    idx = np.sort(torch.randperm(K, generator=g)[:ko].numpy()).astype(np.int32)
    X[:, idx.tolist()] *= 30
    for features, exact in ((idx, False), (np.zeros(0, np.int32), True)):
        lin = bq.DecomposedLinear(W.cuda(), features)
        persistent = name.startswith("bn256") and len(features) <= 16
        for path in (2, 3, 4) if persistent else (2, 3):          # pair kernel where it applies / one tile per CTA / persistent without pairs
            for out in (torch.float32, None):
                y = lin.linear(X.cuda(), out, path=path)
                assert lin.kernel_status() == 0
                check_output(y, X, W, features, dt, exact_expected=exact)
        yg = lin.linear(X.cuda(), torch.float32, path=1)
        if exact:
            assert torch.equal(yg, lin.linear(X.cuda(), torch.float32, path=2))
            assert torch.equal(yg, lin.linear(X.cuda(), torch.float32, path=3))
            if persistent:
                assert torch.equal(yg, lin.linear(X.cuda(), torch.float32, path=4))
        lin.close()


@pytest.mark.parametrize("M,K,N,ko", [(64, 4096, 7688, 4), (100, 4096, 5120, 0), (7, 1024, 2048, 9), (64, 8192, 1024, 8), (128, 2048, 3000, 3),
                                      (64, 1024, 20488, 5), (100, 512, 30000, 0), (33, 256, 37888, 70),
                                      (64, 2048, 20488, 5), (40, 4096, 19208, 3), (128, 2048, 24000, 0),
                                      (64, 4096, 4736, 2), (48, 3072, 6272, 0)])
def test_linear_one_row_of_tiles_shares_k_steps(bq, M, K, N, ko):
    """Decode-size calls: over narrow layers clusters of 2-4 CTAs split a tile's K steps and add their integer sums
    through shared memory; layers with more 128-row tiles than SMs run their whole waves without the split and, in a
    second launch, the few tiles left over with it (13, 3 and 40 tiles left); 37 and 49 tiles ask for clusters of 4 and
    3 on every SM, more than a device with uneven GPCs runs at once, so the split is lowered.  Both the 64-row and the
    128-row accumulator shapes, ragged N."""
    g = torch.Generator().manual_seed(M * 7 + N)
    X = (torch.randn(M, K, generator=g) * 0.6).to(torch.float16)
    W = (torch.randn(N, K, generator=g) * 0.03).to(torch.float16)
    idx = np.sort(torch.randperm(K, generator=g)[:ko].numpy()).astype(np.int32)
    X[:, idx.tolist()] *= 25
    lin = bq.DecomposedLinear(W.cuda(), idx)
    for out in (torch.float32, None):
        y = lin.linear(X.cuda(), out, path=3)
        assert lin.kernel_status() == 0
        check_output(y, X, W, idx, F16, exact_expected=(ko == 0))
    lin.close()


def test_linear_seeded_fuzz(bq):
    """Random small shapes, feature counts, element types and value scales through every kernel that takes them."""
    rng = np.random.default_rng(2024)
    for case in range(16):
        M = int(rng.integers(1, 300)); K = 16 * int(rng.integers(1, 40)); N = 8 * int(rng.integers(1, 70))
        ko = int(rng.integers(0, min(20, K - 1)))
        tdt = torch.bfloat16 if case % 2 else torch.float16
        dt = DT[tdt]
        g = torch.Generator().manual_seed(1000 + case)
        scale_x = float(10.0 ** rng.uniform(-2, 1)); scale_w = float(10.0 ** rng.uniform(-3, 0))
        X = (torch.randn(M, K, generator=g) * scale_x).to(tdt)
        W = (torch.randn(N, K, generator=g) * scale_w).to(tdt)
        if case % 5 == 0:
            X[int(rng.integers(0, M))] = 0                      # a zero activation row
            W[int(rng.integers(0, N))] = 0
        idx = np.sort(rng.choice(K, ko, replace=False)).astype(np.int32)
        X[:, idx.tolist()] *= 20
        lin = bq.DecomposedLinear(W.cuda(), idx)
        for path in (1, 2, 3):
            y = lin.linear(X.cuda(), torch.float32 if case % 3 else None, path=path)
            assert lin.kernel_status() == 0
            check_output(y, X, W, idx, dt, exact_expected=(ko == 0))
        lin.close()


def test_linear_integer_part_saturating_inputs(bq):
    """Every code at +-127 over a long row: sums far above 2^24 must come back exactly."""
    M, K, N = 130, 4096, 264
    X = torch.full((M, K), 2.0).to(torch.bfloat16)
    W = torch.full((N, K), -0.5).to(torch.bfloat16)
    W[::2] *= -1
    none = np.zeros(0, np.int32)
    lin = bq.DecomposedLinear(W.cuda(), none)
    for path in (1, 2):
        y = lin.linear(X.cuda(), torch.float32, path=path)
        assert lin.kernel_status() == 0
        check_output(y, X, W, none, BF16, exact_expected=True)
        assert torch.allclose(y.cpu(), torch.tensor([4096.0, -4096.0]).repeat(N // 2).expand(M, N), rtol=1e-6)


def test_decode_workload_rows(bq):
    """The decode workload (fp16, K = 8192, 8 critical features) on a slice of the weights."""
    X, W, idx = workloads.make_linear("mmd_decode70b", out_features=1024)
    lin = bq.DecomposedLinear(W.cuda(), idx)
    for path in (1, 2):
        y = lin.linear(X.cuda(), torch.float32, path=path)
        assert lin.kernel_status() == 0
        check_output(y, X, W, idx, F16, exact_expected=False)
    y16 = lin.linear(X.cuda(), None)
    check_output(y16, X, W, idx, F16, exact_expected=False)


def test_full_size_layer_all_tensor_kernels_every_row(bq):
    """The benchmark's layer at full size (4096 x 6144 -> 16384, bf16, 6 critical features) in the launch configurations
    bench.py times: the CTA-pair and the single-CTA persistent kernels add the side features in the same order, so they
    must agree bit for bit; the one-tile-per-CTA kernel accumulates them on the tensor cores (other order).  Every row of
    every output is checked against the oracle (512 rows at a time, so that the oracle's float64 matrices stay small),
    and so is every int8 code, scale and side column of the decomposed weights."""
    X, W, idx = workloads.make_linear("mmd_prefill_moe")
    Xd = X.cuda()
    lin = bq.DecomposedLinear(W.cuda(), idx)
    y_pair = lin.linear(Xd, path=2)
    assert lin.kernel_status() == 0
    y_solo = lin.linear(Xd, path=4)
    assert lin.kernel_status() == 0
    assert torch.equal(y_pair, y_solo)
    y_tile = lin.linear(Xd, path=3)
    assert lin.kernel_status() == 0
    y_gen = lin.linear(Xd, path=1)
    qw, sw, wo = mo.rowquant(bits(W), BF16, idx)
    q_dev, s_dev, side_dev, _ = lin.view()
    assert np.array_equal(q_dev.cpu().numpy(), qw) and np.array_equal(s_dev.cpu().numpy().view(np.uint32), sw.view(np.uint32))
    assert np.array_equal(bits(side_dev), wo)
    same = {"pair": 0, "tile": 0, "general": 0}
    for r0 in range(0, X.shape[0], 512):
        Xr = bits(X[r0:r0 + 512])
        y_ref, _, _, sabs = mo.linear(Xr, BF16, qw, sw, wo, idx, BF16, parts=True)
        y32 = mo.linear(Xr, BF16, qw, sw, wo, idx, F32).astype(np.float64)
        tol = 2.0 ** -23 * np.abs(y32) + (wo.shape[1] + 2) * 2.0 ** -22 * sabs
        lo = mo.widen(mo.narrow((y32 - tol).astype(np.float32), BF16), BF16)
        hi = mo.widen(mo.narrow((y32 + tol).astype(np.float32), BF16), BF16)
        for name, y in (("pair", y_pair), ("tile", y_tile), ("general", y_gen)):
            got = bits(y[r0:r0 + 512])
            g = mo.widen(got, BF16)
            assert np.all((g >= lo) & (g <= hi)), f"{name} kernel, rows {r0}..{r0 + 511}"
            same[name] += int(np.sum(got == y_ref))
    for name, cnt in same.items():
        assert cnt > 0.999 * X.shape[0] * W.shape[0], name       # and nearly all are the oracle's own bits
    lin.close()


@pytest.mark.parametrize("M,K,N", [(64, 2048, 4096), (64, 2048, 20488), (128, 1024, 1536)])
def test_back_to_back_calls_share_a_workspace(bq, M, K, N):
    """A chain of calls with different activations through one workspace and no synchronisation in between: the row kernel
    and the product kernel of consecutive calls are launched so that each may become resident before the one before it has
    ended, and each must still wait before it touches the shared buffers.  Without critical features the tensor-core path
    and the general kernel agree bit for bit, so every output of the chain is compared with a call of its own."""
    g = torch.Generator().manual_seed(M + N)
    W = (torch.randn(N, K, generator=g) * 0.03).to(torch.float16)
    lin = bq.DecomposedLinear(W.cuda(), np.zeros(0, np.int32))
    ws = lin.workspace(M)
    xs = [(torch.randn(M, K, generator=g) * (0.2 + 0.3 * i)).to(torch.float16).cuda() for i in range(8)]
    ys = [torch.empty(M, N, dtype=torch.float32, device="cuda") for _ in xs]
    for _ in range(3):
        for x, y in zip(xs, ys):
            lin.linear(x, y_out=y, workspace=ws)
    torch.cuda.synchronize()
    assert lin.kernel_status() == 0
    for x, y in zip(xs, ys):
        assert torch.equal(y, lin.linear(x, torch.float32, path=1))
    check_output(ys[3], xs[3].cpu(), W, np.zeros(0, np.int32), F16, exact_expected=True)
    lin.close()


def test_a_bounded_wait_that_runs_out_leaves_a_status_and_a_usable_handle(bq):
    """The give-up path of the tensor-core kernels, exercised the safe way: a diagnostic CTA with the kernels' roles waits
    (2 ms limit instead of 2 s) for a barrier that nothing arms.  It must return, leave its code in the status word, free
    its tensor memory (the product kernels after it need all of it) and leave the handle and the context working."""
    X, W, idx = workloads.make_linear("mmd_decode70b", tokens=48, out_features=512)
    lin = bq.DecomposedLinear(W.cuda(), idx)
    before = lin.linear(X.cuda(), torch.float32, path=3)
    assert lin.kernel_status() == 0
    for limit_us in (2000, 50):
        assert lin.selftest_bounded_wait(limit_us) == 160            # warps 0 and 2..5 left through the give-up path
        assert lin.kernel_status() == bq.mmd.SELFTEST_CODE           # recorded ...
        assert lin.kernel_status() == 0                              # ... and cleared by the read
        after = lin.linear(X.cuda(), torch.float32, path=3)          # tensor memory was given back, the context is intact
        assert lin.kernel_status() == 0 and torch.equal(after, before)
    check_output(before, X, W, idx, F16, exact_expected=False)
    with pytest.raises(bq.BqError):
        lin.selftest_bounded_wait(0)
    lin.close()


@pytest.mark.parametrize("M,K,N,ko", [(64, 8192, 8192, 8), (64, 4096, 4736, 2), (33, 2048, 6272, 0), (64, 8192, 1024, 70), (1, 4096, 18816, 3),
                                       (64, 2048, 18944 - 128, 0)])
def test_decode_step_with_the_k_steps_of_all_tiles_dealt_out(bq, M, K, N, ko):
    """The stream-K kernel of decode-size calls: every CTA takes the same number of K steps across the tiles, tiles shared by
    several CTAs are finished by the last one to arrive.  Its integer sums are exact and its side sums are accumulated by one
    CTA in the order of the one-tile-per-CTA kernel, so the two must agree bit for bit; the oracle decides the rest.  Calls
    alternate with the other kernel through the same workspace; a workspace without the extra room is refused."""
    g = torch.Generator().manual_seed(M * 7 + N + ko)
    X = (torch.randn(M, K, generator=g) * 0.6).to(torch.float16)
    W = (torch.randn(N, K, generator=g) * 0.03).to(torch.float16)
    idx = np.sort(torch.randperm(K, generator=g)[:ko].numpy()).astype(np.int32)
    X[:, idx.tolist()] *= 25
    lin = bq.DecomposedLinear(W.cuda(), idx)
    Xd = X.cuda()
    assert lin.workspace_bytes(M) > lin.workspace_layout(M)[1]
    for out in (torch.float32, None):
        y_tile = lin.linear(Xd, out, path=bq.mmd.PATH_TENSOR_TILE)
        for _ in range(3):                                        # the counters are zeroed by every call's row kernel
            y_sk = lin.linear(Xd, out, path=bq.mmd.PATH_TENSOR_STREAMK)
            assert lin.kernel_status() == 0
            assert torch.equal(y_sk, y_tile)
        check_output(y_sk, X, W, idx, F16, exact_expected=(ko == 0))
    small = lin.workspace(M)
    with pytest.raises(bq.BqError):
        lin.linear(Xd, torch.float32, path=bq.mmd.PATH_TENSOR_STREAMK, workspace=small)
    lin.close()


def test_stream_k_is_refused_for_shapes_it_does_not_take(bq):
    g = torch.Generator().manual_seed(3)
    W = (torch.randn(512, 2048, generator=g) * 0.03).to(torch.float16)                # N below 1024
    lin = bq.DecomposedLinear(W.cuda(), np.zeros(0, np.int32))
    X = torch.randn(16, 2048, generator=g).to(torch.float16).cuda()
    assert lin.workspace_bytes(16) == lin.workspace_layout(16)[1]
    with pytest.raises(bq.BqError):
        lin.linear(X, torch.float32, path=bq.mmd.PATH_TENSOR_STREAMK)
    lin.close()
    W = (torch.randn(2048, 2048, generator=g) * 0.03).to(torch.float16)
    lin = bq.DecomposedLinear(W.cuda(), np.zeros(0, np.int32))
    X = torch.randn(100, 2048, generator=g).to(torch.float16).cuda()                   # more than 64 rows
    with pytest.raises(bq.BqError):
        lin.linear(X, torch.float32, path=bq.mmd.PATH_TENSOR_STREAMK)
    lin.close()


def test_output_of_more_than_2_32_elements(bq):
    """32768 tokens through a 256 -> 131080 layer: the output has 2^32 + 262144 elements, so the rows from 32766 on lie past
    element 2^32 (and every row past 16383 past byte 2^32).  No critical features, so every kernel's result is the oracle's
    bit for bit: the kernels are compared with each other on the whole output and with the oracle on the first, the last and
    64 drawn rows."""
    M, K, N = 32768, 256, 131080
    g = torch.Generator().manual_seed(77)
    X = (torch.randn((M, K), generator=g) * 0.5).to(torch.bfloat16)
    W = (torch.randn((N, K), generator=g) * 0.02).to(torch.bfloat16)
    idx = np.zeros(0, np.int32)
    lin = bq.DecomposedLinear(W.cuda(), idx)
    Xd = X.cuda()
    assert M * N > 1 << 32
    y_auto = lin.linear(Xd, None)
    assert lin.kernel_status() == 0
    rows = sorted(set(range(64)) | set(range(M - 64, M)) | set(np.random.default_rng(5).choice(M, 64, replace=False).tolist()))
    qw, sw, wo = mo.rowquant(bits(W), BF16, idx)
    y_ref = mo.linear(bits(X[rows]), BF16, qw, sw, wo, idx, BF16)
    assert np.array_equal(bits(y_auto[rows]), y_ref)
    for path in (1, 3, 4):
        y = lin.linear(Xd, None, path=path)
        assert lin.kernel_status() == 0
        assert torch.equal(y.view(torch.int16), y_auto.view(torch.int16)), path
        del y
    lin.close()
