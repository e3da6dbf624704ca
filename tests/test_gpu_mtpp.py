"""GPU parity of the slicing of topological orders (include/mtpp.h) against the CPU oracle: the decoded
orders, the bottleneck cost, the number of blocks and the cut positions are integers and must be identical."""
import random

import numpy as np
import pytest
import torch

from oracle import mtpp_oracle as mo
from paper_2407_19775_b200 import workloads

pytestmark = pytest.mark.gpu


def oracle_graph(n, edges, work, sizeparam, sizeout):
    return mo.Graph(n, [tuple(e) for e in edges.tolist()], work.tolist(), sizeparam.tolist(), sizeout.tolist())


def check_population(bq, name, population, ks, sample=None):
    w = workloads.GRAPH_WORKLOADS[name]
    n, edges, work, sizeparam, sizeout = workloads.make_graph(name)
    g = oracle_graph(n, edges, work, sizeparam, sizeout)
    dg = bq.mtpp.SliceGraph(n, edges, work, sizeparam, sizeout, device="cuda:0")
    keys = workloads.make_keys(name, population)
    orders = dg.decode_orders(keys.cuda())
    torch.cuda.synchronize()
    got_orders = orders.cpu().numpy()
    rows = range(population) if sample is None else sample
    for p in rows:
        assert got_orders[p].tolist() == mo.decode_order(g, keys[p].tolist()), f"order {p}"
    for k in ks:
        cost, blocks, cuts, status = dg.slice_orders(orders, k, w.B, w.M)
        torch.cuda.synchronize()
        assert int(status.sum()) == 0
        cost, blocks, cuts = cost.cpu().numpy(), blocks.cpu().numpy(), cuts.cpu().numpy()
        for p in rows:
            want = mo.slice_order(g, got_orders[p].tolist(), k, w.B, w.M)
            got = (int(cost[p]), int(blocks[p]), cuts[p][:blocks[p]].tolist())
            assert got == want, f"order {p}, k {k}"
            assert not cuts[p][blocks[p]:].any()
        # every order: the cuts it returns have the bottleneck it returns, under the oracle's block cost (cheap: k blocks each)
        if sample is not None:
            for p in range(0, population, max(1, population // 64)):
                ends = cuts[p][:blocks[p]].tolist()
                starts = [1] + [e + 1 for e in ends[:-1]]
                pi = got_orders[p].tolist()
                assert mo.is_topological(g, pi) and ends[-1] == n
                assert max(mo.segment_cost(g, pi, s, e, w.B, w.M) for s, e in zip(starts, ends)) == int(cost[p])
    dg.close()


def test_tiny_graph_every_order_every_k(bq):
    check_population(bq, "mtpp_tiny", 6, [1, 2, 3, 5, 14, 16])


def test_trunk_with_heads(bq):
    check_population(bq, "mtpp_heads", 24, [1, 4, 7], sample=range(0, 24, 2))


def test_unet_population_sampled_orders(bq):
    """The benchmark's population in its launch configuration (2048 orders of 256 nodes, 8 blocks): three orders in full
    against the oracle, and on every 32nd order the returned cuts re-costed by the oracle."""
    check_population(bq, "mtpp_unet", 2048, [8], sample=[0, 1, 2047])


def test_random_graphs_fuzz(bq):
    rng = random.Random(7)
    for case in range(12):
        n = rng.choice([1, 2, 3, 17, 33, 64, 100])
        edges = np.asarray([(u, v) for u in range(n) for v in range(u + 1, n) if rng.random() < rng.choice([0.0, 0.05, 0.3])], np.int32).reshape(-1, 2)
        scale = 1 << 21 if case % 2 else 1                                   # odd cases: costs beyond 32 bits, the wide instances
        work = np.asarray([rng.randrange(0, 50) for _ in range(n)], np.int64)
        sizeparam = np.asarray([rng.randrange(0, 500) for _ in range(n)], np.int64) * scale
        sizeout = np.asarray([rng.randrange(0, 80) for _ in range(n)], np.int64) * scale
        g = oracle_graph(n, edges, work, sizeparam, sizeout)
        dg = bq.mtpp.SliceGraph(n, edges, work, sizeparam, sizeout, device="cuda:0")
        P = 5
        keys = torch.rand((P, n), generator=torch.Generator().manual_seed(case))
        if case % 3 == 0:
            keys = (keys * 3).floor() / 3                                    # many equal keys: the node index decides
        orders = dg.decode_orders(keys.cuda())
        B, M, k = rng.randrange(1, 9) * scale, rng.randrange(0, 2000) * scale, rng.choice([1, 2, 5, 16])
        cost, blocks, cuts, status = dg.slice_orders(orders, k, B, M)
        torch.cuda.synchronize()
        for p in range(P):
            pi = orders[p].cpu().tolist()
            assert pi == mo.decode_order(g, keys[p].tolist())
            assert (int(cost[p]), int(blocks[p]), cuts[p][:int(blocks[p])].cpu().tolist()) == mo.slice_order(g, pi, k, B, M), (case, p)
        dg.close()


def banded_graph(n, seed, scale=1, density=0.08):
    rng = random.Random(seed)
    edges = np.asarray([(u, v) for u in range(n) for v in range(u + 1, min(n, u + 40)) if rng.random() < density], np.int32).reshape(-1, 2)
    work = np.asarray([rng.randrange(0, 50) for _ in range(n)], np.int64)
    sizeparam = np.asarray([rng.randrange(0, 500) for _ in range(n)], np.int64) * scale
    sizeout = np.asarray([rng.randrange(0, 80) for _ in range(n)], np.int64) * scale
    return edges, work, sizeparam, sizeout


@pytest.mark.parametrize("n,k,scale", [(130, 3, 1), (200, 4, 1 << 21), (257, 16, 1), (300, 5, 1 << 21), (520, 3, 1), (513, 2, 1 << 21)])
def test_graphs_wider_than_one_position_per_thread(bq, n, k, scale):
    """Above 128 nodes a thread of the slicing kernel owns two first positions, above 256 the CTA has eight warps, above 512 a
    thread owns four: one order of each in full against the oracle, with costs inside 32 bits and beyond them."""
    edges, work, sizeparam, sizeout = banded_graph(n, n, scale)
    g = oracle_graph(n, edges, work, sizeparam, sizeout)
    dg = bq.mtpp.SliceGraph(n, edges, work, sizeparam, sizeout, device="cuda:0")
    keys = torch.rand((3, n), generator=torch.Generator().manual_seed(n))
    orders = dg.decode_orders(keys.cuda())
    cost, blocks, cuts, status = dg.slice_orders(orders, k, 3 * scale, 20000 * scale)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, 0, 0]
    pi = orders[1].cpu().tolist()
    assert pi == mo.decode_order(g, keys[1].tolist())
    assert (int(cost[1]), int(blocks[1]), cuts[1][:int(blocks[1])].cpu().tolist()) == mo.slice_order(g, pi, k, 3 * scale, 20000 * scale)
    dg.close()


@pytest.mark.parametrize("scale,density", [(1, 0.08), (1 << 21, 0.08), (1, 0.4)])
def test_largest_graph(bq, scale, density):
    """1024 nodes, 16 blocks, the limits of the call.  A chain of equal nodes has a closed form: every block's cost grows with
    its length, so the best slicing is the balanced one and its bottleneck is the cost of an inner block of ceil(n / k) nodes.
    On a banded random graph the oracle re-costs the returned cuts (16 blocks an order) and no perturbed cut set does better.
    With costs beyond 32 bits, or with some 15,000 edges, the order's edges no longer fit in shared memory beside the programme's
    arrays and are looked up in global memory."""
    n, k, B, M = 1024, 16, 3 * scale, 20000 * scale
    chain = np.asarray([(i, i + 1) for i in range(n - 1)], np.int32)
    ones = np.ones(n, np.int64) * scale
    g = oracle_graph(n, chain, 7 * ones // scale, 300 * ones, 11 * ones)
    dg = bq.mtpp.SliceGraph(n, chain, 7 * ones // scale, 300 * ones, 11 * ones, device="cuda:0")
    orders = dg.decode_orders(torch.rand((2, n), generator=torch.Generator().manual_seed(1)).cuda())
    assert orders.cpu().tolist() == [list(range(n))] * 2                   # a chain has one topological order
    cost, blocks, cuts, status = dg.slice_orders(orders, k, B, M)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, 0]
    assert cost.cpu().tolist() == [mo.segment_cost(g, list(range(n)), 65, 128, B, M)] * 2
    ends = cuts[0][:int(blocks[0])].cpu().tolist()
    assert max(e - s for s, e in zip([0] + ends[:-1], ends)) == 64 and ends[-1] == n
    dg.close()

    edges, work, sizeparam, sizeout = banded_graph(n, 5, scale, density)
    g = oracle_graph(n, edges, work, sizeparam, sizeout)
    dg = bq.mtpp.SliceGraph(n, edges, work, sizeparam, sizeout, device="cuda:0")
    keys = torch.rand((4, n), generator=torch.Generator().manual_seed(2))
    orders = dg.decode_orders(keys.cuda())
    cost, blocks, cuts, status = dg.slice_orders(orders, k, B, M)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0] * 4
    rng = random.Random(9)

    def bottleneck(pi, ends):
        return max(mo.segment_cost(g, pi, s, e, B, M) for s, e in zip([1] + [e + 1 for e in ends[:-1]], ends))

    for p in range(4):
        pi = orders[p].cpu().tolist()
        assert pi == mo.decode_order(g, keys[p].tolist())
        ends = cuts[p][:int(blocks[p])].cpu().tolist()
        assert ends == sorted(set(ends)) and ends[-1] == n and 1 <= len(ends) <= k
        assert bottleneck(pi, ends) == int(cost[p])
        for _ in range(6):                                                # other cut sets: a nudge of every cut, and a fresh draw
            nudged = sorted({min(n - 1, max(1, e + rng.randrange(-2, 3))) for e in ends[:-1]}) + [n]
            drawn = sorted(rng.sample(range(1, n), k - 1)) + [n]
            assert bottleneck(pi, nudged) >= int(cost[p]) and bottleneck(pi, drawn) >= int(cost[p])
    dg.close()


@pytest.mark.parametrize("pad", [-3, -2, -1, 0, 1, 2])
@pytest.mark.parametrize("M", [0, 10 ** 9, (1 << 62) - 1])
def test_costs_on_either_side_of_the_32_bit_bound(bq, pad, M):
    """The library runs the programme in 32-bit words when its bound on any segment cost, sum of outputs + 2 largest output
    + sum of parameters + B * sum of work, is below 2^31 - 1, and in 64-bit words otherwise: graphs whose bound sits at
    2^31 - 1 + pad, and whose whole-order cost comes close to it, against the oracle."""
    n, B, k = 40, 3, 4
    rng = random.Random(pad * 7 + 100)
    edges = np.asarray([(i, i + 1) for i in range(n - 1)] + [(i, i + 5) for i in range(0, n - 5, 3)], np.int32)
    work = np.asarray([rng.randrange(1, 10 ** 6) for _ in range(n)], np.int64)
    sizeout = np.asarray([rng.randrange(1, 10 ** 6) for _ in range(n)], np.int64)
    sizeparam = np.asarray([rng.randrange(0, 10 ** 7) for _ in range(n)], np.int64)
    bound = int(sizeout.sum() + 2 * sizeout.max() + sizeparam.sum() + B * work.sum())
    sizeparam[7] += (1 << 31) - 1 + pad - bound                              # parameters take up the slack
    assert int(sizeout.sum() + 2 * sizeout.max() + sizeparam.sum() + B * work.sum()) == (1 << 31) - 1 + pad
    g = oracle_graph(n, edges, work, sizeparam, sizeout)
    dg = bq.mtpp.SliceGraph(n, edges, work, sizeparam, sizeout, device="cuda:0")
    orders = dg.decode_orders(torch.rand((2, n), generator=torch.Generator().manual_seed(3)).cuda())
    for kk in (1, k):
        cost, blocks, cuts, status = dg.slice_orders(orders, kk, B, M)
        torch.cuda.synchronize()
        assert status.cpu().tolist() == [0, 0]
        for p in range(2):
            pi = orders[p].cpu().tolist()
            assert (int(cost[p]), int(blocks[p]), cuts[p][:int(blocks[p])].cpu().tolist()) == mo.slice_order(g, pi, kk, B, M), (kk, p)
    dg.close()


def test_decoding_with_keys_of_either_sign_zeros_and_repeats(bq):
    """Keys are compared as floats: negative keys, -0.0 beside +0.0 (equal: the smaller node goes first), repeated values,
    huge and tiny magnitudes, infinities; on graphs with one word of ready bits, several, and the most (1024 nodes), with the
    consumer lists in shared memory and, for the dense one, in global memory."""
    rng = random.Random(11)
    pool = [0.0, -0.0, 1.0, -1.0, 0.5, -0.5, 1e-38, -1e-38, 3e38, -3e38, float("inf"), float("-inf"), 0.25, 0.25, 2.0 ** -149, -(2.0 ** -149)]
    for n, density in ((20, 0.2), (100, 0.05), (333, 0.08), (1024, 0.08), (1024, 0.3)):
        edges = np.asarray([(u, v) for u in range(n) for v in range(u + 1, min(n, u + 40)) if rng.random() < density], np.int32).reshape(-1, 2)
        ones = np.ones(n, np.int64)
        g = oracle_graph(n, edges, ones, ones, ones)
        dg = bq.mtpp.SliceGraph(n, edges, ones, ones, ones, device="cuda:0")
        P = 6
        keys = torch.tensor([[rng.choice(pool) if p % 2 else rng.uniform(-1, 1) for _ in range(n)] for p in range(P)], dtype=torch.float32)
        keys[2] = -0.0
        keys[2, ::3] = 0.0
        orders = dg.decode_orders(keys.cuda()).cpu()
        for p in range(P if n <= 333 else 3):
            assert orders[p].tolist() == mo.decode_order(g, keys[p].tolist()), (n, density, p)
        dg.close()


@pytest.mark.parametrize("scale", [1, 1 << 21])
def test_complete_graph_whose_edges_stay_in_global_memory(bq, scale):
    """Every pair (u, v), u < v, is an edge: 232 nodes have 26,796 edges, more than fit in shared memory beside the
    programme's arrays, so the four-warp instance looks them up in global memory.  One topological order; in full against the oracle."""
    n, k = 232, 4
    edges = np.asarray([(u, v) for u in range(n) for v in range(u + 1, n)], np.int32)
    work = np.full(n, 3, np.int64)
    sizeparam = np.full(n, 5, np.int64) * scale
    sizeout = np.asarray([7 + i % 5 for i in range(n)], np.int64) * scale
    g = oracle_graph(n, edges, work, sizeparam, sizeout)
    dg = bq.mtpp.SliceGraph(n, edges, work, sizeparam, sizeout, device="cuda:0")
    orders = dg.decode_orders(torch.rand((2, n), generator=torch.Generator().manual_seed(4)).cuda())
    assert orders.cpu().tolist() == [list(range(n))] * 2
    cost, blocks, cuts, status = dg.slice_orders(orders, k, 2 * scale, 100 * scale)
    torch.cuda.synchronize()
    want = mo.slice_order(g, list(range(n)), k, 2 * scale, 100 * scale)
    for p in range(2):
        assert int(status[p]) == 0 and (int(cost[p]), int(blocks[p]), cuts[p][:int(blocks[p])].cpu().tolist()) == want
    dg.close()


def test_rows_that_are_not_topological_orders_are_flagged(bq):
    n, edges, work, sizeparam, sizeout = workloads.make_graph("mtpp_tiny")
    g = oracle_graph(n, edges, work, sizeparam, sizeout)
    dg = bq.mtpp.SliceGraph(n, edges, work, sizeparam, sizeout, device="cuda:0")
    good = mo.decode_order(g, [0.5] * n)
    u, v = edges[0]
    swapped = list(good)
    iu, iv = swapped.index(u), swapped.index(v)
    swapped[iu], swapped[iv] = swapped[iv], swapped[iu]                   # a consumer before its producer
    twice = list(good); twice[3] = twice[4]
    outside = list(good); outside[0] = n + 5
    negative = list(good); negative[2] = -1
    orders = torch.tensor([good, swapped, twice, outside, negative, good], dtype=torch.int32, device="cuda:0")
    cost, blocks, cuts, status = dg.slice_orders(orders, 3, 2, 1000)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, 1, 1, 1, 1, 0]
    assert cost.cpu().tolist()[1:5] == [-1] * 4 and blocks.cpu().tolist()[1:5] == [0] * 4 and not cuts[1:5].any()
    want = mo.slice_order(g, good, 3, 2, 1000)
    for p in (0, 5):
        assert (int(cost[p]), int(blocks[p]), cuts[p][:int(blocks[p])].cpu().tolist()) == want
    with pytest.raises(bq.BqError):
        dg.slice_orders(orders, 17, 2, 1000)
    with pytest.raises(bq.BqError):
        dg.slice_orders(orders, 3, 0, 1000)
    dg.close()
