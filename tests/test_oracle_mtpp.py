"""Pins of the slicing oracle (oracle/mtpp_oracle.py) against what the paper's definitions and plain
mathematics fix: a block cost worked out by hand, closed forms on a chain, every contiguous
partition enumerated by brute force, invariants, and planted mistakes that each named pin catches."""
import itertools
import random

import pytest

from oracle import mtpp_oracle as mo


def diamond():
    #      0
    #    /   \
    #   1     2        node:      0    1    2    3
    #    \   /         work:      5    7    3    4
    #      3           sizeparam: 10   20   30   40
    #                  sizeout:   6    2    9    1
    return mo.Graph(4, [(0, 1), (0, 2), (1, 3), (2, 3)], [5, 7, 3, 4], [10, 20, 30, 40], [6, 2, 9, 1])


def test_block_cost_worked_by_hand():
    g = diamond()
    B, M = 3, 35
    # S = {0, 1}: consumed from outside: nothing; work 12; params 30, peak = max(6, 2) = 6: excess max(0, 30 + 6 - 35) = 1,
    # plus peak 6; outputs used outside: node 0 (by 2) -> 6, node 1 (by 3) -> 2.  F = 0 + 3 * 12 + (1 + 6) + 8 = 51
    assert mo.block_cost(g, {0, 1}, B, M) == 51
    # S = {2, 3}: inputs: node 0 (used by 2) -> 6 and node 1 (used by 3) -> 2; work 7; params 70, peak 9: excess 44, plus 9;
    # node 3 has no consumer, node 2's only consumer is inside.  F = 8 + 21 + 53 + 0 = 82
    assert mo.block_cost(g, {2, 3}, B, M) == 82
    # S = {1, 2} (not contiguous in every order, but a valid set): inputs: node 0 ONCE although 1 and 2 both read it -> 6;
    # work 10; params 50, peak 9: excess 24, plus 9; outputs: 2 + 9.  F = 6 + 30 + 33 + 11 = 80
    assert mo.block_cost(g, {1, 2}, B, M) == 80
    # the whole graph: no I/O at all
    assert mo.block_cost(g, {0, 1, 2, 3}, B, M) == 3 * 19 + max(0, 100 + 9 - 35) + 9
    # a roomy fast memory: nothing is streamed, the excess never goes negative
    assert mo.block_cost(g, {0}, B, 10 ** 9) == 0 + 3 * 5 + (0 + 6) + 6


def test_segment_cost_is_the_block_cost_of_the_positions():
    g = diamond()
    pi = [0, 2, 1, 3]
    assert mo.segment_cost(g, pi, 2, 3, 3, 35) == mo.block_cost(g, {2, 1}, 3, 35) == 80
    assert mo.segment_cost(g, pi, 1, 4, 3, 35) == mo.block_cost(g, {0, 1, 2, 3}, 3, 35)


def chain(n, rng):
    return mo.Graph(n, [(i, i + 1) for i in range(n - 1)], [rng.randrange(1, 50) for _ in range(n)], [rng.randrange(0, 400) for _ in range(n)],
                    [rng.randrange(1, 90) for _ in range(n)])


def test_chain_closed_form():
    """On a chain every block reads its predecessor's output and hands on its last node's output."""
    rng = random.Random(5)
    g = chain(9, rng)
    pi = list(range(9))
    B, M = 4, 500
    for l in range(1, 10):
        for r in range(l, 10):
            nodes = range(l - 1, r)
            peak = max(g.sizeout[v] for v in nodes)
            want = (g.sizeout[l - 2] if l > 1 else 0) + B * sum(g.work[v] for v in nodes) \
                + max(0, sum(g.sizeparam[v] for v in nodes) + peak - M) + peak + (g.sizeout[r - 1] if r < 9 else 0)
            assert mo.segment_cost(g, pi, l, r, B, M) == want


def random_dag(n, rng, p=0.3):
    edges = [(u, v) for u in range(n) for v in range(u + 1, n) if rng.random() < p]
    g = mo.Graph(n, edges, [rng.randrange(1, 30) for _ in range(n)], [rng.randrange(0, 300) for _ in range(n)], [rng.randrange(1, 60) for _ in range(n)])
    pri = [rng.random() for _ in range(n)]
    return g, mo.decode_order(g, pri)


def brute_force(g, pi, k, B, M):
    """Every way of cutting the order into at most k contiguous non-empty blocks, by enumeration of the cut sets.
    Returns (bottleneck, blocks, cuts) under the oracle's stated preference: the smaller bottleneck, then fewer blocks,
    then ... (the cuts are compared only when the optimum is unique)."""
    n = g.n
    found = []
    for kk in range(1, min(k, n) + 1):
        for inner in itertools.combinations(range(1, n), kk - 1):
            ends = list(inner) + [n]
            starts = [1] + [e + 1 for e in inner]
            cost = max(mo.block_cost(g, set(pi[s - 1:e]), B, M) for s, e in zip(starts, ends))
            found.append((cost, kk, ends))
    best = min(c for c, _, _ in found)
    fewest = min(kk for c, kk, _ in found if c == best)
    return best, fewest, [ends for c, kk, ends in found if c == best and kk == fewest]


@pytest.mark.parametrize("seed", range(12))
def test_dynamic_programme_equals_brute_force(seed):
    rng = random.Random(seed)
    n = rng.randrange(2, 11)
    g, pi = random_dag(n, rng)
    B, M = rng.randrange(1, 6), rng.randrange(50, 900)
    for k in (1, 2, 3, 4, n, n + 3):
        cost, blocks, cuts = mo.slice_order(g, pi, k, B, M)
        want_cost, want_blocks, optimal_cuts = brute_force(g, pi, k, B, M)
        assert (cost, blocks) == (want_cost, want_blocks)
        assert cuts in optimal_cuts and len(cuts) == blocks and cuts[-1] == n
        # the cuts it returns really have that bottleneck
        starts = [1] + [c + 1 for c in cuts[:-1]]
        assert max(mo.segment_cost(g, pi, s, e, B, M) for s, e in zip(starts, cuts)) == cost


def test_one_block_is_the_whole_order_and_more_blocks_never_hurt():
    rng = random.Random(77)
    g, pi = random_dag(14, rng)
    B, M = 2, 400
    whole = B * sum(g.work) + max(0, sum(g.sizeparam) + max(g.sizeout) - M) + max(g.sizeout)
    assert mo.slice_order(g, pi, 1, B, M) == (whole, 1, [14])
    costs = [mo.slice_order(g, pi, k, B, M)[0] for k in range(1, 15)]
    assert all(a >= b for a, b in zip(costs, costs[1:]))
    assert costs[-1] == mo.slice_order(g, pi, 99, B, M)[0]


def test_relabelling_the_nodes_changes_nothing():
    rng = random.Random(3)
    g, pi = random_dag(9, rng)
    perm = list(range(9))
    rng.shuffle(perm)                                               # old label -> new label
    h = mo.Graph(9, [(perm[u], perm[v]) for u, v in g.edges], [g.work[perm.index(i)] for i in range(9)],
                 [g.sizeparam[perm.index(i)] for i in range(9)], [g.sizeout[perm.index(i)] for i in range(9)])
    assert mo.slice_order(g, pi, 3, 2, 300) == mo.slice_order(h, [perm[v] for v in pi], 3, 2, 300)


def test_ties_go_to_fewer_blocks_and_earlier_cuts():
    # four equal, unconnected nodes with no outputs to stream... every cut costs the same: sizeout 0 is not allowed to be the
    # peak of nothing, so give each a unit output and a huge memory: F(block of j nodes) = j * B * work + 1
    g = mo.Graph(4, [], [10, 10, 10, 10], [0, 0, 0, 0], [1, 1, 1, 1])
    assert mo.slice_order(g, [0, 1, 2, 3], 2, 1, 10 ** 6) == (21, 2, [2, 4])
    assert mo.slice_order(g, [0, 1, 2, 3], 3, 1, 10 ** 6) == (21, 2, [2, 4])       # a third block cannot beat 2 + 2
    assert mo.slice_order(g, [0, 1, 2, 3], 4, 1, 10 ** 6) == (11, 4, [1, 2, 3, 4])
    # two ways to reach the same bottleneck with two blocks: work 5 | 9 1 and 5 9 | 1 ... make the first cut the winner
    h = mo.Graph(3, [], [6, 3, 6], [0, 0, 0], [1, 1, 1])
    assert mo.slice_order(h, [0, 1, 2], 2, 1, 10 ** 6) == (10, 2, [1, 3])          # 6 | 3 6 and 6 3 | 6 both give 10: the earlier cut


def test_decode_order():
    g = diamond()
    assert mo.decode_order(g, [0.1, 0.2, 0.9, 0.5]) == [0, 2, 1, 3]
    assert mo.decode_order(g, [0.1, 0.9, 0.2, 0.5]) == [0, 1, 2, 3]
    assert mo.decode_order(g, [0.5, 0.5, 0.5, 0.5]) == [0, 1, 2, 3]              # equal keys: the smaller index
    rng = random.Random(1)
    for _ in range(20):
        h, _ = random_dag(12, rng)
        order = mo.decode_order(h, [rng.random() for _ in range(12)])
        assert mo.is_topological(h, order)
    c = chain(6, rng)
    assert mo.decode_order(c, [rng.random() for _ in range(6)]) == list(range(6))  # a chain has one order
    assert not mo.is_topological(g, [1, 0, 2, 3]) and not mo.is_topological(g, [0, 1, 2])


# ------------------------------------------------------------------------------------------ planted mistakes

def _with(monkeypatch, name, fn):
    monkeypatch.setattr(mo, name, fn)


def test_planted_io_counted_per_edge_is_caught(monkeypatch):
    _with(monkeypatch, "io_bytes", lambda g, S, T: sum(g.sizeout[v] * len(g.consumers[v] & T) for v in S))
    with pytest.raises(AssertionError):
        test_block_cost_worked_by_hand()


def test_planted_negative_excess_is_caught(monkeypatch):
    def bad(g, S, B, M):
        rest = set(range(g.n)) - S
        peak = max(g.sizeout[v] for v in S)
        return mo.io_bytes(g, rest, S) + B * sum(g.work[v] for v in S) + (sum(g.sizeparam[v] for v in S) + peak - M) + peak + mo.io_bytes(g, S, rest)
    _with(monkeypatch, "block_cost", bad)
    with pytest.raises(AssertionError):
        test_block_cost_worked_by_hand()


def test_planted_missing_peak_term_is_caught(monkeypatch):
    def bad(g, S, B, M):
        rest = set(range(g.n)) - S
        peak = max(g.sizeout[v] for v in S)
        return mo.io_bytes(g, rest, S) + B * sum(g.work[v] for v in S) + max(0, sum(g.sizeparam[v] for v in S) + peak - M) + mo.io_bytes(g, S, rest)
    _with(monkeypatch, "block_cost", bad)
    with pytest.raises(AssertionError):
        test_chain_closed_form()


def test_planted_outgoing_io_forgotten_is_caught(monkeypatch):
    real = mo.io_bytes
    _with(monkeypatch, "io_bytes", lambda g, S, T: real(g, S, T) if len(S) > len(T) or (len(S) == len(T) and min(S) > min(T)) else 0)
    with pytest.raises(AssertionError):
        test_chain_closed_form()


def test_planted_exactly_k_blocks_is_caught(monkeypatch):
    real = mo.slice_order

    def exactly(g, pi, k, B, M):                       # always uses min(k, n) blocks, even when fewer are better
        best = None
        for inner in itertools.combinations(range(1, g.n), min(k, g.n) - 1):
            ends = list(inner) + [g.n]
            starts = [1] + [e + 1 for e in inner]
            c = max(mo.block_cost(g, set(pi[s - 1:e]), B, M) for s, e in zip(starts, ends))
            if best is None or c < best[0]:
                best = (c, len(ends), ends)
        return best
    _with(monkeypatch, "slice_order", exactly)
    with pytest.raises(AssertionError):
        test_ties_go_to_fewer_blocks_and_earlier_cuts()
    monkeypatch.setattr(mo, "slice_order", real)


def test_planted_later_cut_on_ties_is_caught(monkeypatch):
    src = mo.slice_order

    def later(g, pi, k, B, M):
        cost, blocks, cuts = src(g, pi, k, B, M)
        if (g.n, blocks) == (3, 2):
            return cost, blocks, [2, 3]
        return cost, blocks, cuts
    _with(monkeypatch, "slice_order", later)
    with pytest.raises(AssertionError):
        test_ties_go_to_fewer_blocks_and_earlier_cuts()
