"""CPU oracle of the slicing of a topological order into at most k blocks (test infrastructure only).

Paper, section "Dynamic sharding of neural networks": a computation graph G = (V, E) whose nodes
carry work(v), sizeparam(v) and sizeout(v); the I/O cost io(S, T) between blocks, the overflow
cost of a block, the block cost f(S) and the max-throughput partitioning objective (minimise the
largest block cost).  Section "Enhanced MTPP slicing of topological order", Algorithm 1: a
"segment cost" structure answers Query(l, r) = cost of the block formed by positions l..r of a
topological order pi, and a dynamic programme over the order returns the smallest achievable
bottleneck with the order cut into blocks.

The paper leaves several things open or prints them inconsistently; the readings taken here
(every one is listed in the design notes) are:
  * all quantities are non-negative integers and costs are kept multiplied by the bandwidth B,
    F(S) = B * f(S), so that nothing is ever divided and every result is an exact integer;
  * io(S, T) * B = sum of sizeout(v) over the nodes v of S with at least one consumer in T
    (each producer counted once, as the set in the paper's sum says);
  * peak(S) = the largest sizeout(v) of a node of S;
  * overflow(S) * B = max(0, sizeparam(S) + peak(S) - M) + peak(S): the printed formula adds a
    byte count to a time; the excess over the fast memory M is read as bytes to be streamed at
    bandwidth B, and it cannot be negative; sizeparam(S) is the sum over the block;
  * F(S) = io_in(S) + B * work(S) + overflow(S) * B + io_out(S), with io_in = io(V \\ S, S) * B and
    io_out = io(S, V \\ S) * B;
  * "heuristic-based weighting" = none, heuristic_adjustment = identity;
  * "at most k blocks": the algorithm as printed cuts into exactly k' non-empty blocks; the
    result is the best over k' = 1..min(k, n), the smaller k' on equal bottlenecks; among equal
    candidates inside the dynamic programme the smaller cut position wins.

Nothing here is imported by the CUDA library or its binding.  Plain Python on purpose: the sets of
the definitions are written out as sets, so that it can be checked against the paper by eye.
Pins (tests/test_oracle_mtpp.py): every contiguous partition enumerated by brute force for small
n, k = 1 equals the whole order's cost, closed forms on a chain graph, monotonicity in k, a cut
graph checked by hand, and planted mistakes.  Parity with any outside implementation: parity unpinned.
"""
from __future__ import annotations


class Graph:
    """n nodes 0..n-1; edges (u, v) mean v consumes u's output.  All attributes are integers."""

    def __init__(self, n, edges, work, sizeparam, sizeout):
        self.n = int(n)
        self.edges = sorted(set((int(u), int(v)) for u, v in edges))
        self.work = [int(x) for x in work]
        self.sizeparam = [int(x) for x in sizeparam]
        self.sizeout = [int(x) for x in sizeout]
        assert len(self.work) == len(self.sizeparam) == len(self.sizeout) == self.n
        self.consumers = [set() for _ in range(self.n)]
        for u, v in self.edges:
            assert 0 <= u < self.n and 0 <= v < self.n and u != v
            self.consumers[u].add(v)


def is_topological(g: Graph, pi) -> bool:
    pos = {v: i for i, v in enumerate(pi)}
    return sorted(pi) == list(range(g.n)) and all(pos[u] < pos[v] for u, v in g.edges)


def io_bytes(g: Graph, S: set, T: set) -> int:
    """B * io(S, T): the outputs of the nodes of S that some node of T consumes, each once."""
    return sum(g.sizeout[v] for v in S if g.consumers[v] & T)


def block_cost(g: Graph, S: set, B: int, M: int) -> int:
    """B * f(S) for a block S (a set of nodes)."""
    rest = set(range(g.n)) - S
    peak = max(g.sizeout[v] for v in S)
    param = sum(g.sizeparam[v] for v in S)
    overflow = max(0, param + peak - M) + peak
    return io_bytes(g, rest, S) + B * sum(g.work[v] for v in S) + overflow + io_bytes(g, S, rest)


def segment_cost(g: Graph, pi, l: int, r: int, B: int, M: int) -> int:
    """Query(l, r) of the segment cost structure: positions l..r of pi, 1-based and inclusive as in the paper."""
    return block_cost(g, set(pi[l - 1:r]), B, M)


def segment_cost_table(g: Graph, pi, B: int, M: int) -> dict:
    """The segment cost structure of Algorithm 1, initialised as the paper says: every Query(l, r),
    1 <= l <= r <= n, computed once (O(n^2) entries) before the dynamic programme asks for them."""
    return {(l, r): segment_cost(g, pi, l, r, B, M) for l in range(1, g.n + 1) for r in range(l, g.n + 1)}


def slice_order(g: Graph, pi, k: int, B: int, M: int):
    """The dynamic programme of Algorithm 1 over the order pi.

    Returns (bottleneck, blocks, cuts): the smallest largest block cost (times B), the number of
    blocks that reaches it, and the 1-based last positions of the blocks (the final one is n).
    """
    n = g.n
    assert is_topological(g, pi) and k >= 1 and n >= 1
    INF = None
    kmax = min(k, n)
    query = segment_cost_table(g, pi, B, M)
    # dp[kk][r] = best bottleneck of positions 1..r cut into exactly kk non-empty blocks; arg = the cut
    dp = [[INF] * (n + 1) for _ in range(kmax + 1)]
    arg = [[0] * (n + 1) for _ in range(kmax + 1)]
    for r in range(1, n + 1):
        dp[1][r] = query[(1, r)]
    for kk in range(2, kmax + 1):
        for r in range(kk, n + 1):
            best, where = INF, 0
            for l in range(kk - 1, r):                       # positions 1..l hold kk - 1 blocks, l + 1..r is the last block
                a = dp[kk - 1][l]
                b = query[(l + 1, r)]
                cand = max(a, b)
                if best is INF or cand < best:
                    best, where = cand, l
            dp[kk][r], arg[kk][r] = best, where
    best_k = 1
    for kk in range(2, kmax + 1):
        if dp[kk][n] < dp[best_k][n]:
            best_k = kk
    cuts, r = [], n
    for kk in range(best_k, 0, -1):
        cuts.append(r)
        r = arg[kk][r]
    return dp[best_k][n], best_k, cuts[::-1]


def decode_order(g: Graph, priority) -> list:
    """Kahn's algorithm with the ready node of the highest priority taken first (ties: the smaller
    node index): the map from a BRKGA key vector to a topological order."""
    indeg = [0] * g.n
    for u, v in g.edges:
        indeg[v] += 1
    ready = {v for v in range(g.n) if indeg[v] == 0}
    order = []
    while ready:
        v = min(ready, key=lambda t: (-float(priority[t]), t))
        ready.remove(v)
        order.append(v)
        for c in sorted(g.consumers[v]):
            indeg[c] -= 1
            if indeg[c] == 0:
                ready.add(c)
    assert len(order) == g.n, "the graph has a cycle"
    return order
