"""Pins for the oracle's neighbour sampler (Sec. 4.1 "Mini-batch and Negative Sampling": mini-batches
are shrunk to a message-flow graph by a GraphSAGE neighbour sampler).

What fixes the result without the routine itself: a sample is a subset of the true neighbourhood of
the right size, drawn without replacement; with a fan-out that covers every degree it is the whole
L-hop neighbourhood (brute force with Python sets); every neighbour of a node is kept with the same
frequency fanout / degree (chi-square over many seeds); the next frontier is the ascending union;
blocks index into it and keep the row order; the selection is the `fanout` smallest keys when the keys
are recomputed from the pinned SplitMix64 step.
"""
import numpy as np

import oracle
from paper_2305_09887_b200 import inputs


def _graph(seed=1, n=300, m=2400):
    g = inputs.uniform_graph(n, m, seed)
    return g.rowptr.astype(np.int64), g.col


def _rows(rp, cp, v):
    return cp[rp[v]:rp[v + 1]]


def test_sample_is_a_subset_of_the_right_size_in_row_order():
    rp, cp = _graph()
    frontier = np.array(sorted(np.random.default_rng(0).choice(300, size=40, replace=False)), dtype=np.int32)
    for fanout in (1, 3, 8, 100):
        brp, bcol, nxt = oracle.sample_hop(rp, cp, frontier, fanout, 1234, 0)
        assert np.all(np.diff(nxt) > 0)                                   # ascending, distinct
        assert set(frontier.tolist()) <= set(nxt.tolist())               # a node keeps itself
        seen = set(frontier.tolist())
        for i, v in enumerate(frontier):
            kept = nxt[bcol[brp[i]:brp[i + 1]]]                            # back to node ids
            full = _rows(rp, cp, v)
            assert kept.size == min(full.size, fanout)
            assert len(set(kept.tolist())) == kept.size                   # without replacement (simple graph)
            # a subsequence of the row: same relative order as in the node's row
            pos = [int(np.flatnonzero(full == u)[0]) for u in kept]
            assert pos == sorted(pos)
            seen |= set(kept.tolist())
        assert set(nxt.tolist()) == seen                                  # nothing else enters the frontier


def test_large_fanout_gives_the_whole_neighbourhood_hop_by_hop():
    rp, cp = _graph(seed=2, n=200, m=500)
    frontier = np.array([3, 57, 120], dtype=np.int32)
    ball = set(frontier.tolist())
    for hop in range(3):
        brp, bcol, nxt = oracle.sample_hop(rp, cp, frontier, 10_000, 5, hop)
        grown = set(ball)
        for v in ball:
            grown |= set(_rows(rp, cp, v).tolist())
        assert set(nxt.tolist()) == grown                                 # brute-force (hop + 1)-hop ball
        for i, v in enumerate(frontier):
            assert np.array_equal(nxt[bcol[brp[i]:brp[i + 1]]], _rows(rp, cp, v))   # the whole row, in order
        frontier, ball = nxt, grown


def test_every_neighbour_is_kept_equally_often():
    # a node with 20 neighbours, fan-out 5, 4000 seeds: each neighbour kept about 1000 times
    n = 21
    rp = np.array([0] + [20] * 1 + list(range(21, 41)), dtype=np.int64)   # node 0 -> 1..20, node k -> 0
    cp = np.array(list(range(1, 21)) + [0] * 20, dtype=np.int32)
    assert rp.size == n + 1
    counts = np.zeros(21)
    for seed in range(4000):
        brp, bcol, nxt = oracle.sample_hop(rp, cp, np.array([0], dtype=np.int32), 5, seed, 0)
        kept = nxt[bcol[brp[0]:brp[1]]]
        assert kept.size == 5
        counts[kept] += 1
    expect = 4000 * 5 / 20
    chi2 = ((counts[1:] - expect) ** 2 / expect).sum()
    assert chi2 < 43.8                                                     # 19 degrees of freedom, p = 0.001
    # different hops of the same seed draw differently
    a = [tuple(oracle.sample_hop(rp, cp, np.array([0], dtype=np.int32), 5, s, 0)[2]) for s in range(50)]
    b = [tuple(oracle.sample_hop(rp, cp, np.array([0], dtype=np.int32), 5, s, 1)[2]) for s in range(50)]
    assert sum(x != y for x, y in zip(a, b)) > 40


def test_selection_is_the_smallest_keys_of_the_pinned_hash():
    rp, cp = _graph(seed=4, n=120, m=1500)
    seed, hop, fanout = 0xABCDEF, 2, 4
    frontier = np.arange(0, 120, 7, dtype=np.int32)
    brp, bcol, nxt = oracle.sample_hop(rp, cp, frontier, fanout, seed, hop)
    base = oracle.splitmix64(seed ^ ((hop + 1) << 48))
    for i, v in enumerate(frontier):
        row = _rows(rp, cp, v)
        if row.size <= fanout:
            continue
        keys = [(oracle.splitmix64(base ^ ((int(v) << 32) | q)), q) for q in range(row.size)]
        want = sorted(q for _, q in sorted(keys)[:fanout])
        assert np.array_equal(nxt[bcol[brp[i]:brp[i + 1]]], row[want])


def test_empty_frontier_and_isolated_nodes():
    rp = np.array([0, 0, 1, 2, 2], dtype=np.int64)
    cp = np.array([2, 1], dtype=np.int32)
    brp, bcol, nxt = oracle.sample_hop(rp, cp, np.empty(0, dtype=np.int32), 3, 1, 0)
    assert brp.tolist() == [0] and bcol.size == 0 and nxt.size == 0
    brp, bcol, nxt = oracle.sample_hop(rp, cp, np.array([0, 3], dtype=np.int32), 3, 1, 0)
    assert brp.tolist() == [0, 0, 0] and nxt.tolist() == [0, 3]           # isolated nodes keep only themselves
