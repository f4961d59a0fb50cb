"""Pins for the oracle's integer half: hash, assignment, relabel, induced CSR.

None of the expected values below come from the oracle itself: they are the
published SplitMix64 vector, ratios printed in the paper, closed forms from
Sec. 3.2.2 and Lemma 1, or brute force written with Python sets.
"""
import os

import numpy as np
import pytest

import oracle
from paper_2305_09887_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
GAMMA = 0x9E3779B97F4A7C15
MASK = 2**64 - 1


def _golden_lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_hash_matches_published_splitmix64_vector():
    expected = [int(t[0], 16) for t in _golden_lines("splitmix64_seed0.txt")]
    got = [oracle.splitmix64((k * GAMMA) & MASK) for k in range(len(expected))]
    assert got == expected


def test_hash_is_a_bijection_step_on_samples():
    # the mixing function is invertible, so distinct inputs give distinct outputs
    xs = np.random.default_rng(1).integers(0, 2**63, size=20000, dtype=np.uint64)
    out = {oracle.splitmix64(int(x)) for x in np.unique(xs)}
    assert len(out) == np.unique(xs).size


@pytest.mark.parametrize("M", [3, 4, 8, 23, 32])
def test_assignment_is_uniform_chi_square(M):
    n = 1_000_000
    part_id = oracle.assign(n, None, 0x5EED0005, M)
    counts = np.bincount(part_id, minlength=M)
    assert counts.size == M
    expected = n / M
    chi2 = float(((counts - expected) ** 2 / expected).sum())
    # chi-square with M-1 dof: mean M-1, sd sqrt(2(M-1)); 6 sd is far in the tail
    assert chi2 < (M - 1) + 6 * np.sqrt(2 * (M - 1)) + 6


def test_assignment_uses_seed_xor_id():
    # h(seed ^ v): flipping the seed by a constant c permutes which node gets which
    # draw: node v under seed s equals node v^c under seed s^c.
    n, M, s, c = 4096, 7, 0xABCDEF12345, 0x3FF
    a = oracle.assign(n, None, s, M)
    b = oracle.assign(n, None, s ^ c, M)
    v = np.arange(n)
    assert np.array_equal(a[v], b[v ^ c])


@pytest.mark.parametrize("n,M", [(1, 1), (5, 8), (2000, 4), (50_000, 32)])
def test_relabel_invariants(n, M):
    part_id, part_offsets, perm, local_id = oracle.partition(n, None, 99, M)
    assert part_offsets[0] == 0 and part_offsets[-1] == n
    assert np.array_equal(np.diff(part_offsets), np.bincount(part_id, minlength=M))
    assert np.array_equal(np.sort(perm), np.arange(n))                # each node exactly once
    assert np.array_equal(perm[part_offsets[part_id] + local_id], np.arange(n))  # inverse maps
    for p in range(M):
        seg = perm[part_offsets[p]:part_offsets[p + 1]]
        assert np.all(part_id[seg] == p)
        assert np.all(np.diff(seg) > 0)                               # ascending global id


def test_relabel_brute_force_small():
    part_id = np.array([2, 0, 2, 1, 0, 0, 2], dtype=np.int32)
    part_offsets, perm, local_id = oracle.relabel(part_id, 4)
    assert part_offsets.tolist() == [0, 3, 4, 7, 7]
    assert perm.tolist() == [1, 4, 5, 3, 0, 2, 6]
    assert local_id.tolist() == [0, 0, 1, 0, 1, 2, 2]


def test_grouped_relabel_hand_example():
    # parts:  node 0..7 -> [1, 0, 1, 0, 1, 0, 1, 1]; super-nodes (negative and sparse ids allowed)
    part_id = np.array([1, 0, 1, 0, 1, 0, 1, 1], dtype=np.int32)
    group = np.array([9, 4, -3, 4, 9, -8, -3, 9], dtype=np.int32)
    part_offsets, perm, local_id = oracle.relabel_grouped(part_id, group, 2)
    assert part_offsets.tolist() == [0, 3, 8]
    # part 0 holds nodes 1, 3 (super-node 4) and 5 (super-node -8): -8 first, then 4 with ids ascending
    # part 1 holds 2, 6 (super-node -3) then 0, 4, 7 (super-node 9)
    assert perm.tolist() == [5, 1, 3, 2, 6, 0, 4, 7]
    assert local_id.tolist() == [2, 1, 0, 2, 3, 0, 1, 4]


@pytest.mark.parametrize("n,M,groups", [(1, 1, 1), (9, 4, 3), (5000, 8, 60), (60_000, 32, 700)])
def test_grouped_relabel_is_the_lexicographic_order_part_group_id(n, M, groups):
    rng = np.random.default_rng(n)
    group = (rng.integers(0, groups, size=n).astype(np.int64) * 2_654_435 - 900_000_000).astype(np.int32)  # sparse, some negative
    part_id, part_offsets, perm, local_id = oracle.partition(n, group, 77, M, grouped=True)
    assert np.array_equal(part_id, oracle.assign(n, group, 77, M))
    # numpy's lexsort (last key is the primary one) is the independent statement of the order
    expect = np.lexsort((np.arange(n), group, part_id)).astype(np.int32)
    assert np.array_equal(perm, expect)
    assert np.array_equal(np.diff(part_offsets), np.bincount(part_id, minlength=M))
    assert np.array_equal(perm[part_offsets[part_id] + local_id], np.arange(n))
    # every super-node is one contiguous run of rows
    g_in_order = group[perm]
    runs = 1 + np.count_nonzero(np.diff(g_in_order) != 0) if n > 1 else 1
    assert runs == np.unique(group).size


def test_grouped_relabel_with_identity_groups_is_the_plain_relabel():
    n, M = 20_000, 16
    ident = np.arange(n, dtype=np.int32)
    a = oracle.partition(n, ident, 5, M, grouped=True)
    b = oracle.partition(n, None, 5, M)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_grouped_order_leaves_the_induced_subgraphs_isomorphic(tiny_workload):
    # the order of the rows inside a part is a relabelling: same kept / cut counts, same degree multiset,
    # same set of kept edges in global ids
    g = tiny_workload.graph
    rng = np.random.default_rng(3)
    group = rng.integers(0, 40, size=g.n).astype(np.int32)
    M = 4
    res = {}
    for grouped in (False, True):
        part_id, part_offsets, perm, local_id = oracle.partition(g.n, group, 11, M, grouped=grouped)
        rowptr_out, col_out, edge_offsets, kept, cut = oracle.induced_csr(g.rowptr, g.col, M, part_id, part_offsets, perm, local_id)
        edges = set()
        for p in range(M):
            rp, cp = oracle.part_graph(rowptr_out, col_out, part_offsets, edge_offsets, p)
            base = int(part_offsets[p])
            for i in range(rp.size - 1):
                for e in range(int(rp[i]), int(rp[i + 1])):
                    edges.add((int(perm[base + i]), int(perm[base + int(cp[e])])))
        res[grouped] = (kept, cut, edges)
    assert res[False] == res[True]


def test_supernodes_stay_whole_and_identity_groups_reproduce_node_scheme():
    n, M, seed = 30_000, 16, 1234
    rng = np.random.default_rng(0)
    group = rng.integers(0, 300, size=n).astype(np.int32) * 7 + 5   # sparse, non-contiguous ids
    part_id = oracle.assign(n, group, seed, M)
    for g in np.unique(group)[:50]:
        assert np.unique(part_id[group == g]).size == 1
    # same cluster id -> same part as a node with that id under the node scheme (N = |V| limit)
    node_scheme = oracle.assign(int(group.max()) + 1, None, seed, M)
    assert np.array_equal(part_id, node_scheme[group])
    ident = np.arange(n, dtype=np.int32)
    assert np.array_equal(oracle.assign(n, ident, seed, M), oracle.assign(n, None, seed, M))


def test_single_cluster_gives_one_part_and_keeps_every_edge(tiny_workload):
    g = tiny_workload.graph
    group = np.full(g.n, 17, dtype=np.int32)
    part_id, part_offsets, perm, local_id = oracle.partition(g.n, group, 5, 4)
    assert np.count_nonzero(np.diff(part_offsets)) == 1
    _, col_out, _, kept, cut = oracle.induced_csr(g.rowptr, g.col, 4, part_id, part_offsets, perm, local_id)
    assert kept == g.num_entries and cut == 0
    assert np.array_equal(col_out, g.col)        # identity relabel inside the only part


def test_induced_csr_brute_force_with_sets(tiny_workload):
    g, M = tiny_workload.graph, tiny_workload.M
    part_id, part_offsets, perm, local_id = oracle.partition(g.n, None, tiny_workload.partition_seed, M)
    rowptr_out, col_out, edge_offsets, kept, cut = oracle.induced_csr(
        g.rowptr, g.col, M, part_id, part_offsets, perm, local_id)
    src = np.repeat(np.arange(g.n), np.diff(g.rowptr))
    want = {(int(u), int(v)) for u, v in zip(src, g.col) if part_id[u] == part_id[v]}
    got = set()
    for p in range(M):
        rp, cp = oracle.part_graph(rowptr_out, col_out, part_offsets, edge_offsets, p)
        n_p = rp.size - 1
        assert rp[0] == 0 and rp[-1] == cp.size
        assert cp.size == 0 or (cp.min() >= 0 and cp.max() < n_p)
        glob = perm[part_offsets[p]:part_offsets[p + 1]]
        rows = np.repeat(np.arange(n_p), np.diff(rp))
        for i, j in zip(rows, cp):
            got.add((int(glob[i]), int(glob[j])))
        for i in range(n_p):                      # sorted input columns stay sorted
            assert np.all(np.diff(cp[rp[i]:rp[i + 1]]) > 0)
    assert got == want
    assert kept == len(want) and kept + cut == g.num_entries
    # undirected input -> undirected output
    assert all((v, u) in got for (u, v) in got)


def test_induced_csr_single_trainer_is_the_input(tiny_workload):
    g = tiny_workload.graph
    part_id, part_offsets, perm, local_id = oracle.partition(g.n, None, 1, 1)
    rowptr_out, col_out, edge_offsets, kept, cut = oracle.induced_csr(
        g.rowptr, g.col, 1, part_id, part_offsets, perm, local_id)
    assert np.array_equal(rowptr_out, g.rowptr) and np.array_equal(col_out, g.col)
    assert (kept, cut) == (g.num_entries, 0)


def test_directed_entries_self_loops_and_duplicates():
    # rows: 0:[0,1,1,2] 1:[] 2:[0] 3:[3]   (self loops kept, duplicates kept as given)
    rowptr = np.array([0, 4, 4, 5, 6])
    col = np.array([0, 1, 1, 2, 0, 3], dtype=np.int32)
    part_id = np.array([0, 0, 1, 1], dtype=np.int32)
    part_offsets, perm, local_id = oracle.relabel(part_id, 2)
    rowptr_out, col_out, edge_offsets, kept, cut = oracle.induced_csr(
        rowptr, col, 2, part_id, part_offsets, perm, local_id)
    assert rowptr_out.tolist() == [0, 3, 3, 0, 0, 1]
    assert col_out.tolist() == [0, 1, 1, 1]
    assert edge_offsets.tolist() == [0, 3, 4] and (kept, cut) == (4, 2)


def test_kept_fraction_matches_the_ratios_the_paper_prints():
    g = inputs.chung_lu_graph(60_000, 30.0, 2.1, 77)
    E = g.num_entries
    for M_str, r_str in _golden_lines("kept_ratio_random.txt"):
        M, r = int(M_str), float(r_str)
        part_id, part_offsets, perm, local_id = oracle.partition(g.n, None, 4242 + M, M)
        *_, kept, cut = oracle.induced_csr(g.rowptr, g.col, M, part_id, part_offsets, perm, local_id)
        frac = kept / E
        assert kept + cut == E
        assert round(frac, 2) == pytest.approx(r, abs=0.0051)
        # closed form 1/M; hubs inflate the variance, 4 generous sigmas
        sd = np.sqrt((1 / M) * (1 - 1 / M) / (E / 2)) * 6
        assert abs(frac - 1 / M) < 4 * sd


def test_kept_fraction_supernodes_closed_form():
    g = inputs.planted_community_graph(600, 100, 20.0, 10.0, 2.1, 5)
    src = np.repeat(np.arange(g.n), np.diff(g.rowptr))
    intra = int(np.count_nonzero(g.group_id[src] == g.group_id[g.col]))
    inter = g.num_entries - intra
    prev = 1.0
    for M in (2, 4, 8, 16):
        part_id, part_offsets, perm, local_id = oracle.partition(g.n, g.group_id, 31 + M, M)
        *_, kept, cut = oracle.induced_csr(g.rowptr, g.col, M, part_id, part_offsets, perm, local_id)
        frac = kept / g.num_entries
        want = (intra + inter / M) / g.num_entries   # intra edges always kept, inter with prob 1/M
        assert abs(frac - want) < 0.03
        assert frac > 2.0 / M or M == 2              # far above the node-level 1/M (Table 5)
        assert frac < prev + 0.02                    # decreasing in M
        prev = frac


@pytest.mark.parametrize("beta", [0.5, 0.7, 1.0])
@pytest.mark.parametrize("h", [0.6, 0.9])
def test_expected_edge_cut_follows_lemma_1(beta, h):
    # Lemma 1: lambda = (1 - 2(1-beta)beta - (2beta-1)^2 h) eta^2 / C, and the expected
    # number of edges over all pairs is eta^2 / C, so the cut fraction is the bracket.
    n = 40_000
    g, y = inputs.two_class_block_graph(n, 20.0, h, 11)
    rng = np.random.default_rng(3)
    part_id = np.empty(n, dtype=np.int32)
    for cls in (0, 1):
        idx = rng.permutation(np.flatnonzero(y == cls))
        k = int(round(beta * idx.size))
        part_id[idx[:k]] = cls          # partition 0 holds a beta share of class 0 ...
        part_id[idx[k:]] = 1 - cls      # ... partition 1 a beta share of class 1
    part_offsets, perm, local_id = oracle.relabel(part_id, 2)
    *_, kept, cut = oracle.induced_csr(g.rowptr, g.col, 2, part_id, part_offsets, perm, local_id)
    want = 1 - 2 * (1 - beta) * beta - (2 * beta - 1) ** 2 * h
    assert abs(cut / g.num_entries - want) < 0.01


def test_gather_rows_is_fancy_indexing():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((100, 7)).astype(np.float32)
    perm = rng.permutation(100).astype(np.int32)
    assert np.array_equal(oracle.gather_rows(X, perm), X[perm])
