"""GPU parity, integer half: partition ids, relabels and induced CSR arrays must be
bit-identical to the oracle's on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2305_09887_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def util():
    import gpu_util
    return gpu_util


@pytest.mark.parametrize("n,M", [(1, 1), (7, 3), (1000, 64), (1024, 5), (1025, 5), (8192, 32), (8193, 23),
                                 (100_003, 4), (1_000_000, 32)])
def test_partition_matches_oracle(util, n, M):
    seed = 0x5EED0005 + n
    got = util.ctx().partition(n, None, seed, M)
    want = oracle.partition(n, None, seed, M)
    for a, b in zip(got, want):
        assert np.array_equal(a.cpu().numpy(), b)


def test_partition_empty_and_supernodes(util):
    part_id, part_offsets, perm, local_id = util.ctx().partition(0, None, 1, 4)
    assert part_offsets.cpu().tolist() == [0] * 5 and part_id.numel() == 0
    n, M, seed = 250_000, 16, 99
    group = (np.random.default_rng(0).integers(0, 2500, size=n) * 11 - 7).astype(np.int32)  # sparse, some negative
    got = util.ctx().partition(n, util.dev(group), seed, M)
    want = oracle.partition(n, group, seed, M)
    for a, b in zip(got, want):
        assert np.array_equal(a.cpu().numpy(), b)


@pytest.mark.parametrize("n,M,groups", [(1, 1, 1), (7, 3, 2), (1024, 5, 9), (1025, 64, 300), (250_000, 16, 2500),
                                        (1_000_003, 32, 10_000)])
def test_grouped_partition_matches_oracle(util, n, M, groups):
    seed = 0x5EED0005 + n
    rng = np.random.default_rng(n)
    group = (rng.integers(0, groups, size=n).astype(np.int64) * 2_654_435 - 900_000_000).astype(np.int32)  # sparse, some negative
    got = util.ctx().partition(n, util.dev(group), seed, M, grouped=True)
    want = oracle.partition(n, group, seed, M, grouped=True)
    for a, b in zip(got, want):
        assert np.array_equal(a.cpu().numpy(), b)


def test_grouped_partition_without_groups_and_empty(util):
    a = util.ctx().partition(5000, None, 3, 8, grouped=True)
    b = util.ctx().partition(5000, None, 3, 8)
    assert all(torch.equal(x, y) for x, y in zip(a, b))
    part_id, part_offsets, perm, local_id = util.ctx().partition(0, util.dev(np.zeros(0, dtype=np.int32)), 1, 4, grouped=True)
    assert part_offsets.cpu().tolist() == [0] * 5


def test_induced_csr_supernodes_grouped_order(util):
    w = inputs.supertma(0.02)
    got = util.gpu_preprocess(w, grouped=True)
    want = util.oracle_preprocess(w, grouped=True)
    util.assert_preprocess_equal(got, want)
    plain = util.oracle_preprocess(w)
    assert want["kept"] == plain["kept"] and want["cut"] == plain["cut"]


def test_partition_is_deterministic(util):
    a = util.ctx().partition(300_000, None, 5, 8)
    b = util.ctx().partition(300_000, None, 5, 8)
    assert all(torch.equal(x, y) for x, y in zip(a, b))


@pytest.mark.parametrize("M", [1, 4, 23])
def test_induced_csr_tiny(util, tiny_workload, M):
    util.assert_preprocess_equal(util.gpu_preprocess(tiny_workload, M=M), util.oracle_preprocess(tiny_workload, M=M))


def test_induced_csr_power_law_int64_rowptr(util):
    w = inputs.medium(0.25)
    w.graph.rowptr = w.graph.rowptr.astype(np.int64)
    got = util.gpu_preprocess(w, M=8)
    want = util.oracle_preprocess(w, M=8)
    util.assert_preprocess_equal(got, want)
    assert abs(want["kept"] / w.graph.num_entries - 1 / 8) < 0.01     # Sec. 3.2.2: kept fraction 1/M


def test_induced_csr_supernodes(util):
    w = inputs.supertma(0.02)
    got = util.gpu_preprocess(w)
    want = util.oracle_preprocess(w)
    util.assert_preprocess_equal(got, want)
    assert want["kept"] / w.graph.num_entries > 0.6                   # most edges live inside super-nodes


def test_induced_csr_fill_with_and_without_the_count_phase_s_bits(util):
    # COUNT leaves one bit per entry for the FILL that follows on the same arrays; a FILL after some other COUNT
    # must not use them and looks every entry's part up again.  Rows that start and end inside a 32-entry word
    # of the bit buffer (degrees 0..70), int32 and int64 offsets: the same col_out either way, equal to the oracle's.
    import ctypes
    import torch
    from paper_2305_09887_b200 import binding
    c = util.ctx()
    for wide in (False, True):
        w = inputs.medium(0.1)
        if wide:
            w.graph.rowptr = w.graph.rowptr.astype(np.int64)
        M = 5
        got = util.gpu_preprocess(w, M=M)                       # COUNT, then FILL from its bits
        want = util.oracle_preprocess(w, M=M)
        util.assert_preprocess_equal(got, want)
        other = util.gpu_preprocess(inputs.tiny(), M=3)          # a COUNT (and FILL) on other arrays in between
        g = w.graph
        rowptr, col = util.dev(g.rowptr), util.dev(g.col)
        again = torch.full_like(got["col_out"], -1)
        st = c._lib.rtma_build_induced_csr(
            c._h, ctypes.c_int64(g.n), ctypes.c_int32(1 if wide else 0), binding._ptr(rowptr), binding._ptr(col),
            ctypes.c_int32(M), binding._ptr(got["part_id"]), binding._ptr(got["part_offsets"]), binding._ptr(got["perm"]),
            binding._ptr(got["local_id"]), binding._ptr(got["rowptr_out"]), binding._ptr(again),
            binding._ptr(got["edge_offsets"]), binding._ptr(got["kept_cut"]), ctypes.c_void_p(0))
        assert st == 0
        torch.cuda.synchronize()
        assert torch.equal(again, got["col_out"]) and other["col_out"].numel() > 0


def test_induced_csr_degenerate_graphs(util):
    c = util.ctx()
    # no edges at all
    n, M = 100, 4
    rowptr = np.zeros(n + 1, dtype=np.int32)
    col = np.zeros(0, dtype=np.int32)
    p = c.partition(n, None, 3, M)
    rowptr_out, col_out, edge_offsets, kept_cut, edge_host = c.build_induced_csr(
        util.dev(rowptr), torch.empty(0, dtype=torch.int32, device="cuda"), M, *p)
    assert edge_host == [0] * (M + 1) and kept_cut.cpu().tolist() == [0, 0]
    assert rowptr_out.cpu().abs().sum().item() == 0
    # one hub row much longer than a warp, directed entries, self loop, duplicates
    rowptr = np.array([0, 1000, 1001, 1001, 1003], dtype=np.int64)
    col = np.concatenate([np.arange(1000) % 4, [1], [3, 3]]).astype(np.int32)
    part_id = oracle.assign(4, None, 11, 2)
    po, perm, lid = oracle.relabel(part_id, 2)
    want = oracle.induced_csr(rowptr, col, 2, part_id, po, perm, lid)
    gp = c.partition(4, None, 11, 2)
    got = c.build_induced_csr(util.dev(rowptr), util.dev(col), 2, *gp)
    assert np.array_equal(got[0].cpu().numpy(), want[0]) and np.array_equal(got[1].cpu().numpy(), want[1])
    assert got[3].cpu().tolist() == [want[3], want[4]]


@pytest.mark.parametrize("shape,dtype", [((1000, 100), np.float32), ((1000,), np.int32), ((333, 3), np.uint8),
                                         ((257, 129), np.float32)])
def test_gather_rows(util, shape, dtype):
    rng = np.random.default_rng(0)
    src = (rng.standard_normal(shape) * 100).astype(dtype)
    perm = rng.permutation(shape[0]).astype(np.int32)
    got = util.ctx().gather_rows(util.dev(src), util.dev(perm)).cpu().numpy()
    assert np.array_equal(got, src[perm])
