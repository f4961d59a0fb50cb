"""The range-checked build of the library (-DRTMA_BOUNDS, librtma_checked.so): every index a kernel
takes from the caller's data is checked before it addresses memory; an index out of range is recorded,
the access is skipped, and the next rtma_check returns RTMA_ERR_BOUNDS.  It stands in for a memory
checker: on healthy inputs it must give the ordinary build's result bit for bit and report nothing; on
inputs with a bad index it must say which, without touching memory out of range.
"""
import numpy as np
import pytest
import torch

from paper_2305_09887_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _whole_path(c, w):
    g = w.graph
    part_id, part_offsets, perm, local_id = c.partition(g.n, None, w.partition_seed, w.M)
    rowptr_out, col_out, edge_offsets, kept_cut, edge_host = c.build_induced_csr(
        _dev(g.rowptr), _dev(g.col), w.M, part_id, part_offsets, perm, local_id)
    yp = c.gather_rows(_dev(w.y), perm)
    params = _dev(np.tile(w.params0, (w.M, 1)))
    loss = torch.zeros(w.M, w.K, dtype=torch.float32, device="cuda")
    c.local_steps(w.dims, w.lr, w.M, part_offsets.cpu().tolist(), edge_host, rowptr_out, col_out, _dev(w.X), yp, params,
                  w.K, loss_out=loss, perm=perm)
    c.aggregate(params)
    c.check()
    return perm, rowptr_out, col_out, params, loss


def test_checked_build_agrees_with_the_ordinary_one(tiny_workload):
    lib = binding.load_library(checked=True)
    assert lib.rtma_bounds_checked() == 1 and binding.load_library().rtma_bounds_checked() == 0
    for w in (tiny_workload, inputs.medium(0.03)):
        plain = _whole_path(binding.Context(0), w)
        checked = _whole_path(binding.Context(0, checked=True), w)
        for a, b in zip(plain, checked):
            assert torch.equal(a, b)


def test_checked_build_reports_a_column_id_out_of_range(tiny_workload):
    w = tiny_workload
    g = w.graph
    c = binding.Context(0, checked=True)
    part_id, part_offsets, perm, local_id = c.partition(g.n, None, w.partition_seed, w.M)
    col = g.col.copy()
    col[123] = g.n + 5                                   # one entry points past the last node
    with pytest.raises(binding.RtmaError, match="column id of the input graph 2005 outside"):
        c.build_induced_csr(_dev(g.rowptr), _dev(col), w.M, part_id, part_offsets, perm, local_id)
        c.check()
    c.check()                                            # reported once; the context stays usable
    good = c.build_induced_csr(_dev(g.rowptr), _dev(g.col), w.M, part_id, part_offsets, perm, local_id)
    c.check()
    assert int(good[3][0]) + int(good[3][1]) == g.num_entries


def test_checked_build_reports_a_label_out_of_range(tiny_workload):
    w = tiny_workload
    g = w.graph
    c = binding.Context(0, checked=True)
    part_id, part_offsets, perm, local_id = c.partition(g.n, None, w.partition_seed, w.M)
    rowptr_out, col_out, edge_offsets, kept_cut, edge_host = c.build_induced_csr(
        _dev(g.rowptr), _dev(g.col), w.M, part_id, part_offsets, perm, local_id)
    y = w.y.copy()
    y[77] = w.dims[-1]                                   # one class id past the last class
    yp = c.gather_rows(_dev(y), perm)
    params = _dev(np.tile(w.params0, (w.M, 1)))
    c.local_steps(w.dims, w.lr, w.M, part_offsets.cpu().tolist(), edge_host, rowptr_out, col_out, _dev(w.X), yp, params, 1,
                  perm=perm)
    with pytest.raises(binding.RtmaError, match="label 8 outside"):
        c.check()
