"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

import oracle
from paper_2305_09887_b200 import binding

_ctx = None


def ctx():
    global _ctx
    if _ctx is None:
        _ctx = binding.Context(0)
    return _ctx


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def rel_err(a, b):
    """max|a-b| / max|b|  (the tolerance convention of the parity bars)."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.abs(a - b).max() / max(np.abs(b).max(), 1e-30)) if b.size else 0.0


def gpu_preprocess(w, M=None, seed=None, use_groups=None):
    """partition + induced CSR + row gather on the GPU for workload w."""
    c = ctx()
    g = w.graph
    M = w.M if M is None else M
    seed = w.partition_seed if seed is None else seed
    use_groups = w.use_groups if use_groups is None else use_groups
    gid = dev(g.group_id) if use_groups else None
    part_id, part_offsets, perm, local_id = c.partition(g.n, gid, seed, M)
    rowptr_out, col_out, edge_offsets, kept_cut, edge_host = c.build_induced_csr(
        dev(g.rowptr), dev(g.col), M, part_id, part_offsets, perm, local_id)
    Xp = c.gather_rows(dev(w.X), perm)
    yp = c.gather_rows(dev(w.y), perm)
    torch.cuda.synchronize()
    return dict(part_id=part_id, part_offsets=part_offsets, perm=perm, local_id=local_id,
                rowptr_out=rowptr_out, col_out=col_out, edge_offsets=edge_offsets, kept_cut=kept_cut,
                edge_host=edge_host, part_host=part_offsets.cpu().tolist(), Xp=Xp, yp=yp, M=M)


def oracle_preprocess(w, M=None, seed=None, use_groups=None):
    g = w.graph
    M = w.M if M is None else M
    seed = w.partition_seed if seed is None else seed
    use_groups = w.use_groups if use_groups is None else use_groups
    gid = g.group_id if use_groups else None
    part_id, part_offsets, perm, local_id = oracle.partition(g.n, gid, seed, M)
    rowptr_out, col_out, edge_offsets, kept, cut = oracle.induced_csr(
        g.rowptr, g.col, M, part_id, part_offsets, perm, local_id)
    return dict(part_id=part_id, part_offsets=part_offsets, perm=perm, local_id=local_id,
                rowptr_out=rowptr_out, col_out=col_out, edge_offsets=edge_offsets, kept=kept, cut=cut,
                Xp=oracle.gather_rows(w.X, perm), yp=oracle.gather_rows(w.y, perm), M=M)


def assert_preprocess_equal(got, want):
    for k in ("part_id", "part_offsets", "perm", "local_id", "rowptr_out", "col_out", "edge_offsets"):
        a = got[k].cpu().numpy()
        assert a.dtype == want[k].dtype, k
        assert np.array_equal(a, want[k]), k
    kc = got["kept_cut"].cpu().tolist()
    assert kc == [want["kept"], want["cut"]]
    assert np.array_equal(got["Xp"].cpu().numpy(), want["Xp"])
    assert np.array_equal(got["yp"].cpu().numpy(), want["yp"])
