"""GPU parity of the neighbour sampler (Sec. 4.1 "Mini-batch and Negative Sampling") against the oracle:
blocks and frontiers of every hop bit for bit, on parts of the Tiny and (scaled) Medium workloads --
hub rows of several hundred entries, isolated nodes, fan-outs below and above the degrees."""
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


def _part(got, want, p):
    """Part p's subgraph as device views of the library's arrays and as the oracle's arrays."""
    lo, hi = got["part_host"][p], got["part_host"][p + 1]
    e0, e1 = got["edge_host"][p], got["edge_host"][p + 1]
    d_rp = got["rowptr_out"][lo + p: hi + p + 1].contiguous()
    d_col = got["col_out"][e0:e1].contiguous()
    rp, cp = oracle.part_graph(want["rowptr_out"], want["col_out"], want["part_offsets"], want["edge_offsets"], p)
    return d_rp, d_col, rp, cp


@pytest.mark.parametrize("which", ["tiny", "medium"])
def test_sampled_blocks_match_the_oracle(util, which):
    w = inputs.tiny() if which == "tiny" else inputs.medium(0.06)
    got = util.gpu_preprocess(w)
    want = util.oracle_preprocess(w)
    c = util.ctx()
    rng = np.random.default_rng(5)
    for p in (0, got["M"] - 1):
        d_rp, d_col, rp, cp = _part(got, want, p)
        n_p = rp.size - 1
        assert np.array_equal(d_rp.cpu().numpy(), rp) and np.array_equal(d_col.cpu().numpy(), cp)
        deg = np.diff(rp)
        seeds = np.unique(np.concatenate([rng.choice(n_p, size=min(n_p, 64), replace=False), [int(np.argmax(deg))]])).astype(np.int32)
        for fanouts, seed in (((5, 3), 11), ((1, 1, 1), 12), ((int(deg.max()) + 1, 2), 13), ((10, 10, 10), 2**63 + 5)):
            frontier = seeds
            for hop, f in enumerate(fanouts):
                brp, bcol, nxt = c.sample_hop(d_rp, d_col, util.dev(frontier), f, seed, hop)
                o_brp, o_bcol, o_nxt = oracle.sample_hop(rp, cp, frontier, f, seed, hop)
                assert np.array_equal(brp.cpu().numpy(), o_brp), (p, fanouts, hop)
                assert np.array_equal(bcol.cpu().numpy(), o_bcol), (p, fanouts, hop)
                assert np.array_equal(nxt.cpu().numpy(), o_nxt), (p, fanouts, hop)
                frontier = o_nxt
        # the whole part as the frontier (every hub, every isolated node), and the empty one
        allv = np.arange(n_p, dtype=np.int32)
        brp, bcol, nxt = c.sample_hop(d_rp, d_col, util.dev(allv), 4, 99, 0)
        o_brp, o_bcol, o_nxt = oracle.sample_hop(rp, cp, allv, 4, 99, 0)
        assert np.array_equal(brp.cpu().numpy(), o_brp) and np.array_equal(bcol.cpu().numpy(), o_bcol)
        assert np.array_equal(nxt.cpu().numpy(), allv)
        again = c.sample_hop(d_rp, d_col, util.dev(allv), 4, 99, 0)
        assert torch.equal(again[1], bcol)                                   # the same from run to run
        e = c.sample_hop(d_rp, d_col, torch.empty(0, dtype=torch.int32, device="cuda"), 4, 99, 0)
        assert e[0].cpu().tolist() == [0] and e[1].numel() == 0 and e[2].numel() == 0
    c.check()
