"""The aggregation Abar H (Theorem 2) and its transpose taken from dense tiles on the tensor cores:
entries whose column lies in the window around their row's 128-row tile come from an MMA against a
0/1 (or 1/deg-weighted) tile expanded in shared memory from per-row bit masks, the others are summed
into the output rows by a gather pass beforehand.

Forced on for every part (mode 2) the path must reproduce the oracle on graphs it was not made for
(power-law parts where most entries fall outside the window, hubs, isolated nodes, rows narrower and
wider than a column tile; parts with repeated entries, which a bit mask cannot count, must find their
way back to the gather kernels); left to decide for itself (mode 1) it must take the super-node-ordered
parts and leave results independent of streams, waves and of which trainers still run.
"""
import numpy as np
import pytest
import torch

from paper_2305_09887_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def util():
    import gpu_util
    return gpu_util


@pytest.fixture()
def forced(util):
    c = util.ctx()
    c.set_dense_aggregation(2)
    yield c
    c.set_dense_aggregation(1)


def test_forced_tiles_on_power_law_parts(util, forced):
    # Medium x 0.06: 1,500 rows per part (11 full tiles and a ragged one), hubs whose entries mostly lie
    # outside the window, isolated nodes; widths 128, 256 and 47
    w = inputs.medium(0.06)
    got, want = util.check_one_step(w)
    util.check_k_steps_and_average(w, got, want, 2)


def test_forced_tiles_on_super_node_ordered_parts(util, forced):
    w = inputs.supertma(0.02, M=4)
    w.grouped_order = True
    w.dims = (100, 256, 47)
    w.params0 = inputs.xavier_params(w.dims, 6)
    got, want = util.check_one_step(w)
    util.check_k_steps_and_average(w, got, want, 2)


@pytest.mark.parametrize("dims", [(33, 20, 3), (17, 130, 24, 2), (24, 300, 16), (520, 64, 5)])
def test_forced_tiles_odd_widths(util, forced, tiny_workload, dims):
    # widths that are not a multiple of 64 (the last atom is partly padding), more than 256 (two column
    # tiles), exactly 16 (the narrowest the tiles take) and below it (left to the gather kernels)
    w = tiny_workload
    w = inputs.Workload(**{**w.__dict__})
    w.dims = dims
    w.X = inputs.normal_features(w.graph.n, dims[0], 11)
    w.y = (w.y % dims[-1]).astype(np.int32)
    w.params0 = inputs.xavier_params(dims, 12)
    got, want = util.check_one_step(w)
    util.check_k_steps_and_average(w, got, want, 2)


def test_forced_tiles_with_repeated_entries_and_unsorted_rows(util, forced, tiny_workload):
    # a multigraph: some edges occur two or three times (both directions), and every row's entries are
    # shuffled; the mean counts an entry as often as it occurs.  Every part has rows that repeat an entry
    # inside their window, so even when forced the tiles hand these parts back to the gather kernels
    base = inputs.uniform_graph(700, 2800, 21)
    rng = np.random.default_rng(22)
    rp = base.rowptr.astype(np.int64)
    rows = np.repeat(np.arange(base.n), np.diff(rp))
    cols = base.col.astype(np.int64)
    upper = rows < cols
    u, v = rows[upper], cols[upper]
    times = rng.choice([1, 1, 1, 2, 3], size=u.size)
    u, v = np.repeat(u, times), np.repeat(v, times)
    r2, c2 = np.concatenate([u, v]), np.concatenate([v, u])
    order = np.lexsort((rng.random(r2.size), r2))          # by row, random inside a row
    r2, c2 = r2[order], c2[order]
    rowptr = np.zeros(base.n + 1, dtype=np.int32)
    np.cumsum(np.bincount(r2, minlength=base.n), out=rowptr[1:])
    w = inputs.Workload(**{**tiny_workload.__dict__})
    w.graph = inputs.Graph(n=base.n, rowptr=rowptr, col=c2.astype(np.int32))
    w.X, w.y = w.X[:base.n].copy(), w.y[:base.n].copy()
    w.M = 2
    got, want = util.check_one_step(w)
    util.check_k_steps_and_average(w, got, want, 2)


def test_forced_tiles_with_prelu_and_layer_normalization(util, forced):
    # the paper's encoder activation and normalisation (Sec. 4.1) round the GraphSAGE aggregation on the tiles
    import test_gpu_variants as tv
    w = inputs.medium(0.04)
    variant = (0, 1, 1)
    p0 = tv._start(variant, w.dims, 11)
    got, want = util.check_one_step(w, variant=variant, params0=p0)
    util.check_k_steps_and_average(w, got, want, 2, variant=variant, params0=p0)


def test_forced_tiles_in_bf16_operand_mode(util, forced, tiny_workload):
    # the aggregation keeps its fp32 sums when the products take bf16 operands
    w = tiny_workload
    got, want = util.check_one_step(w, gemm_dtype=1)
    util.check_k_steps_and_average(w, got, want, w.K, gemm_dtype=1)


def test_forced_tiles_under_link_prediction(util, forced, tiny_workload):
    # GraphSAGE encoder + PReLU + LayerNorm, MLP decoder on pairs (Sec. 4.1): the encoder's last layer is as
    # wide as the hidden ones there (no head form), all its aggregations go through the tiles
    import test_gpu_link as tl
    tl._check_link(util, tiny_workload, (0, 1, 1), (8, 16, 5, 1), per_part=300, K=3)


def test_one_part_with_a_repeated_entry_gathers_while_the_others_take_the_tiles(util, forced):
    # the same launch then serves both kinds of parts: the gather kernels skip the flagged parts, the tiles
    # the others.  One edge inside one super-node is stored twice (in both directions).
    w = inputs.supertma(0.02, M=4)
    w.grouped_order = True
    w.dims = (100, 64, 47)
    w.params0 = inputs.xavier_params(w.dims, 8)
    g = w.graph
    rp = g.rowptr.astype(np.int64)
    members = np.flatnonzero(g.group_id == g.group_id[0])
    u = v = -1
    for cand in members:   # an edge between two members of that super-node
        row = g.col[rp[cand]:rp[cand + 1]]
        inside = row[np.isin(row, members)]
        if inside.size:
            u, v = int(cand), int(inside[0])
            break
    assert u >= 0
    rows = np.repeat(np.arange(g.n), np.diff(rp))
    rows = np.concatenate([rows, [u, v]])
    cols = np.concatenate([g.col.astype(np.int64), [v, u]])
    order = np.lexsort((cols, rows))
    rowptr = np.zeros(g.n + 1, dtype=g.rowptr.dtype)
    np.cumsum(np.bincount(rows, minlength=g.n), out=rowptr[1:])
    w.graph = inputs.Graph(n=g.n, rowptr=rowptr, col=cols[order].astype(np.int32), group_id=g.group_id)
    got, want = util.check_one_step(w)
    tiles = util.check_k_steps_and_average(w, got, want, 2)
    c = forced
    c.set_dense_aggregation(0)
    gathered = util.check_k_steps_and_average(w, got, want, 2)
    # the part that holds the repeated entry: the same bits either way; the other parts: not
    same = [np.array_equal(tiles[p], gathered[p]) for p in range(w.M)]
    assert sum(same) == 1 and same[int(want["part_id"][u])]


def test_forced_tiles_do_not_depend_on_streams_waves_or_who_else_runs(util, forced, tiny_workload):
    w = tiny_workload
    c = forced
    got = util.gpu_preprocess(w)
    want = util.oracle_preprocess(w)
    one = util.check_k_steps_and_average(w, got, want, 3)
    streams = [torch.cuda.Stream() for _ in range(w.M)]
    torch.cuda.synchronize()
    many = util.check_k_steps_and_average(w, got, want, 3, streams=streams)
    assert np.array_equal(one, many)
    # two waves: a context of its own, its arena capped at a little over half of what one wave takes
    from paper_2305_09887_b200 import binding

    def run(ctx_):
        params = util.dev(np.tile(w.params0, (w.M, 1)))
        ctx_.local_steps(w.dims, w.lr, w.M, got["part_host"], got["edge_host"], got["rowptr_out"], got["col_out"],
                         got["Xp"], got["yp"], params, 3)
        torch.cuda.synchronize()
        ctx_.check()
        return params.cpu().numpy()

    whole = binding.Context(0)
    whole.set_dense_aggregation(2)
    assert np.array_equal(run(whole), one)
    need = whole.workspace_bytes
    whole.close()
    capped = binding.Context(0)
    capped.set_dense_aggregation(2)
    capped.set_workspace_limit(int(need * 0.55))
    waves = run(capped)
    assert capped.workspace_bytes <= int(need * 0.55)
    capped.close()
    assert np.array_equal(one, waves)
    # trainer 0 sees the same arithmetic whether or not the others are still running
    params = util.dev(np.tile(w.params0, (w.M, 1)))
    steps = [3, 1, 0, 2][:w.M]
    c.local_steps(w.dims, w.lr, w.M, got["part_host"], got["edge_host"], got["rowptr_out"], got["col_out"],
                  got["Xp"], got["yp"], params, steps)
    both = util.dev(np.tile(w.params0, (w.M, 1)))
    c.local_steps(w.dims, w.lr, w.M, got["part_host"], got["edge_host"], got["rowptr_out"], got["col_out"],
                  got["Xp"], got["yp"], both, 3)
    torch.cuda.synchronize()
    assert np.array_equal(params.cpu().numpy()[0], both.cpu().numpy()[0])


def test_parts_choose_for_themselves(util):
    # default mode: super-node-ordered parts of degree 20 take the tiles, the same graph partitioned node by
    # node does not (its neighbours are anywhere in the part); both are held to the oracle, and the choice
    # shows in the results: the tile path and the gather path round differently
    c = util.ctx()
    w = inputs.supertma(0.02, M=4)
    w.grouped_order = True
    w.dims = (100, 64, 47)
    w.params0 = inputs.xavier_params(w.dims, 7)
    got = util.gpu_preprocess(w)
    want = util.oracle_preprocess(w)

    def run(mode):
        c.set_dense_aggregation(mode)
        try:
            return util.check_k_steps_and_average(w, got, want, 2)
        finally:
            c.set_dense_aggregation(1)

    auto, never, always = run(1), run(0), run(2)
    assert np.array_equal(auto, always) and not np.array_equal(auto, never)
    w2 = inputs.supertma(0.02, M=4, use_groups=False)
    w2.dims, w2.params0 = w.dims, w.params0
    got2 = util.gpu_preprocess(w2)
    want2 = util.oracle_preprocess(w2)
    w, got, want = w2, got2, want2
    auto, never = run(1), run(0)
    assert np.array_equal(auto, never)
