"""Pins for the oracle's floating-point half: aggregation, layers, loss,
gradients, SGD and averaging.

Expected values come from dense brute force, closed forms in the proof of
Theorem 2, central finite differences, the textbook softmax-regression gradient
and algebraic identities, never from the oracle's own routines.
"""
import numpy as np
import pytest

import oracle
from paper_2305_09887_b200 import inputs


def _part(workload, p, dtype=np.float64):
    g = workload.graph
    part_id, part_offsets, perm, local_id = oracle.partition(g.n, None, workload.partition_seed, workload.M)
    rowptr_out, col_out, edge_offsets, _, _ = oracle.induced_csr(
        g.rowptr, g.col, workload.M, part_id, part_offsets, perm, local_id)
    rp, cp = oracle.part_graph(rowptr_out, col_out, part_offsets, edge_offsets, p)
    lo, hi = int(part_offsets[p]), int(part_offsets[p + 1])
    return rp, cp, workload.X[perm[lo:hi]].astype(dtype), workload.y[perm[lo:hi]]


def _dense_mean_adjacency(rp, cp):
    n = rp.size - 1
    A = np.zeros((n, n))
    rows = np.repeat(np.arange(n), np.diff(rp))
    np.add.at(A, (rows, cp), 1.0)
    deg = A.sum(1, keepdims=True)
    return np.divide(A, deg, out=np.zeros_like(A), where=deg > 0)


@pytest.mark.parametrize("p", [0, 3])
def test_spmm_equals_dense_row_normalised_product(tiny_workload, p):
    rp, cp, X, _ = _part(tiny_workload, p)
    want = _dense_mean_adjacency(rp, cp) @ X
    got = oracle.spmm_mean(rp, cp, X)
    assert np.abs(got - want).max() < 1e-12
    got32 = oracle.spmm_mean(rp, cp, X.astype(np.float32))
    assert got32.dtype == np.float32 and np.abs(got32 - want).max() < 1e-6
    empty = np.flatnonzero(np.diff(rp) == 0)
    assert empty.size > 0                        # M=4 on degree 10 leaves isolated local nodes
    assert np.all(got[empty] == 0.0)


def test_spmm_counts_duplicates_and_self_loops_in_the_mean():
    rowptr = np.array([0, 3, 4, 4])
    col = np.array([0, 1, 1, 2], dtype=np.int32)
    H = np.array([[1.0, 2.0], [4.0, 8.0], [10.0, 20.0]])
    got = oracle.spmm_mean(rowptr, col, H)
    assert np.allclose(got, [[3.0, 6.0], [10.0, 20.0], [0.0, 0.0]])


@pytest.mark.parametrize("h", [0.6, 0.8])
def test_mean_aggregation_matches_theorem_2_expectations(h):
    # Eq. (proof-2-exp-agg-central): for a class-1 node, E[(1/d_v) sum x_u] = [(1-h), h]
    n = 60_000
    g, y = inputs.two_class_block_graph(n, 20.0, h, 21)
    X = np.eye(2)[y]
    agg = oracle.spmm_mean(g.rowptr, g.col, X)
    has_nb = np.diff(g.rowptr) > 0
    m1 = agg[(y == 1) & has_nb].mean(0)
    m0 = agg[(y == 0) & has_nb].mean(0)
    assert np.abs(m1 - [1 - h, h]).max() < 0.01
    assert np.abs(m0 - [h, 1 - h]).max() < 0.01

    # Eq. (proof-2-exp-grad-central): w = 0, sigmoid + L2 loss -> E[grad] = -(1/8)[(1-h), h]
    grad = oracle.sigmoid_l2_grad(g.rowptr, g.col, X, y.astype(np.float64), np.zeros(2))
    g1 = grad[(y == 1) & has_nb].mean(0)
    assert np.abs(g1 - (-0.125) * np.array([1 - h, h])).max() < 0.002

    # Corollary: under random node assignment every trainer sees the same expectation.
    M = 2
    part_id, part_offsets, perm, local_id = oracle.partition(n, None, 7, M)
    rowptr_out, col_out, edge_offsets, _, _ = oracle.induced_csr(
        g.rowptr, g.col, M, part_id, part_offsets, perm, local_id)
    for p in range(M):
        rp, cp = oracle.part_graph(rowptr_out, col_out, part_offsets, edge_offsets, p)
        ids = perm[part_offsets[p]:part_offsets[p + 1]]
        local = oracle.spmm_mean(rp, cp, X[ids])
        sel = (y[ids] == 1) & (np.diff(rp) > 0)
        assert np.abs(local[sel].mean(0) - [1 - h, h]).max() < 0.015


@pytest.mark.parametrize("beta", [0.5, 0.8])
def test_local_aggregation_under_class_skew_follows_eq_exp_agg_1(beta):
    # Eq. (proof-2-exp-agg-1): trainer 1 holds a beta share of class 0; for its class-1 nodes
    # E[mean of local neighbours] = [(1-h)beta, h(1-beta)] / ((1-h)beta + h(1-beta)).
    # The per-node ratio is replaced by the ratio of sums (degree-weighted mean) so that the
    # identity holds without a concentration argument.
    h, n = 0.7, 80_000
    g, y = inputs.two_class_block_graph(n, 30.0, h, 5)
    rng = np.random.default_rng(9)
    part_id = np.empty(n, dtype=np.int32)
    for cls in (0, 1):
        idx = rng.permutation(np.flatnonzero(y == cls))
        k = int(round(beta * idx.size))
        part_id[idx[:k]] = cls
        part_id[idx[k:]] = 1 - cls
    part_offsets, perm, local_id = oracle.relabel(part_id, 2)
    rowptr_out, col_out, edge_offsets, _, _ = oracle.induced_csr(
        g.rowptr, g.col, 2, part_id, part_offsets, perm, local_id)
    rp, cp = oracle.part_graph(rowptr_out, col_out, part_offsets, edge_offsets, 0)
    ids = perm[part_offsets[0]:part_offsets[1]]
    X = np.eye(2)[y[ids]]
    local = oracle.spmm_mean(rp, cp, X)
    deg = np.diff(rp).astype(np.float64)
    sel = y[ids] == 1
    got = (local[sel] * deg[sel, None]).sum(0) / deg[sel].sum()
    want = np.array([(1 - h) * beta, h * (1 - beta)]) / ((1 - h) * beta + h * (1 - beta))
    assert np.abs(got - want).max() < 0.01


def test_one_layer_model_is_softmax_regression_on_self_and_mean_features(tiny_workload):
    rp, cp, X, y = _part(tiny_workload, 1)
    n, F, C = X.shape[0], X.shape[1], 8
    dims = (F, C)
    rng = np.random.default_rng(0)
    params = rng.standard_normal(oracle.param_count(dims)) * 0.1
    Ws = params[:F * C].reshape(F, C)
    Wn = params[F * C:2 * F * C].reshape(F, C)
    b = params[2 * F * C:]
    N = _dense_mean_adjacency(rp, cp) @ X
    Z = X @ Ws + N @ Wn + b
    Zs = Z - Z.max(1, keepdims=True)
    logp = Zs - np.log(np.exp(Zs).sum(1, keepdims=True))
    want_loss = -logp[np.arange(n), y].mean()
    D = (np.exp(logp) - np.eye(C)[y]) / n
    want = np.concatenate([(X.T @ D).ravel(), (N.T @ D).ravel(), D.sum(0)])
    loss, grads, acts = oracle.forward_backward(dims, rp, cp, X, y, params, want_acts=True)
    assert abs(loss - want_loss) < 1e-12
    assert np.abs(grads - want).max() < 1e-12
    assert np.abs(acts["N0"] - N).max() < 1e-12 and np.abs(acts["H1"] - Z).max() < 1e-12


@pytest.mark.parametrize("dims", [(64, 64, 8), (64, 16, 24, 8)])
def test_gradients_match_central_finite_differences(tiny_workload, dims):
    rp, cp, X, y = _part(tiny_workload, 2)
    rng = np.random.default_rng(4)
    params = inputs.xavier_params(dims, 3).astype(np.float64)
    params += 0.05 * rng.standard_normal(params.size)       # non-zero biases too
    loss, grads, acts = oracle.forward_backward(dims, rp, cp, X, y, params, want_acts=True)
    eps = 1e-6
    # ReLU kinks: a perturbation of size eps moves pre-activations by far less than 1e-4
    hidden = np.concatenate([acts[f"H{l}"].ravel() for l in range(1, len(dims) - 1)])
    assert np.count_nonzero((hidden > 0) & (hidden < 1e-7)) == 0
    picks = rng.choice(params.size, size=60, replace=False)
    offs = np.cumsum([0] + [2 * dims[l] * dims[l + 1] + dims[l + 1] for l in range(len(dims) - 1)])
    picks = np.concatenate([picks, offs[1:] - 1, offs[:-1]])   # last bias / first weight of each layer
    for j in picks:
        hi, lo = params.copy(), params.copy()
        hi[j] += eps
        lo[j] -= eps
        lp, _, _ = oracle.forward_backward(dims, rp, cp, X, y, hi, want_grads=False)
        lm, _, _ = oracle.forward_backward(dims, rp, cp, X, y, lo, want_grads=False)
        fd = (lp - lm) / (2 * eps)
        assert abs(fd - grads[j]) <= 1e-6 * max(1.0, abs(grads).max()) + 1e-5 * abs(grads[j])


def test_loss_identities(tiny_workload):
    rp, cp, X, y = _part(tiny_workload, 0)
    dims = tiny_workload.dims
    P = oracle.param_count(dims)
    assert P == inputs.param_count(dims) == 9288
    loss0, g0, _ = oracle.forward_backward(dims, rp, cp, X, y, np.zeros(P))
    assert abs(loss0 - np.log(8)) < 1e-12                       # zero weights -> uniform softmax
    params = tiny_workload.params0.astype(np.float64)
    loss, g, _ = oracle.forward_backward(dims, rp, cp, X, y, params)
    assert loss > 0
    assert abs(g[-8:].sum()) < 1e-12                            # rows of softmax - onehot sum to 0
    shifted = params.copy()
    shifted[-8:] += 3.25                                        # same constant on every logit
    loss_s, g_s, _ = oracle.forward_backward(dims, rp, cp, X, y, shifted)
    assert abs(loss_s - loss) < 1e-12 and np.abs(g_s - g).max() < 1e-12


def test_empty_part_and_edgeless_part():
    dims = (4, 3, 2)
    P = oracle.param_count(dims)
    params = inputs.xavier_params(dims, 0).astype(np.float64)
    loss, g, _ = oracle.forward_backward(dims, np.zeros(1, np.int64), np.zeros(0, np.int32),
                                         np.zeros((0, 4)), np.zeros(0, np.int32), params)
    assert loss == 0.0 and np.all(g == 0) and g.size == P
    # no edges: the neighbour weights get zero gradient, the node still trains through W_self
    X = np.random.default_rng(0).standard_normal((5, 4))
    y = np.array([0, 1, 0, 1, 1], dtype=np.int32)
    loss, g, _ = oracle.forward_backward(dims, np.zeros(6, np.int64), np.zeros(0, np.int32), X, y, params)
    assert np.all(g[12:24] == 0) and np.any(g[:12] != 0)


def test_sgd_step_is_w_minus_lr_times_gradient(tiny_workload):
    rp, cp, X, y = _part(tiny_workload, 0)
    dims, lr = tiny_workload.dims, 0.01
    params = tiny_workload.params0.astype(np.float64)
    loss, g, _ = oracle.forward_backward(dims, rp, cp, X, y, params)
    after, losses = oracle.local_steps(dims, lr, rp, cp, X, y, params, 1)
    assert np.abs(after - (params - lr * g)).max() < 1e-15 and abs(losses[0] - loss) < 1e-15
    frozen, _ = oracle.local_steps(dims, 0.0, rp, cp, X, y, params, 3)
    assert np.array_equal(frozen, params)
    none, _ = oracle.local_steps(dims, lr, rp, cp, X, y, params, 0)
    assert np.array_equal(none, params)
    two, _ = oracle.local_steps(dims, lr, rp, cp, X, y, params, 2)
    one_by_one, _ = oracle.local_steps(dims, lr, rp, cp, X, y, after, 1)
    assert np.array_equal(two, one_by_one)


def test_float32_oracle_tracks_float64_oracle(tiny_workload):
    rp, cp, X, y = _part(tiny_workload, 0)
    dims = tiny_workload.dims
    p64, l64 = oracle.local_steps(dims, 0.01, rp, cp, X, y, tiny_workload.params0.astype(np.float64), 5)
    p32, l32 = oracle.local_steps(dims, 0.01, rp, cp, X.astype(np.float32), y, tiny_workload.params0, 5)
    assert p32.dtype == np.float32
    assert np.abs(p32 - p64).max() <= 1e-6 * np.abs(p64).max()
    assert np.abs(l32 - l64).max() < 1e-6


def test_averaging_identities():
    rng = np.random.default_rng(0)
    P = 1000
    one = rng.standard_normal((1, P))
    out, glob = oracle.average(one)
    assert np.array_equal(out, one) and np.array_equal(glob, one[0])       # M = 1
    same = np.tile(rng.standard_normal(P).astype(np.float32), (5, 1))
    out, glob = oracle.average(same)
    assert np.array_equal(out, same)                                       # identical replicas
    const = np.full((7, P), 0.3)
    out, _ = oracle.average(const)
    assert np.allclose(out, 0.3, rtol=0, atol=1e-16)
    W = rng.standard_normal((6, P))
    out, glob = oracle.average(W)
    assert np.abs(glob - W.mean(0)).max() < 1e-15                           # numpy's mean as the library routine
    assert all(np.array_equal(out[i], glob) for i in range(6))              # every copy overwritten


def test_whole_method_on_tiny(tiny_workload):
    w = tiny_workload
    # zero local steps: averaging returns the initial weights on every trainer
    res0 = oracle.run_method(w.graph.rowptr, w.graph.col, w.X, w.y, w.dims, w.M, 0, 1, w.lr,
                             w.partition_seed, w.params0)
    assert np.array_equal(res0["params"], np.tile(w.params0.astype(np.float64), (w.M, 1)))
    # class-shifted features make the loss fall on every trainer, and trainers stay close
    y = w.y
    X = inputs.normal_features(w.graph.n, 64, 1, y, 8, 1.0)
    res = oracle.run_method(w.graph.rowptr, w.graph.col, X, y, w.dims, w.M, 30, 1, 0.1,
                            w.partition_seed, w.params0)
    losses = res["losses"][0]
    assert np.all(losses[:, -1] < losses[:, 0] - 0.05)
    assert np.ptp(losses[:, 0]) < 0.15           # similar initial loss across random parts (Fig. 3)
    assert res["kept"] + res["cut"] == w.graph.num_entries
    for i in range(1, w.M):
        assert np.array_equal(res["params"][i], res["params"][0])


def test_relu_branch_override_only_moves_the_chosen_units(tiny_workload):
    # The override exists for units whose pre-activation is within rounding error of 0, where
    # the ReLU branch is not determined.  Natural gates (-1 everywhere) must reproduce the plain
    # result; forcing one unit's branch must agree with finite differences of the loss in which
    # that unit is replaced by the identity (open) or by zero (closed) -- checked here through
    # the bias gradient of that unit, which is the sum over rows of dL/dZ.
    rp, cp, X, y = _part(tiny_workload, 1)
    dims = tiny_workload.dims
    params = tiny_workload.params0.astype(np.float64)
    loss, g, named = oracle.forward_backward(dims, rp, cp, X, y, params, want_preact=True)
    Z1 = named["Z1"]
    natural = [np.full(Z1.shape, -1, dtype=np.int8)]
    loss_n, g_n, _ = oracle.forward_backward(dims, rp, cp, X, y, params, gates=natural)
    assert loss_n == loss and np.array_equal(g_n, g)
    same = [(Z1 > 0).astype(np.int8)]
    loss_s, g_s, _ = oracle.forward_backward(dims, rp, cp, X, y, params, gates=same)
    assert loss_s == loss and np.array_equal(g_s, g)
    # close the open unit closest to the kink (its value is ~1e-5, so the forward pass barely
    # moves): node v stops contributing to column j of the first layer's gradients, by exactly
    # x_v (and the mean of its neighbours) times dL/dz, and nothing else moves beyond O(z).
    pos = np.where(Z1 > 0, Z1, np.inf)
    v, j = np.unravel_index(np.argmin(pos), pos.shape)
    z = Z1[v, j]
    assert 0 < z < 1e-3
    forced = [np.full(Z1.shape, -1, dtype=np.int8)]
    forced[0][v, j] = 0
    _, g_f, _ = oracle.forward_backward(dims, rp, cp, X, y, params, gates=forced)
    d0, d1 = dims[0], dims[1]
    delta_b = (g - g_f)[2 * d0 * d1: 2 * d0 * d1 + d1]
    dldz = delta_b[j]
    assert abs(dldz) > 1e-7
    assert np.abs(np.delete(delta_b, j)).max() < 50 * z * abs(dldz) + 1e-12
    dWs = (g - g_f)[:d0 * d1].reshape(d0, d1)
    assert np.allclose(dWs[:, j], X[v] * dldz, rtol=0, atol=50 * z * abs(dldz) * np.abs(X[v]).max() + 1e-12)
    dWn = (g - g_f)[d0 * d1:2 * d0 * d1].reshape(d0, d1)
    Nv = (_dense_mean_adjacency(rp, cp) @ X)[v]
    assert np.allclose(dWn[:, j], Nv * dldz, rtol=0, atol=50 * z * abs(dldz) * max(np.abs(Nv).max(), 1e-3) + 1e-12)
