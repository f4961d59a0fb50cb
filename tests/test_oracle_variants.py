"""Pins for the oracle's model variants (Sec. 4.1 "GNN Encoders"): GCN or GraphSAGE-mean layers,
PReLU, Layer Normalization before the activation.

Expected values come from dense numpy algebra (the renormalised adjacency written as a matrix),
central finite differences, special cases that reduce to a known model, and the invariances that
define layer normalisation — never from the routine under test.
"""
import itertools

import numpy as np
import pytest

import oracle
from paper_2305_09887_b200 import inputs

VARIANTS = list(itertools.product((0, 1), (0, 1), (0, 1)))   # (encoder, act, norm)


def _small_part(seed=0, n=60, m=150, F=7, C=4):
    g = inputs.uniform_graph(n, m, seed + 1)
    X = inputs.normal_features(n, F, seed + 2).astype(np.float64)
    y = inputs.uniform_labels(n, C, seed + 3)
    return g.rowptr.astype(np.int64), g.col, X, y


def _dense_gcn_adjacency(rp, cp):
    n = rp.size - 1
    A = np.zeros((n, n))
    np.add.at(A, (np.repeat(np.arange(n), np.diff(rp)), cp), 1.0)
    A += np.eye(n)                                    # self loops
    s = 1.0 / np.sqrt(np.diff(rp) + 1.0)              # D~^-1/2 with D~ = degree + 1
    return s[:, None] * A * s[None, :]


def test_gcn_aggregation_is_the_renormalised_adjacency_product():
    rp, cp, X, _ = _small_part()
    assert np.abs(oracle.spmm_gcn(rp, cp, X) - _dense_gcn_adjacency(rp, cp) @ X).max() < 1e-12
    # an isolated node keeps its own features (only the self loop), unlike the mean aggregation
    rp2 = np.array([0, 0, 1, 2])
    cp2 = np.array([2, 1], dtype=np.int32)
    H = np.array([[3.0], [5.0], [7.0]])
    assert np.allclose(oracle.spmm_gcn(rp2, cp2, H), [[3.0], [(5 + 7) / 2], [(5 + 7) / 2]])


def test_sage_relu_variant_is_the_base_model(tiny_workload):
    rp, cp, X, y = _small_part(5, F=6, C=3)
    dims = (6, 5, 4, 3)
    p = inputs.xavier_params(dims, 3).astype(np.float64)
    l0, g0, a0 = oracle.forward_backward(dims, rp, cp, X, y, p, want_acts=True, want_preact=True)
    l1, g1, a1 = oracle.forward_backward_variant((0, 0, 0), dims, rp, cp, X, y, p, want_acts=True, want_preact=True)
    # same model, summed in a different order: equal to rounding
    assert abs(l0 - l1) < 1e-14 and np.abs(g0 - g1).max() < 1e-14
    assert all(np.abs(a0[k] - a1[k]).max() < 1e-13 for k in a0)
    assert oracle.variant_param_count((0, 0, 0), dims) == oracle.param_count(dims)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("dims", [(7, 6, 4), (7, 5, 6, 4)])
def test_variant_gradients_match_central_finite_differences(variant, dims):
    rp, cp, X, y = _small_part(11)
    rng = np.random.default_rng(4)
    p = oracle.variant_init_params(variant, dims, 9)
    p += 0.05 * rng.standard_normal(p.size)           # gamma, beta, slope away from their special values
    loss, grads, named = oracle.forward_backward_variant(variant, dims, rp, cp, X, y, p, want_preact=True)
    # the finite difference is only meaningful where no unit crosses its kink
    margin = min(np.abs(named[k]).min() for k in named if k.startswith("Z"))
    eps = 1e-6
    assert margin > 50 * eps
    idx = rng.choice(p.size, size=min(60, p.size), replace=False)
    layout = oracle.variant_layout(variant, dims)
    for lay in layout:                                 # every kind of parameter is sampled
        for key in ("bias", "gamma", "beta", "slope"):
            if lay[key] >= 0:
                idx = np.append(idx, lay[key])
    for i in idx:
        q = p.copy()
        q[i] += eps
        up = oracle.forward_backward_variant(variant, dims, rp, cp, X, y, q, want_grads=False)[0]
        q[i] -= 2 * eps
        dn = oracle.forward_backward_variant(variant, dims, rp, cp, X, y, q, want_grads=False)[0]
        fd = (up - dn) / (2 * eps)
        assert abs(fd - grads[i]) <= 2e-7 + 1e-5 * abs(fd), (variant, int(i))


def test_one_layer_gcn_is_softmax_regression_on_aggregated_features():
    rp, cp, X, y = _small_part(21, F=5, C=3)
    dims = (5, 3)
    p = oracle.variant_init_params((1, 0, 0), dims, 1)
    p[15:] = np.array([0.1, -0.2, 0.3])
    W, b = p[:15].reshape(5, 3), p[15:]
    F = _dense_gcn_adjacency(rp, cp) @ X
    Z = F @ W + b
    Z -= Z.max(1, keepdims=True)
    logp = Z - np.log(np.exp(Z).sum(1, keepdims=True))
    n = X.shape[0]
    want_loss = -logp[np.arange(n), y].mean()
    D = (np.exp(logp) - np.eye(3)[y]) / n
    loss, grads, _ = oracle.forward_backward_variant((1, 0, 0), dims, rp, cp, X, y, p)
    assert abs(loss - want_loss) < 1e-12
    assert np.abs(grads[:15].reshape(5, 3) - F.T @ D).max() < 1e-12
    assert np.abs(grads[15:] - D.sum(0)).max() < 1e-12


def test_prelu_with_slope_one_makes_the_gcn_linear_and_slope_zero_is_relu():
    rp, cp, X, y = _small_part(31, F=5, C=3)
    dims = (5, 4, 3)
    lay = oracle.variant_layout((1, 1, 0), dims)
    p = oracle.variant_init_params((1, 1, 0), dims, 2)
    p[lay[0]["bias"]:lay[0]["bias"] + 4] = [0.3, -0.1, 0.2, 0.0]
    p[lay[0]["slope"]] = 1.0
    A = _dense_gcn_adjacency(rp, cp)
    W0 = p[lay[0]["w0"]:lay[0]["w0"] + 20].reshape(5, 4)
    W1 = p[lay[1]["w0"]:lay[1]["w0"] + 12].reshape(4, 3)
    want_logits = A @ (A @ X @ W0 + p[lay[0]["bias"]:lay[0]["bias"] + 4]) @ W1 + p[lay[1]["bias"]:lay[1]["bias"] + 3]
    _, _, acts = oracle.forward_backward_variant((1, 1, 0), dims, rp, cp, X, y, p, want_grads=False, want_acts=True)
    assert np.abs(acts["H2"] - want_logits).max() < 1e-12
    # slope 0: the same numbers as the ReLU variant (whose parameter vector lacks the slope)
    p[lay[0]["slope"]] = 0.0
    relu_p = np.delete(p, lay[0]["slope"])
    l_p, g_p, _ = oracle.forward_backward_variant((1, 1, 0), dims, rp, cp, X, y, p)
    l_r, g_r, _ = oracle.forward_backward_variant((1, 0, 0), dims, rp, cp, X, y, relu_p)
    assert l_p == l_r and np.array_equal(np.delete(g_p, lay[0]["slope"]), g_r)


@pytest.mark.parametrize("encoder", [0, 1])
def test_layer_normalisation_statistics_and_invariances(encoder):
    rp, cp, X, y = _small_part(41, n=80, m=200, F=6, C=3)
    dims = (6, 16, 3)
    v = (encoder, 1, 1)
    lay = oracle.variant_layout(v, dims)
    p = oracle.variant_init_params(v, dims, 5)          # gamma = 1, beta = 0
    _, _, named = oracle.forward_backward_variant(v, dims, rp, cp, X, y, p, want_grads=False, want_acts=True,
                                                  want_preact=True)
    U = named["Z1"]
    assert np.abs(U.mean(1)).max() < 1e-12               # every row has mean 0 ...
    assert np.all(U.var(1) < 1.0) and np.abs(U.var(1) - 1.0).max() < 5e-3   # ... and variance var / (var + eps)
    base = named["H2"].copy()
    # adding the same constant to every bias entry of the normalised layer changes nothing
    q = p.copy()
    q[lay[0]["bias"]:lay[0]["bias"] + 16] += 3.0
    shifted = oracle.forward_backward_variant(v, dims, rp, cp, X, y, q, want_grads=False, want_acts=True)[2]["H2"]
    assert np.abs(shifted - base).max() < 1e-10
    # scaling the layer's weights and bias changes the output only through eps
    q = p.copy()
    end = lay[0]["bias"] + 16
    q[:end] *= 7.0
    scaled = oracle.forward_backward_variant(v, dims, rp, cp, X, y, q, want_grads=False, want_acts=True)[2]["H2"]
    assert np.abs(scaled - base).max() < 5e-3
    # gamma and beta act as an affine map of the normalised rows
    q = p.copy()
    q[lay[0]["gamma"]:lay[0]["gamma"] + 16] = 2.0
    q[lay[0]["beta"]:lay[0]["beta"] + 16] = 0.5
    U2 = oracle.forward_backward_variant(v, dims, rp, cp, X, y, q, want_grads=False, want_preact=True)[2]["Z1"]
    assert np.abs(U2 - (2.0 * U + 0.5)).max() < 1e-12


@pytest.mark.parametrize("variant", [(1, 1, 1), (0, 1, 1), (1, 0, 0)])
def test_variant_sgd_step_is_w_minus_lr_times_gradient(variant):
    rp, cp, X, y = _small_part(51)
    dims = (7, 6, 4)
    p = oracle.variant_init_params(variant, dims, 6)
    loss, g, _ = oracle.forward_backward_variant(variant, dims, rp, cp, X, y, p)
    q, losses = oracle.local_steps_variant(variant, dims, 0.05, rp, cp, X, y, p, 1)
    assert losses[0] == loss and np.abs(q - (p - 0.05 * g)).max() < 1e-15
    q2, l2 = oracle.local_steps_variant(variant, dims, 0.05, rp, cp, X, y, p, 3)
    r, _ = oracle.local_steps_variant(variant, dims, 0.05, rp, cp, X, y, q, 2)
    assert np.array_equal(q2, r)
    assert l2[2] < l2[0]                                   # SGD descends on a fixed batch


@pytest.mark.parametrize("variant", VARIANTS)
def test_input_generator_lays_parameters_out_as_the_oracle_reads_them(variant):
    dims = (7, 6, 5, 3)
    p = inputs.variant_params(variant, dims, 3)
    assert p.size == inputs.variant_param_count(variant, dims) == oracle.variant_param_count(variant, dims)
    for l, lay in enumerate(oracle.variant_layout(variant, dims)):
        d_out = dims[l + 1]
        assert np.all(p[lay["bias"]:lay["bias"] + d_out] == 0)
        if lay["gamma"] >= 0:
            assert np.all(p[lay["gamma"]:lay["gamma"] + d_out] == 1) and np.all(p[lay["beta"]:lay["beta"] + d_out] == 0)
        if lay["slope"] >= 0:
            assert p[lay["slope"]] == 0.25
        bound = np.sqrt(6.0 / (dims[l] + d_out))
        w = p[lay["w0"]:lay["bias"]]
        assert np.abs(w).max() <= bound and np.abs(w).max() > 0.5 * bound
