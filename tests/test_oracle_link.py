"""Pins for the oracle's link-prediction path (Sec. 4.1 "Link Prediction Decoder" and App.
"Formulation of MLP Decoder"): Hadamard-product MLP decoder with PReLU on top of any encoder
variant, binary cross-entropy on given positive / negative pairs.

Expected values: the encoder output of the already pinned variant routine, numpy closed forms for
the one-layer decoder, central finite differences, and identities of the loss."""
import numpy as np
import pytest

import oracle
from paper_2305_09887_b200 import inputs


def _case(seed=0, n=50, m=120, F=6, B=40):
    g = inputs.uniform_graph(n, m, seed + 1)
    X = inputs.normal_features(n, F, seed + 2).astype(np.float64)
    rng = np.random.default_rng(seed + 3)
    pu = rng.integers(0, n, size=B).astype(np.int32)
    pv = rng.integers(0, n, size=B).astype(np.int32)
    label = (np.arange(B) % 2).astype(np.int32)
    return g.rowptr.astype(np.int64), g.col, X, pu, pv, label


def test_embeddings_are_the_encoder_output():
    rp, cp, X, pu, pv, label = _case()
    for variant in [(0, 0, 0), (1, 1, 1), (0, 1, 1)]:
        dims, ddims = (6, 5, 4), (4, 3, 1)
        p = oracle.link_init_params(variant, dims, ddims, 3)
        _, _, emb, _ = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, p, want_grads=False)
        enc = p[:oracle.variant_param_count(variant, dims)]
        y = np.zeros(rp.size - 1, dtype=np.int32)
        acts = oracle.forward_backward_variant(variant, dims, rp, cp, X, y, enc, want_grads=False, want_acts=True)[2]
        assert np.abs(emb - acts["H2"]).max() < 1e-13


def test_one_layer_decoder_closed_form():
    rp, cp, X, pu, pv, label = _case(4)
    variant, dims, ddims = (1, 0, 0), (6, 5), (5, 1)
    p = oracle.link_init_params(variant, dims, ddims, 5)
    loss, grads, emb, scores = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, p)
    theta_off, _ = oracle.link_decoder_layout(variant, dims, ddims)[0]
    theta = p[theta_off:theta_off + 5]
    E0 = emb[pu] * emb[pv]
    s = E0 @ theta
    assert np.abs(scores - s).max() < 1e-13
    prob = 1 / (1 + np.exp(-s))
    want = -(label * np.log(prob) + (1 - label) * np.log(1 - prob)).mean()
    assert abs(loss - want) < 1e-12
    assert np.abs(grads[theta_off:theta_off + 5] - E0.T @ ((prob - label) / label.size)).max() < 1e-13


@pytest.mark.parametrize("variant", [(0, 0, 0), (1, 1, 1), (0, 1, 1), (1, 0, 1)])
@pytest.mark.parametrize("ddims", [(4, 1), (4, 3, 1), (4, 5, 3, 1)])
def test_link_gradients_match_central_finite_differences(variant, ddims):
    rp, cp, X, pu, pv, label = _case(7)
    dims = (6, 5, 4)
    rng = np.random.default_rng(8)
    p = oracle.link_init_params(variant, dims, ddims, 9)
    p += 0.05 * rng.standard_normal(p.size)
    loss, grads, _, _ = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, p)
    eps = 1e-6
    idx = rng.choice(p.size, size=min(70, p.size), replace=False)
    for theta, slope in oracle.link_decoder_layout(variant, dims, ddims):
        idx = np.append(idx, [theta] + ([slope] if slope >= 0 else []))
    bad = 0
    for i in idx:
        q = p.copy()
        q[i] += eps
        up = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, q, want_grads=False)[0]
        q[i] -= 2 * eps
        dn = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, q, want_grads=False)[0]
        fd = (up - dn) / (2 * eps)
        if abs(fd - grads[i]) > 2e-7 + 1e-5 * abs(fd):
            bad += 1                      # a unit crossing its kink inside the difference stencil
    assert bad <= 1


def test_loss_identities():
    rp, cp, X, pu, pv, label = _case(11)
    variant, dims, ddims = (1, 1, 1), (6, 5, 4), (4, 3, 1)
    p = oracle.link_init_params(variant, dims, ddims, 12)
    # zero decoder weights: every score is 0, every probability 1/2
    q = p.copy()
    for theta, _ in oracle.link_decoder_layout(variant, dims, ddims):
        q[theta:] = 0.0
        break
    loss0, _, _, s0 = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, q, want_grads=False)
    assert np.all(s0 == 0) and abs(loss0 - np.log(2.0)) < 1e-15
    # the decoder input r_u (.) r_v is symmetric in (u, v)
    a = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, p)
    b = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pv, pu, label, p)
    assert a[0] == b[0] and np.abs(a[1] - b[1]).max() < 1e-15
    # huge scores stay finite: loss -> |s| for the wrong label, 0 for the right one
    big = p.copy()
    theta_last, _ = oracle.link_decoder_layout(variant, dims, ddims)[-1]
    big[theta_last:theta_last + 3] *= 1e6
    lb, gb, _, sb = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, big)
    assert np.isfinite(lb) and np.all(np.isfinite(gb)) and np.abs(sb).max() > 1e3
    # an empty batch and an empty part cost nothing
    e = np.empty(0, dtype=np.int32)
    assert oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, e, e, e, p)[0] == 0.0


def test_branch_override_reproduces_the_natural_branches_and_moves_only_chosen_units():
    rp, cp, X, pu, pv, label = _case(13)
    variant, dims, ddims = (1, 1, 1), (6, 5, 4), (4, 3, 1)
    p = oracle.link_init_params(variant, dims, ddims, 14)
    n, B = rp.size - 1, pu.size
    pre = np.zeros(oracle.link_gate_count(dims, ddims, n, B))
    assert pre.size == n * 5 + B * 3
    base = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, p, preact_out=pre)
    natural = (pre > 0).astype(np.int8)
    same = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, p, gates=natural)
    assert same[0] == base[0] and np.array_equal(same[1], base[1])
    free = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, p, gates=np.full(pre.size, -1, np.int8))
    assert free[0] == base[0] and np.array_equal(free[1], base[1])
    # flipping the unit closest to its kink changes the loss by O(|input|) only
    i = int(np.argmin(np.abs(pre)))
    g = natural.copy()
    g[i] ^= 1
    moved = oracle.link_forward_backward(variant, dims, ddims, rp, cp, X, pu, pv, label, p, gates=g)
    assert moved[0] != base[0] and abs(moved[0] - base[0]) <= 2.0 * abs(pre[i])
