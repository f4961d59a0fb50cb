"""Pins for the oracle's reduced-precision mode (operands of every dense product rounded to bf16,
everything else unchanged): the rounding itself against hand-worked ties and torch's conversion,
and the whole forward / backward pass against a dense numpy restatement with the adjacency written
as a matrix.
"""
import numpy as np
import torch

import oracle
from paper_2305_09887_b200 import inputs


def _bf16(x):
    """Round to nearest even into the upper 16 bits of binary32, with integer arithmetic on the bits."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


def test_rounding_to_bf16():
    # bf16 keeps 8 significant bits: neighbours of 1 are 2^-7 apart; ties go to the even mantissa
    assert oracle.round_to_bf16(1.0 + 2.0 ** -8) == 1.0                    # tie, 1.0 is even
    assert oracle.round_to_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6    # tie, the upper neighbour is even
    assert oracle.round_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -20) == 1.0 + 2.0 ** -7
    assert oracle.round_to_bf16(-0.3) == -oracle.round_to_bf16(0.3)
    assert oracle.round_to_bf16(0.0) == 0.0
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(2000), rng.standard_normal(2000) * 1e-6, rng.standard_normal(2000) * 1e6])
    got = np.array([oracle.round_to_bf16(float(v)) for v in x])
    lib = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()   # the library's conversion
    assert np.array_equal(got, lib)
    assert np.array_equal(got, _bf16(x))
    assert np.abs(got - x).max() <= 2.0 ** -8 * np.abs(x).max()


def _dense_mean_adjacency(rp, cp):
    n = rp.size - 1
    A = np.zeros((n, n))
    np.add.at(A, (np.repeat(np.arange(n), np.diff(rp)), cp), 1.0)
    deg = np.diff(rp).astype(np.float64)
    return A / np.maximum(deg, 1.0)[:, None]


def _numpy_two_layer(dims, A, X, y, p):
    F, Hd, C = dims
    o = 0
    Ws0 = p[o:o + F * Hd].reshape(F, Hd); o += F * Hd
    Wn0 = p[o:o + F * Hd].reshape(F, Hd); o += F * Hd
    b0 = p[o:o + Hd]; o += Hd
    Ws1 = p[o:o + Hd * C].reshape(Hd, C); o += Hd * C
    Wn1 = p[o:o + Hd * C].reshape(Hd, C); o += Hd * C
    b1 = p[o:o + C]
    r = _bf16
    n = X.shape[0]
    N0 = A @ X
    Z1 = r(X) @ r(Ws0) + r(N0) @ r(Wn0) + b0
    H1 = np.maximum(Z1, 0.0)
    N1 = A @ H1
    Z2 = r(H1) @ r(Ws1) + r(N1) @ r(Wn1) + b1
    zs = Z2 - Z2.max(axis=1, keepdims=True)
    lse = np.log(np.exp(zs).sum(axis=1, keepdims=True))
    loss = float((lse[:, 0] - zs[np.arange(n), y]).mean())
    dZ2 = np.exp(zs - lse)
    dZ2[np.arange(n), y] -= 1.0
    dZ2 /= n
    g = [r(H1).T @ r(dZ2), r(N1).T @ r(dZ2), r(dZ2).sum(axis=0)]
    Q = A.T @ dZ2
    dH1 = r(dZ2) @ r(Ws1).T + r(Q) @ r(Wn1).T
    dZ1 = dH1 * (Z1 > 0)
    g = [r(X).T @ r(dZ1), r(N0).T @ r(dZ1), r(dZ1).sum(axis=0)] + g
    return loss, np.concatenate([a.ravel() for a in g]), Z2


def test_bf16_operand_mode_against_dense_numpy():
    g = inputs.uniform_graph(80, 240, 21)
    rp, cp = g.rowptr.astype(np.int64), g.col
    dims = (9, 7, 5)
    X = inputs.normal_features(80, 9, 22).astype(np.float64)
    y = inputs.uniform_labels(80, 5, 23)
    p = inputs.xavier_params(dims, 24).astype(np.float64)
    p += 0.05 * np.random.default_rng(25).standard_normal(p.size)      # biases away from zero
    A = _dense_mean_adjacency(rp, cp)
    loss, grads, acts = oracle.forward_backward(dims, rp, cp, X, y, p, want_acts=True, bf16_operands=True)
    n_loss, n_grads, n_logits = _numpy_two_layer(dims, A, X, y, p)
    assert abs(loss - n_loss) < 1e-12
    assert np.abs(acts["H2"] - n_logits).max() < 1e-12
    assert np.abs(grads - n_grads).max() < 1e-12 * max(1.0, np.abs(n_grads).max())
    # one layer: softmax regression on [X | A X] with rounded operands (no dgrad product at all)
    dims1 = (9, 5)
    p1 = inputs.xavier_params(dims1, 26).astype(np.float64)
    l1, g1, _ = oracle.forward_backward(dims1, rp, cp, X, y, p1, bf16_operands=True)
    W = np.concatenate([p1[:45].reshape(9, 5), p1[45:90].reshape(9, 5)])
    U = np.concatenate([X, A @ X], axis=1)
    Z = _bf16(U) @ _bf16(W) + p1[90:]
    zs = Z - Z.max(axis=1, keepdims=True)
    P = np.exp(zs) / np.exp(zs).sum(axis=1, keepdims=True)
    assert abs(l1 - float(-np.log(P[np.arange(80), y]).mean())) < 1e-12
    dZ = P.copy()
    dZ[np.arange(80), y] -= 1.0
    dZ /= 80
    want = np.concatenate([(_bf16(U).T @ _bf16(dZ)).ravel(), _bf16(dZ).sum(axis=0)])
    assert np.abs(g1 - want).max() < 1e-13
    # the mode moves the result by about the rounding (2^-9 per operand), no more
    l0, g0, _ = oracle.forward_backward(dims, rp, cp, X, y, p)
    rel = np.abs(grads - g0).max() / np.abs(g0).max()
    assert 1e-5 < rel < 2e-2 and 0 < abs(loss - l0) < 1e-2


def test_bf16_operand_mode_steps():
    g = inputs.uniform_graph(60, 150, 31)
    rp, cp = g.rowptr.astype(np.int64), g.col
    dims = (6, 8, 4)
    X = inputs.normal_features(60, 6, 32).astype(np.float64)
    y = inputs.uniform_labels(60, 4, 33)
    p = inputs.xavier_params(dims, 34).astype(np.float64)
    lr = 0.05
    p2, losses = oracle.local_steps(dims, lr, rp, cp, X, y, p, 2, bf16_operands=True)
    l_a, g_a, _ = oracle.forward_backward(dims, rp, cp, X, y, p, bf16_operands=True)
    l_b, g_b, _ = oracle.forward_backward(dims, rp, cp, X, y, p - lr * g_a, bf16_operands=True)
    assert np.array_equal(p2, (p - lr * g_a) - lr * g_b)     # the parameters themselves stay unrounded
    assert np.array_equal(losses, [l_a, l_b])
