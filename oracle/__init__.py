"""ctypes front end of the CPU oracle (``rtma_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg, never by the product package.  Argument
marshalling only; all arithmetic lives in the C++ file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rtma_oracle.cpp")
_LIB = os.path.join(_HERE, "librtma_oracle.so")
_lib = None

c_i32p = ctypes.POINTER(ctypes.c_int32)
c_i64p = ctypes.POINTER(ctypes.c_int64)
c_f32p = ctypes.POINTER(ctypes.c_float)
c_f64p = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> str:
    """Compile the oracle with g++ -O2 (single-threaded, no CUDA)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_splitmix64.restype = ctypes.c_uint64
        _lib.orc_splitmix64.argtypes = [ctypes.c_uint64]
        _lib.orc_induced_csr.restype = ctypes.c_int64
        _lib.orc_param_count.restype = ctypes.c_int64
        _lib.orc_forward_backward_f32.restype = ctypes.c_double
        _lib.orc_forward_backward_f64.restype = ctypes.c_double
    return _lib


def _p(a, ty):
    return None if a is None else a.ctypes.data_as(ty)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def splitmix64(x: int) -> int:
    return int(lib().orc_splitmix64(ctypes.c_uint64(x & (2**64 - 1))))


def assign(n: int, group_id, seed: int, M: int) -> np.ndarray:
    part_id = np.empty(n, dtype=np.int32)
    g = None if group_id is None else _i32(group_id)
    lib().orc_assign(ctypes.c_int64(n), _p(g, c_i32p), ctypes.c_uint64(seed), ctypes.c_int32(M),
                     _p(part_id, c_i32p))
    return part_id


def relabel(part_id: np.ndarray, M: int):
    n = part_id.size
    part_id = _i32(part_id)
    part_offsets = np.empty(M + 1, dtype=np.int64)
    perm = np.empty(n, dtype=np.int32)
    local_id = np.empty(n, dtype=np.int32)
    lib().orc_relabel(ctypes.c_int64(n), ctypes.c_int32(M), _p(part_id, c_i32p),
                      _p(part_offsets, c_i64p), _p(perm, c_i32p), _p(local_id, c_i32p))
    return part_offsets, perm, local_id


def relabel_grouped(part_id: np.ndarray, group_id: np.ndarray, M: int):
    """Within a part: by super-node id, then by global id."""
    n = part_id.size
    part_id = _i32(part_id)
    group_id = _i32(group_id)
    part_offsets = np.empty(M + 1, dtype=np.int64)
    perm = np.empty(n, dtype=np.int32)
    local_id = np.empty(n, dtype=np.int32)
    lib().orc_relabel_grouped(ctypes.c_int64(n), ctypes.c_int32(M), _p(part_id, c_i32p), _p(group_id, c_i32p),
                              _p(part_offsets, c_i64p), _p(perm, c_i32p), _p(local_id, c_i32p))
    return part_offsets, perm, local_id


def partition(n: int, group_id, seed: int, M: int, grouped: bool = False):
    part_id = assign(n, group_id, seed, M)
    if grouped:
        part_offsets, perm, local_id = relabel_grouped(part_id, group_id, M)
    else:
        part_offsets, perm, local_id = relabel(part_id, M)
    return part_id, part_offsets, perm, local_id


def induced_csr(rowptr, col, M, part_id, part_offsets, perm, local_id):
    """Returns (rowptr_out[n+M], col_out[E_kept], edge_offsets[M+1], kept, cut)."""
    rowptr = _i64(rowptr)
    col = _i32(col)
    n = rowptr.size - 1
    rowptr_out = np.empty(n + M, dtype=np.int64)
    edge_offsets = np.empty(M + 1, dtype=np.int64)
    kept_cut = np.empty(2, dtype=np.int64)
    args = [ctypes.c_int64(n), _p(rowptr, c_i64p), _p(col, c_i32p), ctypes.c_int32(M),
            _p(_i32(part_id), c_i32p), _p(_i64(part_offsets), c_i64p), _p(_i32(perm), c_i32p),
            _p(_i32(local_id), c_i32p), _p(rowptr_out, c_i64p)]
    tail = [_p(edge_offsets, c_i64p), _p(kept_cut, c_i64p)]
    kept = lib().orc_induced_csr(*args, None, *tail)
    col_out = np.empty(kept, dtype=np.int32)
    lib().orc_induced_csr(*args, _p(col_out, c_i32p), *tail)
    return rowptr_out, col_out, edge_offsets, int(kept_cut[0]), int(kept_cut[1])


def gather_rows(src: np.ndarray, perm: np.ndarray) -> np.ndarray:
    src = np.ascontiguousarray(src)
    perm = _i32(perm)
    dst = np.empty((perm.size,) + src.shape[1:], dtype=src.dtype)
    row_bytes = src.dtype.itemsize * int(np.prod(src.shape[1:], dtype=np.int64))
    lib().orc_gather_rows(ctypes.c_int64(perm.size), ctypes.c_int64(row_bytes),
                          src.ctypes.data_as(ctypes.c_void_p), _p(perm, c_i32p),
                          dst.ctypes.data_as(ctypes.c_void_p))
    return dst


def param_count(dims) -> int:
    d = _i32(dims)
    return int(lib().orc_param_count(ctypes.c_int32(len(dims) - 1), _p(d, c_i32p)))


def _fp(dtype):
    if np.dtype(dtype) == np.float32:
        return "f32", c_f32p, np.float32
    return "f64", c_f64p, np.float64


def spmm_mean(rowptr, col, H: np.ndarray) -> np.ndarray:
    tag, ptr, dt = _fp(H.dtype)
    H = np.ascontiguousarray(H, dtype=dt)
    rowptr = _i64(rowptr)
    col = _i32(col)
    n = rowptr.size - 1
    d = H.shape[1]
    N = np.empty((n, d), dtype=dt)
    getattr(lib(), f"orc_spmm_mean_{tag}")(ctypes.c_int64(n), _p(rowptr, c_i64p), _p(col, c_i32p),
                                          ctypes.c_int64(d), _p(H, ptr), _p(N, ptr))
    return N


def acts_layout(dims, n: int):
    """[(name, offset, rows, width)] of the activation record of one part."""
    out, off = [], 0
    for l in range(len(dims) - 1):
        out.append((f"N{l}", off, n, dims[l]))
        off += n * dims[l]
        out.append((f"H{l + 1}", off, n, dims[l + 1]))
        off += n * dims[l + 1]
    return out, off


def round_to_bf16(x: float) -> float:
    f = lib().orc_round_to_bf16
    f.restype = ctypes.c_double
    return float(f(ctypes.c_double(x)))


def forward_backward(dims, rowptr, col, X, y, params, want_grads=True, want_acts=False, want_preact=False,
                     gates=None, bf16_operands=False):
    """Returns (loss, grads or None, {name: array} or None) for one part.
    bf16_operands: the reduced-precision mode (operands of every dense product rounded to bf16; fp64 only).
    want_preact adds the hidden pre-activations as "Z1".."Z{L-1}" to the dict.
    gates: None, or a list of int8 arrays [n, d_{l+1}] for l = 0..L-2 (-1 natural, 0 closed,
    1 open) overriding the ReLU branch of individual units."""
    tag, ptr, dt = _fp(params.dtype)
    if bf16_operands:
        assert dt == np.float64
        tag = "bf16ops_f64"
        lib().orc_forward_backward_bf16ops_f64.restype = ctypes.c_double
    X = np.ascontiguousarray(X, dtype=dt)
    params = np.ascontiguousarray(params, dtype=dt)
    rowptr = _i64(rowptr)
    col = _i32(col)
    y = _i32(y)
    n = rowptr.size - 1
    d = _i32(dims)
    grads = np.empty(params.size, dtype=dt) if want_grads else None
    acts = None
    layout = None
    if want_acts:
        layout, total = acts_layout(dims, n)
        acts = np.empty(total, dtype=dt)
    hidden = [n * dims[l + 1] for l in range(len(dims) - 2)]
    preact = np.empty(sum(hidden), dtype=dt) if want_preact else None
    gate_buf = None
    if gates is not None:
        gate_buf = np.concatenate([np.ascontiguousarray(g, dtype=np.int8).ravel() for g in gates]) if gates else \
            np.empty(0, dtype=np.int8)
        assert gate_buf.size == sum(hidden)
    loss = getattr(lib(), f"orc_forward_backward_{tag}")(
        ctypes.c_int32(len(dims) - 1), _p(d, c_i32p), ctypes.c_int64(n), _p(rowptr, c_i64p),
        _p(col, c_i32p), _p(X, ptr), _p(y, c_i32p), _p(params, ptr), _p(grads, ptr), _p(acts, ptr),
        _p(preact, ptr), _p(gate_buf, ctypes.POINTER(ctypes.c_int8)))
    named = None
    if want_acts or want_preact:
        named = {}
        if want_acts:
            named.update({nm: acts[o:o + r * w].reshape(r, w) for nm, o, r, w in layout})
        if want_preact:
            off = 0
            for l, size in enumerate(hidden):
                named[f"Z{l + 1}"] = preact[off:off + size].reshape(n, dims[l + 1])
                off += size
    return float(loss), grads, named


def local_steps(dims, lr, rowptr, col, X, y, params, K, bf16_operands=False):
    """K plain-SGD steps on one part.  Returns (new params, loss[K])."""
    tag, ptr, dt = _fp(params.dtype)
    if bf16_operands:
        assert dt == np.float64
        tag = "bf16ops_f64"
    X = np.ascontiguousarray(X, dtype=dt)
    params = np.array(params, dtype=dt, copy=True)
    rowptr = _i64(rowptr)
    col = _i32(col)
    y = _i32(y)
    d = _i32(dims)
    loss = np.empty(K, dtype=np.float64)
    getattr(lib(), f"orc_local_steps_{tag}")(
        ctypes.c_int32(len(dims) - 1), _p(d, c_i32p), ctypes.c_double(lr),
        ctypes.c_int64(rowptr.size - 1), _p(rowptr, c_i64p), _p(col, c_i32p), _p(X, ptr),
        _p(y, c_i32p), _p(params, ptr), ctypes.c_int32(K), _p(loss, c_f64p))
    return params, loss


# ---- model variants: (encoder, act, norm); encoder 0 = GraphSAGE-mean, 1 = GCN; act 0 = ReLU,
# 1 = PReLU; norm 0 = none, 1 = Layer Normalization before the activation -------------------
SAGE_RELU = (0, 0, 0)


def _variant(v):
    return _i32(list(v))


def variant_param_count(variant, dims) -> int:
    d = _i32(dims)
    f = lib().orc_variant_param_count
    f.restype = ctypes.c_int64
    return int(f(_p(_variant(variant), c_i32p), ctypes.c_int32(len(dims) - 1), _p(d, c_i32p)))


def variant_layout(variant, dims):
    """Per layer a dict of offsets into the flat parameter vector: w0, w1, bias, gamma, beta,
    slope (-1 = absent).  GraphSAGE: w0 = Ws, w1 = Wn; GCN: w0 = W."""
    L = len(dims) - 1
    off = np.empty(6 * L, dtype=np.int64)
    lib().orc_variant_layout(_p(_variant(variant), c_i32p), ctypes.c_int32(L), _p(_i32(dims), c_i32p), _p(off, c_i64p))
    names = ("w0", "w1", "bias", "gamma", "beta", "slope")
    return [dict(zip(names, (int(x) for x in off[6 * l:6 * l + 6]))) for l in range(L)]


def variant_init_params(variant, dims, seed) -> np.ndarray:
    """Xavier-uniform weights, zero biases, gamma = 1, beta = 0, PReLU slope = 0.25 (fp64)."""
    rng = np.random.default_rng(seed)
    P = variant_param_count(variant, dims)
    p = np.zeros(P, dtype=np.float64)
    for l, lay in enumerate(variant_layout(variant, dims)):
        d_in, d_out = dims[l], dims[l + 1]
        a = np.sqrt(6.0 / (d_in + d_out))
        for key in ("w0", "w1"):
            if lay[key] >= 0:
                p[lay[key]:lay[key] + d_in * d_out] = rng.uniform(-a, a, size=d_in * d_out)
        if lay["gamma"] >= 0:
            p[lay["gamma"]:lay["gamma"] + d_out] = 1.0
        if lay["slope"] >= 0:
            p[lay["slope"]] = 0.25
    return p


def spmm_gcn(rowptr, col, H: np.ndarray) -> np.ndarray:
    H = np.ascontiguousarray(H, dtype=np.float64)
    rowptr = _i64(rowptr)
    col = _i32(col)
    n, d = rowptr.size - 1, H.shape[1]
    N = np.empty((n, d), dtype=np.float64)
    lib().orc_spmm_gcn_f64(ctypes.c_int64(n), _p(rowptr, c_i64p), _p(col, c_i32p), ctypes.c_int64(d),
                           _p(H, c_f64p), _p(N, c_f64p))
    return N


def forward_backward_variant(variant, dims, rowptr, col, X, y, params, want_grads=True, want_acts=False,
                             want_preact=False, gates=None):
    """forward_backward for a model variant (fp64).  want_preact adds the activations' inputs
    (after the normalisation, if any) of the hidden layers as "Z1".."Z{L-1}"."""
    dt, ptr = np.float64, c_f64p
    X = np.ascontiguousarray(X, dtype=dt)
    params = np.ascontiguousarray(params, dtype=dt)
    rowptr = _i64(rowptr)
    col = _i32(col)
    y = _i32(y)
    n = rowptr.size - 1
    d = _i32(dims)
    assert params.size == variant_param_count(variant, dims)
    grads = np.empty(params.size, dtype=dt) if want_grads else None
    acts, layout = None, None
    if want_acts:
        layout, total = acts_layout(dims, n)
        acts = np.empty(total, dtype=dt)
    hidden = [n * dims[l + 1] for l in range(len(dims) - 2)]
    preact = np.empty(sum(hidden), dtype=dt) if want_preact else None
    gate_buf = None
    if gates is not None:
        gate_buf = np.concatenate([np.ascontiguousarray(g, dtype=np.int8).ravel() for g in gates]) if gates else \
            np.empty(0, dtype=np.int8)
        assert gate_buf.size == sum(hidden)
    f = lib().orc_forward_backward_variant_f64
    f.restype = ctypes.c_double
    loss = f(_p(_variant(variant), c_i32p), ctypes.c_int32(len(dims) - 1), _p(d, c_i32p), ctypes.c_int64(n),
             _p(rowptr, c_i64p), _p(col, c_i32p), _p(X, ptr), _p(y, c_i32p), _p(params, ptr), _p(grads, ptr),
             _p(acts, ptr), _p(preact, ptr), _p(gate_buf, ctypes.POINTER(ctypes.c_int8)))
    named = None
    if want_acts or want_preact:
        named = {}
        if want_acts:
            named.update({nm: acts[o:o + r * w].reshape(r, w) for nm, o, r, w in layout})
        if want_preact:
            off = 0
            for l, size in enumerate(hidden):
                named[f"Z{l + 1}"] = preact[off:off + size].reshape(n, dims[l + 1])
                off += size
    return float(loss), grads, named


def local_steps_variant(variant, dims, lr, rowptr, col, X, y, params, K):
    """K plain-SGD steps on one part for a model variant.  Returns (new params, loss[K])."""
    X = np.ascontiguousarray(X, dtype=np.float64)
    params = np.array(params, dtype=np.float64, copy=True)
    rowptr = _i64(rowptr)
    col = _i32(col)
    y = _i32(y)
    loss = np.empty(K, dtype=np.float64)
    lib().orc_local_steps_variant_f64(
        _p(_variant(variant), c_i32p), ctypes.c_int32(len(dims) - 1), _p(_i32(dims), c_i32p), ctypes.c_double(lr),
        ctypes.c_int64(rowptr.size - 1), _p(rowptr, c_i64p), _p(col, c_i32p), _p(X, c_f64p), _p(y, c_i32p),
        _p(params, c_f64p), ctypes.c_int32(K), _p(loss, c_f64p))
    return params, loss


# ---- link prediction --------------------------------------------------------------------------
def link_param_count(variant, dims, ddims) -> int:
    f = lib().orc_link_param_count
    f.restype = ctypes.c_int64
    return int(f(_p(_variant(variant), c_i32p), ctypes.c_int32(len(dims) - 1), _p(_i32(dims), c_i32p),
                 ctypes.c_int32(len(ddims) - 1), _p(_i32(ddims), c_i32p)))


def link_decoder_layout(variant, dims, ddims):
    """[(theta offset, slope offset or -1)] per decoder layer."""
    Kd = len(ddims) - 1
    off = np.empty(2 * Kd, dtype=np.int64)
    lib().orc_link_decoder_layout(_p(_variant(variant), c_i32p), ctypes.c_int32(len(dims) - 1), _p(_i32(dims), c_i32p),
                                  ctypes.c_int32(Kd), _p(_i32(ddims), c_i32p), _p(off, c_i64p))
    return [(int(off[2 * k]), int(off[2 * k + 1])) for k in range(Kd)]


def link_init_params(variant, dims, ddims, seed) -> np.ndarray:
    """Encoder as variant_init_params; decoder Xavier-uniform weights, slopes 0.25 (fp64)."""
    enc = variant_init_params(variant, dims, seed)
    rng = np.random.default_rng(seed + 1000)
    p = np.zeros(link_param_count(variant, dims, ddims), dtype=np.float64)
    p[:enc.size] = enc
    for k, (theta, slope) in enumerate(link_decoder_layout(variant, dims, ddims)):
        a = np.sqrt(6.0 / (ddims[k] + ddims[k + 1]))
        p[theta:theta + ddims[k] * ddims[k + 1]] = rng.uniform(-a, a, size=ddims[k] * ddims[k + 1])
        if slope >= 0:
            p[slope] = 0.25
    return p


def link_forward_backward(variant, dims, ddims, rowptr, col, X, pu, pv, label, params, want_grads=True,
                          preact_out=None, gates=None):
    """Encoder + MLP decoder + binary cross-entropy on the given pairs of one part (fp64).
    Returns (loss, grads or None, embeddings [n, dims[-1]], scores [B]).
    preact_out: None or a float64 array of link_gate_count() entries that receives the input of
    every hidden ReLU / PReLU (encoder layers, then decoder layers); gates: None or an int8 array
    of the same length (-1 natural, 0 closed, 1 open)."""
    X = np.ascontiguousarray(X, dtype=np.float64)
    params = np.ascontiguousarray(params, dtype=np.float64)
    rowptr, col = _i64(rowptr), _i32(col)
    pu, pv, label = _i32(pu), _i32(pv), _i32(label)
    n, B = rowptr.size - 1, pu.size
    assert ddims[0] == dims[-1] and ddims[-1] == 1 and params.size == link_param_count(variant, dims, ddims)
    grads = np.empty(params.size, dtype=np.float64) if want_grads else None
    emb = np.empty((n, dims[-1]), dtype=np.float64)
    scores = np.empty(B, dtype=np.float64)
    f = lib().orc_link_forward_backward_f64
    f.restype = ctypes.c_double
    loss = f(_p(_variant(variant), c_i32p), ctypes.c_int32(len(dims) - 1), _p(_i32(dims), c_i32p),
             ctypes.c_int32(len(ddims) - 1), _p(_i32(ddims), c_i32p), ctypes.c_int64(n), _p(rowptr, c_i64p),
             _p(col, c_i32p), _p(X, c_f64p), ctypes.c_int64(B), _p(pu, c_i32p), _p(pv, c_i32p), _p(label, c_i32p),
             _p(params, c_f64p), _p(grads, c_f64p), _p(emb, c_f64p), _p(scores, c_f64p), _p(preact_out, c_f64p),
             _p(None if gates is None else np.ascontiguousarray(gates, dtype=np.int8), ctypes.POINTER(ctypes.c_int8)))
    return float(loss), grads, emb, scores


def link_gate_count(dims, ddims, n: int, B: int) -> int:
    return n * sum(dims[1:-1]) + B * sum(ddims[1:-1])


def average(params: np.ndarray):
    """params [M, P] -> (averaged copies [M, P], global [P])."""
    tag, ptr, dt = _fp(params.dtype)
    out = np.array(params, dtype=dt, copy=True, order="C")
    M, P = out.shape
    glob = np.empty(P, dtype=dt)
    getattr(lib(), f"orc_average_{tag}")(_p(out, ptr), ctypes.c_int64(P), ctypes.c_int32(M), _p(glob, ptr))
    return out, glob


def sample_hop(rowptr, col, frontier, fanout: int, seed: int, hop: int):
    """One hop of the neighbour sampler on one part's subgraph.  frontier: ascending distinct local
    ids.  Returns (block_rowptr[len(frontier)+1], block_col, next_frontier)."""
    rowptr = _i64(rowptr)
    col = _i32(col)
    frontier = _i32(frontier)
    n = rowptr.size - 1
    fs = frontier.size
    block_rowptr = np.empty(fs + 1, dtype=np.int64)
    next_frontier = np.empty(n, dtype=np.int32)
    f = lib().orc_sample_hop
    f.restype = ctypes.c_int64
    args = [ctypes.c_int64(n), _p(rowptr, c_i64p), _p(col, c_i32p), ctypes.c_int64(fs), _p(frontier, c_i32p),
            ctypes.c_int32(fanout), ctypes.c_uint64(seed), ctypes.c_int32(hop), _p(block_rowptr, c_i64p)]
    f(*args, None, _p(next_frontier, c_i32p))
    block_col = np.empty(int(block_rowptr[-1]), dtype=np.int32)
    size = f(*args, _p(block_col, c_i32p), _p(next_frontier, c_i32p))
    return block_rowptr, block_col, next_frontier[:int(size)].copy()


def sigmoid_l2_grad(rowptr, col, X, y, w):
    rowptr = _i64(rowptr)
    col = _i32(col)
    X = np.ascontiguousarray(X, dtype=np.float64)
    y = np.ascontiguousarray(y, dtype=np.float64)
    w = np.ascontiguousarray(w, dtype=np.float64)
    n, d = X.shape
    g = np.empty((n, d), dtype=np.float64)
    lib().orc_sigmoid_l2_grad(ctypes.c_int64(n), _p(rowptr, c_i64p), _p(col, c_i32p), ctypes.c_int64(d),
                              _p(X, c_f64p), _p(y, c_f64p), _p(w, c_f64p), _p(g, c_f64p))
    return g


def part_graph(rowptr_out, col_out, part_offsets, edge_offsets, p: int):
    """Slice part p's CSR out of the packed induced-CSR arrays."""
    lo = int(part_offsets[p]) + p
    n_p = int(part_offsets[p + 1] - part_offsets[p])
    rp = rowptr_out[lo:lo + n_p + 1]
    cp = col_out[int(edge_offsets[p]):int(edge_offsets[p + 1])]
    return rp, cp


def run_method(rowptr, col, X, y, dims, M, K, R, lr, seed, params0, group_id=None, dtype=np.float64):
    """The whole path on the CPU: partition, induced CSR, R rounds of K local
    steps on each of the M parts followed by averaging.  Returns a dict."""
    n = len(rowptr) - 1
    part_id, part_offsets, perm, local_id = partition(n, group_id, seed, M)
    rowptr_out, col_out, edge_offsets, kept, cut = induced_csr(
        rowptr, col, M, part_id, part_offsets, perm, local_id)
    Xp = gather_rows(X, perm)
    yp = gather_rows(y, perm)
    params = np.tile(np.asarray(params0, dtype=dtype), (M, 1))
    losses = np.zeros((R, M, K))
    for r in range(R):
        for p in range(M):
            rp, cp = part_graph(rowptr_out, col_out, part_offsets, edge_offsets, p)
            lo, hi = int(part_offsets[p]), int(part_offsets[p + 1])
            params[p], losses[r, p] = local_steps(dims, lr, rp, cp, Xp[lo:hi], yp[lo:hi], params[p], K)
        params, _ = average(params)
    return dict(part_id=part_id, part_offsets=part_offsets, perm=perm, local_id=local_id,
                rowptr_out=rowptr_out, col_out=col_out, edge_offsets=edge_offsets,
                kept=kept, cut=cut, Xp=Xp, yp=yp, params=params, losses=losses)
