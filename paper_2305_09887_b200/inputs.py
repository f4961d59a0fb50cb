"""Seeded synthetic inputs: graphs, features, labels and initial weights.

Everything here is input plumbing.  It holds none of the method's arithmetic
(no partition hash, no aggregation, no training maths): randomness comes from
numpy's ``default_rng(seed)`` or, for the arrays with up to billions of
elements (endpoint pairs, CSR construction, normal features), from the
counter-based draws of the multi-threaded host library ``inputs_native.cpp``;
the arrays produced are handed unchanged to whichever implementation consumes
them.  The shapes stand in for the paper's
workloads (Table 1: social / citation / e-commerce graphs with power-law
degrees, 100-768 wide features), which are not redistributed with this code.

Graph convention: CSR over directed entries, both directions of every
undirected edge stored, no self loops, no duplicates, columns sorted.
"""
from __future__ import annotations

import ctypes
import dataclasses
import math
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_NATIVE_SRC = os.path.join(_HERE, "inputs_native.cpp")
_NATIVE_LIB = os.path.join(_HERE, "libinputs_native.so")
_native_handle = None


def build_native(force: bool = False) -> str:
    """Compiles inputs_native.cpp (g++, host only) next to this file."""
    if force or not os.path.exists(_NATIVE_LIB) or os.path.getmtime(_NATIVE_LIB) < os.path.getmtime(_NATIVE_SRC):
        tmp = f"{_NATIVE_LIB}.{os.getpid()}.tmp"
        subprocess.run(["g++", "-O3", "-std=c++17", "-fPIC", "-shared", "-pthread", _NATIVE_SRC, "-o", tmp], check=True)
        os.replace(tmp, _NATIVE_LIB)
    return _NATIVE_LIB


def _native():
    global _native_handle
    if _native_handle is None:
        lib = ctypes.CDLL(build_native())
        i64, u64, f64, ptr = ctypes.c_int64, ctypes.c_uint64, ctypes.c_double, ctypes.c_void_p
        lib.rin_threads.restype = ctypes.c_int32
        lib.rin_power_law_pairs.argtypes = [i64, i64, f64, f64, u64, ptr, ptr]
        lib.rin_power_law_pairs.restype = None
        lib.rin_csr_rows.argtypes = [i64, i64, ptr, ptr, ptr, ptr, ptr]
        lib.rin_csr_rows.restype = i64
        lib.rin_csr_compact.argtypes = [i64, ptr, ptr, ptr, ptr]
        lib.rin_csr_compact.restype = None
        lib.rin_normal_f32.argtypes = [i64, u64, ptr]
        lib.rin_normal_f32.restype = None
        lib.rin_add_rows_f32.argtypes = [i64, i64, ptr, ptr, ctypes.c_float, ptr]
        lib.rin_add_rows_f32.restype = None
        _native_handle = lib
    return _native_handle


def native_threads() -> int:
    """Host threads the native producers use."""
    return int(_native().rin_threads())


def _p(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


@dataclasses.dataclass
class Graph:
    n: int
    rowptr: np.ndarray  # int32 or int64, [n+1]
    col: np.ndarray     # int32, [E]
    group_id: np.ndarray | None = None  # int32 [n], super-node id per node

    @property
    def num_entries(self) -> int:
        return int(self.rowptr[-1])


@dataclasses.dataclass
class Workload:
    name: str
    graph: Graph
    X: np.ndarray        # float32 [n, F]
    y: np.ndarray        # int32 [n]
    dims: tuple          # (F, hidden..., C)
    M: int
    K: int               # local steps per round
    R: int               # aggregation rounds
    lr: float
    partition_seed: int
    params0: np.ndarray  # float32 [P], identical start for every trainer
    use_groups: bool = False
    grouped_order: bool = False  # with use_groups: rows of a part ordered by super-node id, then node id
    gemm_dtype: int = 0  # 0: fp32-accurate GEMMs, 1: bf16 inputs / fp32 accumulate
    variant: tuple = (0, 0, 0)  # (encoder, act, norm): 0,0,0 = GraphSAGE-mean, ReLU, no normalisation


def _csr_from_pairs(n: int, u: np.ndarray, v: np.ndarray, wide_rowptr: bool) -> Graph:
    """Symmetrise, drop loops and duplicates, sort the columns of every row, and build CSR."""
    u = np.ascontiguousarray(u, dtype=np.int32)
    v = np.ascontiguousarray(v, dtype=np.int32)
    m = int(u.size)
    lib = _native()
    tmp_rowptr = np.empty(n + 1, dtype=np.int64)
    rowptr = np.empty(n + 1, dtype=np.int64)
    col_tmp = np.empty(2 * m, dtype=np.int32)
    entries = int(lib.rin_csr_rows(n, m, _p(u), _p(v), _p(tmp_rowptr), _p(col_tmp), _p(rowptr)))
    del u, v
    col = np.empty(entries, dtype=np.int32)
    lib.rin_csr_compact(n, _p(tmp_rowptr), _p(rowptr), _p(col_tmp), _p(col))
    del col_tmp, tmp_rowptr
    if not wide_rowptr:
        assert rowptr[-1] < 2**31
        rowptr = rowptr.astype(np.int32)
    return Graph(n=n, rowptr=rowptr, col=col)


def uniform_graph(n: int, m_undirected: int, seed: int, wide_rowptr: bool = False) -> Graph:
    """G(n, m): m distinct undirected pairs chosen uniformly, no loops."""
    rng = np.random.default_rng(seed)
    have = np.empty(0, dtype=np.int64)
    while have.size < m_undirected:
        need = m_undirected - have.size
        a = rng.integers(0, n, size=need + need // 8 + 16, dtype=np.int64)
        b = rng.integers(0, n, size=a.size, dtype=np.int64)
        ok = a != b
        lo = np.minimum(a[ok], b[ok])
        hi = np.maximum(a[ok], b[ok])
        have = np.unique(np.concatenate([have, lo * n + hi]))
    if have.size > m_undirected:
        have = rng.permutation(have)[:m_undirected]
    return _csr_from_pairs(n, have // n, have % n, wide_rowptr)


def _power_law_offset(n: int, gamma: float, target_entries: float):
    """Endpoint weights w(x) = (x + i0)^expo over ranks x in [0, n), expo = -1/(gamma-1).  i0 caps
    the largest expected degree, target * W(0,1) / W(0,n) with W the integral of w, at
    sqrt(target_entries).  Returns (i0, expo)."""
    expo = -1.0 / (gamma - 1.0)
    e1 = expo + 1.0
    cap = math.sqrt(target_entries)

    def integral(a: float, b: float, i0: float) -> float:
        if abs(e1) < 1e-12:
            return math.log((b + i0) / (a + i0))
        return ((b + i0) ** e1 - (a + i0) ** e1) / e1

    def top_degree(i0: float) -> float:
        return target_entries * integral(0.0, 1.0, i0) / integral(0.0, float(n), i0)

    lo, hi = 1e-3, float(n)
    if top_degree(lo) <= cap:
        return lo, expo
    for _ in range(80):
        mid = math.sqrt(lo * hi)
        if top_degree(mid) > cap:
            lo = mid
        else:
            hi = mid
    return hi, expo


def _power_law_pairs(n: int, m: int, gamma: float, target_entries: float, seed: int):
    """m endpoint pairs, each endpoint drawn in proportion to its power-law weight; node ids are a
    keyed permutation of the ranks, so hubs are spread over the id range."""
    i0, expo = _power_law_offset(n, gamma, target_entries)
    u = np.empty(m, dtype=np.int32)
    v = np.empty(m, dtype=np.int32)
    _native().rin_power_law_pairs(n, m, i0, expo, seed, _p(u), _p(v))
    return u, v


def chung_lu_graph(n: int, avg_degree: float, gamma: float, seed: int,
                   wide_rowptr: bool = False) -> Graph:
    """Chung-Lu power-law graph by endpoint sampling, node ids shuffled so that
    hubs are spread over the id range."""
    target = float(n) * avg_degree
    u, v = _power_law_pairs(n, int(target // 2), gamma, target, seed)
    return _csr_from_pairs(n, u, v, wide_rowptr)


def planted_community_graph(n_clusters: int, cluster_size: int, intra_degree: float,
                            inter_degree: float, gamma: float, seed: int,
                            wide_rowptr: bool = False) -> Graph:
    """Clusters of equal size with Bernoulli edges inside each cluster and a
    power-law Chung-Lu overlay between clusters.  ``group_id`` holds each
    node's cluster; clusters are scattered over the node-id range."""
    rng = np.random.default_rng(seed)
    n = n_clusters * cluster_size
    node_of_slot = rng.permutation(n).astype(np.int64)  # slot = cluster*size + k
    group_id = np.empty(n, dtype=np.int32)
    group_id[node_of_slot] = (np.arange(n) // cluster_size).astype(np.int32)

    iu, iv = np.triu_indices(cluster_size, k=1)
    pairs_per = iu.size
    p = intra_degree / (cluster_size - 1)
    us, vs = [], []
    chunk = max(1, (1 << 24) // pairs_per)
    for c0 in range(0, n_clusters, chunk):
        c1 = min(n_clusters, c0 + chunk)
        hit = np.flatnonzero(rng.random((c1 - c0) * pairs_per) < p)
        c = hit // pairs_per + c0
        k = hit % pairs_per
        us.append(node_of_slot[c * cluster_size + iu[k]])
        vs.append(node_of_slot[c * cluster_size + iv[k]])

    target = float(n) * inter_degree
    if target > 0:
        a, b = _power_law_pairs(n, int(target // 2), gamma, target, seed)
        differ = group_id[a] != group_id[b]
        us.append(a[differ])
        vs.append(b[differ])
    g = _csr_from_pairs(n, np.concatenate(us), np.concatenate(vs), wide_rowptr)
    g.group_id = group_id
    return g


def two_class_block_graph(n: int, avg_degree: float, h: float, seed: int):
    """Two equal classes; an edge joins same-class nodes with probability
    proportional to h and different-class nodes proportional to 1-h (the
    compatibility-matrix model of Lemma 1).  Returns (graph, labels)."""
    rng = np.random.default_rng(seed)
    y = (rng.permutation(n) % 2).astype(np.int32)
    m = int(n * avg_degree / 2)
    u = rng.integers(0, n, size=m, dtype=np.int64)
    same = rng.random(m) < h
    members = [np.flatnonzero(y == 0), np.flatnonzero(y == 1)]
    v = np.empty(m, dtype=np.int64)
    for cls in (0, 1):
        for want_same in (False, True):
            sel = (y[u] == cls) & (same == want_same)
            pool = members[cls if want_same else 1 - cls]
            v[sel] = pool[rng.integers(0, pool.size, size=int(sel.sum()))]
    return _csr_from_pairs(n, u, v, False), y


def normal_features(n: int, F: int, seed: int, y: np.ndarray | None = None,
                    n_classes: int = 0, shift: float = 0.0, native: bool = False) -> np.ndarray:
    """N(0,1) features; with ``shift`` a class-dependent mean shift*mu_y, mu_c ~ N(0,I).
    ``native``: draw with the multi-threaded host library (the named workloads, whose feature
    matrices have up to billions of elements) instead of numpy's generator (a different stream)."""
    rng = np.random.default_rng(seed)
    if not native:
        X = rng.standard_normal((n, F), dtype=np.float32)
        if shift != 0.0 and y is not None:
            mu = rng.standard_normal((n_classes, F), dtype=np.float32)
            X += np.float32(shift) * mu[y]
        return X
    X = np.empty((n, F), dtype=np.float32)
    _native().rin_normal_f32(n * F, seed, _p(X))
    if shift != 0.0 and y is not None:
        mu = rng.standard_normal((n_classes, F), dtype=np.float32)
        _native().rin_add_rows_f32(n, F, _p(np.ascontiguousarray(y, dtype=np.int32)), _p(mu), shift, _p(X))
    return X


def uniform_labels(n: int, n_classes: int, seed: int) -> np.ndarray:
    return np.random.default_rng(seed).integers(0, n_classes, size=n, dtype=np.int32)


def rare_positive_labels(n: int, positive_rate: float, seed: int) -> np.ndarray:
    return (np.random.default_rng(seed).random(n) < positive_rate).astype(np.int32)


def param_count(dims) -> int:
    return sum(2 * dims[l] * dims[l + 1] + dims[l + 1] for l in range(len(dims) - 1))


def xavier_params(dims, seed: int) -> np.ndarray:
    """Flat parameter vector, layer-major: W_self[d_in][d_out], W_neigh[d_in][d_out],
    b[d_out].  Weights U(-a, a) with a = sqrt(6/(d_in+d_out)); biases zero."""
    rng = np.random.default_rng(seed)
    out = []
    for l in range(len(dims) - 1):
        d_in, d_out = dims[l], dims[l + 1]
        a = math.sqrt(6.0 / (d_in + d_out))
        out.append(rng.uniform(-a, a, size=2 * d_in * d_out).astype(np.float32))
        out.append(np.zeros(d_out, dtype=np.float32))
    return np.concatenate(out)


def variant_param_count(variant, dims) -> int:
    """Parameters of a model variant (encoder, act, norm): GCN (encoder 1) has one weight matrix
    per layer; hidden layers add gamma, beta (norm 1) and one PReLU slope (act 1)."""
    encoder, act, norm = variant
    total = 0
    for l in range(len(dims) - 1):
        total += (1 if encoder == 1 else 2) * dims[l] * dims[l + 1] + dims[l + 1]
        if l < len(dims) - 2:
            total += (2 * dims[l + 1] if norm == 1 else 0) + (1 if act == 1 else 0)
    return total


def variant_params(variant, dims, seed: int) -> np.ndarray:
    """Initial parameters of a model variant, in the library's order (weights, b, gamma, beta,
    slope per layer): Xavier-uniform weights, zero biases, gamma 1, beta 0, slope 0.25."""
    encoder, act, norm = variant
    rng = np.random.default_rng(seed)
    out = []
    for l in range(len(dims) - 1):
        d_in, d_out = dims[l], dims[l + 1]
        a = math.sqrt(6.0 / (d_in + d_out))
        out.append(rng.uniform(-a, a, size=(1 if encoder == 1 else 2) * d_in * d_out).astype(np.float32))
        out.append(np.zeros(d_out, dtype=np.float32))
        if l < len(dims) - 2:
            if norm == 1:
                out.append(np.ones(d_out, dtype=np.float32))
                out.append(np.zeros(d_out, dtype=np.float32))
            if act == 1:
                out.append(np.full(1, 0.25, dtype=np.float32))
    return np.concatenate(out)


def link_param_count(variant, dims, ddims) -> int:
    """Encoder variant + MLP decoder (Theta^k [ddims[k]][ddims[k+1]], one PReLU slope per hidden layer)."""
    dec = sum(ddims[k] * ddims[k + 1] for k in range(len(ddims) - 1)) + (len(ddims) - 2)
    return variant_param_count(variant, dims) + dec


def link_params(variant, dims, ddims, seed: int) -> np.ndarray:
    """Initial parameters for link prediction in the library's order: the encoder's
    (variant_params), then per decoder layer Xavier-uniform Theta^k and (hidden layers) slope 0.25."""
    rng = np.random.default_rng(seed + 1)
    out = [variant_params(variant, dims, seed)]
    for k in range(len(ddims) - 1):
        a = math.sqrt(6.0 / (ddims[k] + ddims[k + 1]))
        out.append(rng.uniform(-a, a, size=ddims[k] * ddims[k + 1]).astype(np.float32))
        if k < len(ddims) - 2:
            out.append(np.full(1, 0.25, dtype=np.float32))
    return np.concatenate(out)


def link_pairs(rowptr_out, col_out, part_offsets, edge_offsets, M: int, seed: int, max_positives: int):
    """Training pairs per part from its induced subgraph (local ids): up to max_positives of the
    part's undirected edges (entries with row < col) as positives, and for each positive (u, v)
    one negative (u, v') with a uniformly drawn tail.  Returns (pair_u, pair_v, label, offsets[M+1])."""
    rng = np.random.default_rng(seed)
    pu, pv, lab, off = [], [], [], [0]
    for p in range(M):
        n_p = int(part_offsets[p + 1] - part_offsets[p])
        base = int(part_offsets[p]) + p
        rp = np.asarray(rowptr_out[base:base + n_p + 1])
        cp = np.asarray(col_out[int(edge_offsets[p]):int(edge_offsets[p + 1])])
        rows = np.repeat(np.arange(n_p, dtype=np.int32), np.diff(rp))
        keep = np.flatnonzero(rows < cp)
        if keep.size > max_positives:
            keep = np.sort(rng.choice(keep, size=max_positives, replace=False))
        k = keep.size
        if k:
            neg = rng.integers(0, n_p, size=k).astype(np.int32)
            pu += [rows[keep], rows[keep]]
            pv += [cp[keep].astype(np.int32), neg]
            lab += [np.ones(k, np.int32), np.zeros(k, np.int32)]
        off.append(off[-1] + 2 * k)
    cat = lambda xs: np.concatenate(xs).astype(np.int32) if xs else np.empty(0, np.int32)
    return cat(pu), cat(pv), cat(lab), off


SEED_GRAPH, SEED_FEAT, SEED_LABEL, SEED_WEIGHT, SEED_PART = (
    0x5EED0001, 0x5EED0002, 0x5EED0003, 0x5EED0004, 0x5EED0005)


def tiny() -> Workload:
    """2,000 nodes, 10,000 undirected edges, 64-d features, 8 classes, M=4."""
    g = uniform_graph(2000, 10000, SEED_GRAPH)
    y = uniform_labels(g.n, 8, SEED_LABEL)
    X = normal_features(g.n, 64, SEED_FEAT)
    dims = (64, 64, 8)
    return Workload("tiny", g, X, y, dims, M=4, K=5, R=1, lr=0.01,
                    partition_seed=SEED_PART, params0=xavier_params(dims, SEED_WEIGHT))


def medium(scale: float = 1.0) -> Workload:
    """Chung-Lu, 200k nodes, exponent 2.1, average degree 25, 128-d class-shifted
    features, 47 classes, M=8, three layers of width 256, 20 steps x 5 rounds."""
    n = int(200_000 * scale)
    g = chung_lu_graph(n, 25.0, 2.1, SEED_GRAPH + 1)
    y = uniform_labels(n, 47, SEED_LABEL + 1)
    X = normal_features(n, 128, SEED_FEAT + 1, y, 47, 0.5, native=True)
    dims = (128, 256, 256, 47)
    return Workload("medium" if scale == 1.0 else f"medium_x{scale:g}", g, X, y, dims,
                    M=8, K=20, R=5, lr=0.01, partition_seed=SEED_PART + 1,
                    params0=xavier_params(dims, SEED_WEIGHT + 1))


def supertma(scale: float = 1.0, width: int | None = None, M: int = 16,
             use_groups: bool = True, gemm_dtype: int = 0) -> Workload:
    """Planted communities: 20,000 super-nodes of 100 nodes, intra degree 20,
    inter-cluster power-law degree 10, labels constant per cluster, 100-d
    features, 47 classes, three layers of width 256, 10 steps x 3 rounds.
    ``width`` = 512 gives the trainer-count / width sweep shape."""
    n_clusters = max(2, int(20_000 * scale))
    g = planted_community_graph(n_clusters, 100, 20.0, 10.0, 2.1, SEED_GRAPH + 2)
    cluster_label = uniform_labels(n_clusters, 47, SEED_LABEL + 2)
    y = cluster_label[g.group_id].astype(np.int32)
    F = 100 if width is None else width
    hid = 256 if width is None else width
    X = normal_features(g.n, F, SEED_FEAT + 2, y, 47, 0.5, native=True)
    dims = (F, hid, hid, 47)
    K, R = (10, 3) if width is None else (5, 1)
    name = "supertma" if width is None else f"sweep_w{width}_M{M}_{'super' if use_groups else 'node'}"
    if scale != 1.0:
        name += f"_x{scale:g}"
    return Workload(name, g, X, y, dims, M=M, K=K, R=R, lr=0.01,
                    partition_seed=SEED_PART + 2, params0=xavier_params(dims, SEED_WEIGHT + 2),
                    use_groups=use_groups, gemm_dtype=gemm_dtype)


def large(scale: float = 1.0) -> Workload:
    """Chung-Lu, 25M nodes, exponent 2.0, ~1.3B directed entries (int64 row
    offsets), 128-d features, 2 classes with 1% positives, M=32, two layers."""
    n = int(25_000_000 * scale)
    g = chung_lu_graph(n, 52.0, 2.0, SEED_GRAPH + 3, wide_rowptr=True)
    y = rare_positive_labels(n, 0.01, SEED_LABEL + 3)
    X = normal_features(n, 128, SEED_FEAT + 3, native=True)
    dims = (128, 256, 2)
    return Workload("large" if scale == 1.0 else f"large_x{scale:g}", g, X, y, dims,
                    M=32, K=5, R=1, lr=0.01, partition_seed=SEED_PART + 3,
                    params0=xavier_params(dims, SEED_WEIGHT + 3))
