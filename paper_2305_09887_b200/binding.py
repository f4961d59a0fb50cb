"""Thin ctypes binding over the CUDA C-ABI library (``librtma.so``, see ``include/rtma.h``).

Argument marshalling only: tensors are allocated with torch (device memory and streams are
all torch is used for) and handed to the library as raw pointers; every step of the path
runs in the library's kernels.  There is no CPU fallback: if the library is missing or no
CUDA device is present the calls raise.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librtma.so")
LIB_CHECKED_PATH = os.path.join(_PKG, "librtma_checked.so")   # built with -DRTMA_BOUNDS: every caller-supplied index checked
MAX_PARTS = 64
MAX_LAYERS = 8

EXPORTS = (
    "rtma_create", "rtma_destroy", "rtma_last_error", "rtma_workspace_bytes", "rtma_partition", "rtma_partition_grouped",
    "rtma_build_induced_csr", "rtma_gather_rows", "rtma_param_count", "rtma_local_steps",
    "rtma_aggregate", "rtma_sgd_aggregate", "rtma_train_host", "rtma_profile", "rtma_profile_read",
    "rtma_kernel_class_name", "rtma_check", "rtma_partition_static", "rtma_partition_static_error",
    "rtma_local_steps_var", "rtma_aggregate_masked", "rtma_selftest_wait_timeout", "rtma_link_param_count",
    "rtma_link_steps", "rtma_set_workspace_limit", "rtma_local_steps_gathered", "rtma_bounds_checked", "rtma_sample_hop",
    "rtma_set_dense_aggregation",
)
KERNEL_CLASSES = 21

_libs = {}


class RtmaError(RuntimeError):
    pass


class ModelDesc(ctypes.Structure):
    _fields_ = [("L", ctypes.c_int32), ("dims", ctypes.c_int32 * (MAX_LAYERS + 1)),
                ("gemm_dtype", ctypes.c_int32), ("lr", ctypes.c_float), ("encoder", ctypes.c_int32),
                ("act", ctypes.c_int32), ("norm", ctypes.c_int32)]


class DecoderDesc(ctypes.Structure):
    _fields_ = [("Kd", ctypes.c_int32), ("ddims", ctypes.c_int32 * (MAX_LAYERS + 1))]


def decoder_desc(ddims) -> DecoderDesc:
    Kd = len(ddims) - 1
    if not 1 <= Kd <= MAX_LAYERS:
        raise ValueError(f"number of decoder layers {Kd} outside [1, {MAX_LAYERS}]")
    dd = DecoderDesc()
    dd.Kd = Kd
    for i, d in enumerate(ddims):
        dd.ddims[i] = int(d)
    return dd


class Taps(ctypes.Structure):
    _fields_ = [("acts", ctypes.c_void_p), ("grads", ctypes.c_void_p), ("step", ctypes.c_int32)]


def load_library(checked: bool = False):
    """Loads the shared library (checked: the range-checked build); raises if it has not been built."""
    path = LIB_CHECKED_PATH if checked else LIB_PATH
    if path not in _libs:
        if not os.path.exists(path):
            raise RtmaError(f"{path} not found: build it with `python -m paper_2305_09887_b200.build"
                            f"{' --checked' if checked else ''}` (there is no CPU fallback)")
        lib = ctypes.CDLL(path)
        lib.rtma_last_error.restype = ctypes.c_char_p
        lib.rtma_last_error.argtypes = [ctypes.c_void_p]
        lib.rtma_workspace_bytes.restype = ctypes.c_size_t
        lib.rtma_workspace_bytes.argtypes = [ctypes.c_void_p]
        lib.rtma_param_count.restype = ctypes.c_int64
        lib.rtma_kernel_class_name.restype = ctypes.c_char_p
        lib.rtma_partition_static_error.restype = ctypes.c_char_p
        _libs[path] = lib
    return _libs[path]


def model_desc(dims, lr: float = 0.01, gemm_dtype: int = 0, variant=(0, 0, 0)) -> ModelDesc:
    L = len(dims) - 1
    if not 1 <= L <= MAX_LAYERS:
        raise ValueError(f"number of layers {L} outside [1, {MAX_LAYERS}]")
    md = ModelDesc()
    md.L = L
    for i, d in enumerate(dims):
        md.dims[i] = int(d)
    md.gemm_dtype = int(gemm_dtype)
    md.lr = float(lr)
    md.encoder, md.act, md.norm = (int(v) for v in variant)
    return md


def link_param_count(dims, ddims, variant=(0, 0, 0)) -> int:
    lib = load_library()
    lib.rtma_link_param_count.restype = ctypes.c_int64
    return int(lib.rtma_link_param_count(ctypes.byref(model_desc(dims, variant=variant)), ctypes.byref(decoder_desc(ddims))))


def param_count(dims, variant=(0, 0, 0)) -> int:
    return int(load_library().rtma_param_count(ctypes.byref(model_desc(dims, variant=variant))))


def _ptr(t):
    if t is None:
        return ctypes.c_void_p(0)
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream_handle(stream) -> int:
    if stream is None:
        return int(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def _need(t, dtype, name, device=None):
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if device is not None and t.device != device:
        raise ValueError(f"{name} must live on {device}, got {t.device}")
    return t


PARTITION_STATIC_MAX_CELLS = 262144


def partition_static(n: int, group_id, seed: int, M: int, device: int = 0, stream=None):
    """rtma_partition for callers that must not allocate while partitioning: no context, scratch
    in a fixed array inside the library, limited to ceil(n/1024)*M <= PARTITION_STATIC_MAX_CELLS.
    The four output tensors are still the caller's (allocated here with torch for convenience;
    a caller that cannot allocate passes its own buffers through the C ABI).  Same results as
    Context.partition, bit for bit.  Calls share the fixed scratch: keep them stream-ordered."""
    lib = load_library()
    dev = torch.device("cuda", device)
    if group_id is not None:
        _need(group_id, torch.int32, "group_id", dev)
    part_id = torch.empty(n, dtype=torch.int32, device=dev)
    part_offsets = torch.empty(M + 1, dtype=torch.int64, device=dev)
    perm = torch.empty(n, dtype=torch.int32, device=dev)
    local_id = torch.empty(n, dtype=torch.int32, device=dev)
    st = lib.rtma_partition_static(ctypes.c_int32(device), ctypes.c_int64(n), _ptr(group_id), ctypes.c_uint64(seed),
                                   ctypes.c_int32(M), _ptr(part_id), _ptr(part_offsets), _ptr(perm), _ptr(local_id),
                                   ctypes.c_void_p(_stream_handle(stream)))
    if st != 0:
        raise RtmaError(f"rtma_partition_static failed ({st}): {lib.rtma_partition_static_error().decode()}")
    return part_id, part_offsets, perm, local_id


class Context:
    """One library context on one CUDA device.  Calls are enqueued on the given (or the
    current torch) stream and share the context's scratch, so keep them stream-ordered."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0, checked: bool = False):
        if not torch.cuda.is_available():
            raise RtmaError("no CUDA device: this library has no CPU path")
        self._lib = load_library(checked)
        self.device = torch.device("cuda", device)
        torch.cuda.init()
        with torch.cuda.device(self.device):
            torch.zeros(1, device=self.device)  # make sure the primary context exists
        h = ctypes.c_void_p()
        st = self._lib.rtma_create(ctypes.byref(h), ctypes.c_int32(device), ctypes.c_size_t(workspace_bytes))
        if st != 0:
            raise RtmaError(f"rtma_create failed with status {st}")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            self._lib.rtma_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st, what):
        if st != 0:
            raise RtmaError(f"{what} failed ({st}): {self._lib.rtma_last_error(self._h).decode()}")

    @property
    def workspace_bytes(self) -> int:
        return int(self._lib.rtma_workspace_bytes(self._h))

    def set_workspace_limit(self, nbytes: int):
        """Caps the context's scratch arena (0 = no cap); rtma_local_steps then runs in waves."""
        self._check(self._lib.rtma_set_workspace_limit(self._h, ctypes.c_size_t(nbytes)), "rtma_set_workspace_limit")

    def set_dense_aggregation(self, mode: int):
        """0: always gather; 1 (default): tensor-core tiles for parts with local neighbourhoods; 2: for every part."""
        self._check(self._lib.rtma_set_dense_aggregation(self._h, ctypes.c_int32(mode)), "rtma_set_dense_aggregation")

    def check(self):
        """Synchronises and raises if a kernel gave up on a bounded device-side wait."""
        self._check(self._lib.rtma_check(self._h), "rtma_check")

    # ---- instrumentation ------------------------------------------------------------
    def profile(self, enable: bool):
        self._check(self._lib.rtma_profile(self._h, ctypes.c_int32(1 if enable else 0)), "rtma_profile")

    def profile_read(self):
        """{class name: (milliseconds, launches)} since the previous read; synchronises."""
        ms = (ctypes.c_double * KERNEL_CLASSES)()
        cnt = (ctypes.c_int64 * KERNEL_CLASSES)()
        self._check(self._lib.rtma_profile_read(self._h, ms, cnt), "rtma_profile_read")
        return {self._lib.rtma_kernel_class_name(ctypes.c_int32(i)).decode(): (float(ms[i]), int(cnt[i]))
                for i in range(KERNEL_CLASSES)}

    # ---- neighbour sampling ---------------------------------------------------------
    def sample_hop(self, rowptr, col, frontier, fanout: int, seed: int, hop: int, stream=None):
        """One hop of the neighbour sampler on one part (rowptr: its n+1 zero-based int64 offsets, col: its
        int32 columns, frontier: ascending distinct int32 local ids).  Returns (block_rowptr, block_col,
        next_frontier), the last two cut to their lengths (which synchronises)."""
        dev = self.device
        _need(rowptr, torch.int64, "rowptr", dev)
        _need(col, torch.int32, "col", dev)
        _need(frontier, torch.int32, "frontier", dev)
        n, fs = int(rowptr.numel()) - 1, int(frontier.numel())
        block_rowptr = torch.empty(fs + 1, dtype=torch.int64, device=dev)
        cap = min(fs * int(fanout), int(col.numel())) if fs else 0
        block_col = torch.empty(max(cap, 1), dtype=torch.int32, device=dev)
        next_frontier = torch.empty(max(n, 1), dtype=torch.int32, device=dev)
        next_size = torch.zeros(1, dtype=torch.int64, device=dev)
        st = self._lib.rtma_sample_hop(
            self._h, ctypes.c_int64(n), _ptr(rowptr), _ptr(col), ctypes.c_int64(fs), _ptr(frontier), ctypes.c_int32(fanout),
            ctypes.c_uint64(seed), ctypes.c_int32(hop), _ptr(block_rowptr), _ptr(block_col), _ptr(next_frontier),
            _ptr(next_size), ctypes.c_void_p(_stream_handle(stream)))
        self._check(st, "rtma_sample_hop")
        return block_rowptr, block_col[:int(block_rowptr[-1].item())], next_frontier[:int(next_size.item())]

    # ---- R1 -------------------------------------------------------------------------
    def partition(self, n: int, group_id, seed: int, M: int, stream=None, grouped: bool = False):
        """Returns (part_id[n] i32, part_offsets[M+1] i64, perm[n] i32, local_id[n] i32).
        grouped: rtma_partition_grouped (inside a part, order by super-node id, then node id)."""
        dev = self.device
        if group_id is not None:
            _need(group_id, torch.int32, "group_id", dev)
        part_id = torch.empty(n, dtype=torch.int32, device=dev)
        part_offsets = torch.empty(M + 1, dtype=torch.int64, device=dev)
        perm = torch.empty(n, dtype=torch.int32, device=dev)
        local_id = torch.empty(n, dtype=torch.int32, device=dev)
        fn = self._lib.rtma_partition_grouped if grouped else self._lib.rtma_partition
        st = fn(self._h, ctypes.c_int64(n), _ptr(group_id), ctypes.c_uint64(seed),
                ctypes.c_int32(M), _ptr(part_id), _ptr(part_offsets), _ptr(perm),
                _ptr(local_id), ctypes.c_void_p(_stream_handle(stream)))
        self._check(st, "rtma_partition_grouped" if grouped else "rtma_partition")
        return part_id, part_offsets, perm, local_id

    def build_induced_csr(self, rowptr, col, M: int, part_id, part_offsets, perm, local_id, stream=None):
        """Count, size, fill.  Returns (rowptr_out[n+M] i64, col_out[E_kept] i32,
        edge_offsets[M+1] i64 (device), kept_cut[2] i64 (device), edge_offsets_host list)."""
        dev = self.device
        n = rowptr.numel() - 1
        is64 = 1 if rowptr.dtype == torch.int64 else 0
        if rowptr.dtype not in (torch.int32, torch.int64):
            raise TypeError("rowptr must be int32 or int64")
        _need(col, torch.int32, "col", dev)
        rowptr_out = torch.empty(n + M, dtype=torch.int64, device=dev)
        edge_offsets = torch.empty(M + 1, dtype=torch.int64, device=dev)
        kept_cut = torch.empty(2, dtype=torch.int64, device=dev)
        s = ctypes.c_void_p(_stream_handle(stream))

        def call(col_out):
            st = self._lib.rtma_build_induced_csr(
                self._h, ctypes.c_int64(n), ctypes.c_int32(is64), _ptr(rowptr), _ptr(col), ctypes.c_int32(M),
                _ptr(part_id), _ptr(part_offsets), _ptr(perm), _ptr(local_id), _ptr(rowptr_out), _ptr(col_out),
                _ptr(edge_offsets), _ptr(kept_cut), s)
            self._check(st, "rtma_build_induced_csr")

        call(None)
        edge_host = edge_offsets.cpu().tolist()  # drains the stream: the size must come back
        col_out = torch.empty(max(edge_host[-1], 1), dtype=torch.int32, device=dev)[:edge_host[-1]]
        if edge_host[-1] > 0:
            call(col_out)
        return rowptr_out, col_out, edge_offsets, kept_cut, edge_host

    def gather_rows(self, src, perm, stream=None):
        n = perm.numel()
        dst = torch.empty((n,) + tuple(src.shape[1:]), dtype=src.dtype, device=self.device)
        row_bytes = src.element_size() * int(src[0].numel()) if src.shape[0] > 0 else src.element_size()
        st = self._lib.rtma_gather_rows(self._h, ctypes.c_int64(n), ctypes.c_int64(row_bytes), _ptr(src),
                                        _ptr(perm), _ptr(dst), ctypes.c_void_p(_stream_handle(stream)))
        self._check(st, "rtma_gather_rows")
        return dst

    # ---- Algorithm 2 ----------------------------------------------------------------
    def local_steps(self, dims, lr, M, part_offsets_host, edge_offsets_host, rowptr_out, col_out, Xp, yp,
                    params, K, loss_out=None, streams=None, gemm_dtype=0, taps=None, symmetric=True,
                    variant=(0, 0, 0), perm=None):
        """K SGD steps on each of the M parts, in place on params [M, P].  K: an int, or a sequence
        of M per-trainer step counts (0 = the trainer does not run; rtma_local_steps_var).
        perm: Xp is the feature matrix in node order and perm the partition's permutation
        (rtma_local_steps_gathered; fixed K only).
        streams: None (all trainers on the current stream), or a list of M torch streams.
        taps: None or (acts tensor or None, grads tensor or None, step).
        variant: (encoder, act, norm) of rtma_model_desc."""
        dev = self.device
        md = model_desc(dims, lr, gemm_dtype, variant)
        _need(params, torch.float32, "params", dev)
        _need(Xp, torch.float32, "Xp", dev)
        _need(yp, torch.int32, "yp", dev)
        _need(rowptr_out, torch.int64, "rowptr_out", dev)
        _need(col_out, torch.int32, "col_out", dev)
        if loss_out is not None:
            _need(loss_out, torch.float32, "loss_out", dev)
        po = (ctypes.c_int64 * (M + 1))(*[int(v) for v in part_offsets_host])
        eo = (ctypes.c_int64 * (M + 1))(*[int(v) for v in edge_offsets_host])
        if streams is None:
            handles = [_stream_handle(None)] * M
        else:
            handles = [_stream_handle(s) for s in streams]
        sarr = (ctypes.c_void_p * M)(*handles)
        tap_struct = None
        if taps is not None:
            acts, grads, step = taps
            tap_struct = Taps(_ptr(acts), _ptr(grads), int(step))
        tap_ref = ctypes.byref(tap_struct) if tap_struct is not None else None
        if perm is not None:
            _need(perm, torch.int32, "perm", dev)
            st = self._lib.rtma_local_steps_gathered(
                self._h, ctypes.byref(md), ctypes.c_int32(M), po, eo, _ptr(rowptr_out), _ptr(col_out),
                ctypes.c_int32(1 if symmetric else 0), _ptr(Xp), _ptr(perm), _ptr(yp), _ptr(params), ctypes.c_int32(int(K)),
                _ptr(loss_out), tap_ref, sarr)
            self._check(st, "rtma_local_steps_gathered")
        elif isinstance(K, int):
            st = self._lib.rtma_local_steps(
                self._h, ctypes.byref(md), ctypes.c_int32(M), po, eo, _ptr(rowptr_out), _ptr(col_out),
                ctypes.c_int32(1 if symmetric else 0), _ptr(Xp), _ptr(yp), _ptr(params), ctypes.c_int32(K),
                _ptr(loss_out), tap_ref, sarr)
            self._check(st, "rtma_local_steps")
        else:
            if len(K) != M:
                raise ValueError("one step count per trainer")
            steps = (ctypes.c_int32 * M)(*[int(v) for v in K])
            stride = int(loss_out.shape[1]) if loss_out is not None else max([int(v) for v in K] + [0])
            st = self._lib.rtma_local_steps_var(
                self._h, ctypes.byref(md), ctypes.c_int32(M), po, eo, _ptr(rowptr_out), _ptr(col_out),
                ctypes.c_int32(1 if symmetric else 0), _ptr(Xp), _ptr(yp), _ptr(params), steps,
                ctypes.c_int32(stride), _ptr(loss_out), tap_ref, sarr)
            self._check(st, "rtma_local_steps_var")

    def link_steps(self, dims, ddims, lr, M, part_offsets_host, edge_offsets_host, rowptr_out, col_out, Xp,
                   pair_offsets_host, pair_u, pair_v, pair_label, params, K, loss_out=None, record_step=-1,
                   grads_out=None, emb_out=None, score_out=None, streams=None, gemm_dtype=0, variant=(0, 0, 0),
                   symmetric=True):
        """K SGD steps of link prediction (encoder `dims` + MLP decoder `ddims`) on the given pairs of
        each part, in place on params [M, P].  pair_u / pair_v / pair_label: int32 device tensors of
        local ids and 0/1 labels, part p's pairs at pair_offsets_host[p]:pair_offsets_host[p+1]."""
        dev = self.device
        md = model_desc(dims, lr, gemm_dtype, variant)
        dd = decoder_desc(ddims)
        _need(params, torch.float32, "params", dev)
        _need(Xp, torch.float32, "Xp", dev)
        _need(rowptr_out, torch.int64, "rowptr_out", dev)
        _need(col_out, torch.int32, "col_out", dev)
        for name, t in (("pair_u", pair_u), ("pair_v", pair_v), ("pair_label", pair_label)):
            _need(t, torch.int32, name, dev)
        po = (ctypes.c_int64 * (M + 1))(*[int(v) for v in part_offsets_host])
        eo = (ctypes.c_int64 * (M + 1))(*[int(v) for v in edge_offsets_host])
        qo = (ctypes.c_int64 * (M + 1))(*[int(v) for v in pair_offsets_host])
        handles = [_stream_handle(None)] * M if streams is None else [_stream_handle(s) for s in streams]
        sarr = (ctypes.c_void_p * M)(*handles)
        st = self._lib.rtma_link_steps(
            self._h, ctypes.byref(md), ctypes.byref(dd), ctypes.c_int32(M), po, eo, _ptr(rowptr_out), _ptr(col_out),
            ctypes.c_int32(1 if symmetric else 0), _ptr(Xp), qo, _ptr(pair_u), _ptr(pair_v), _ptr(pair_label),
            _ptr(params), ctypes.c_int32(K), _ptr(loss_out), ctypes.c_int32(record_step), _ptr(grads_out),
            _ptr(emb_out), _ptr(score_out), sarr)
        self._check(st, "rtma_link_steps")

    # ---- R2 -------------------------------------------------------------------------
    def aggregate(self, params, global_out=None, stream=None):
        M, P = params.shape
        _need(params, torch.float32, "params", self.device)
        st = self._lib.rtma_aggregate(self._h, _ptr(params), ctypes.c_int64(P), ctypes.c_int32(M),
                                      _ptr(global_out), ctypes.c_void_p(_stream_handle(stream)))
        self._check(st, "rtma_aggregate")

    def aggregate_masked(self, params, active, global_out=None, stream=None):
        """Average over the replicas whose entry of `active` (M truthy / falsy values) is set."""
        M, P = params.shape
        _need(params, torch.float32, "params", self.device)
        if len(active) != M:
            raise ValueError("one flag per trainer")
        mask = (ctypes.c_uint8 * M)(*[1 if a else 0 for a in active])
        st = self._lib.rtma_aggregate_masked(self._h, _ptr(params), ctypes.c_int64(P), ctypes.c_int32(M), mask,
                                             _ptr(global_out), ctypes.c_void_p(_stream_handle(stream)))
        self._check(st, "rtma_aggregate_masked")

    def sgd_aggregate(self, params, grads, lr, global_out=None, stream=None):
        M, P = params.shape
        st = self._lib.rtma_sgd_aggregate(self._h, _ptr(params), _ptr(grads), ctypes.c_float(lr),
                                          ctypes.c_int64(P), ctypes.c_int32(M), _ptr(global_out),
                                          ctypes.c_void_p(_stream_handle(stream)))
        self._check(st, "rtma_sgd_aggregate")

    def selftest_wait_timeout(self, stream=None):
        """Launches a kernel whose bounded wait runs out; the next check() raises a timeout error."""
        st = self._lib.rtma_selftest_wait_timeout(self._h, ctypes.c_void_p(_stream_handle(stream)))
        self._check(st, "rtma_selftest_wait_timeout")

    # ---- whole path from host buffers -----------------------------------------------
    def train_host(self, rowptr, col, X, y, dims, M, K, R, lr, seed, params0, group_id=None, gemm_dtype=0,
                   variant=(0, 0, 0)):
        """The whole path on HOST (numpy) buffers: copies the inputs to the device, runs
        partition, induced CSR, row gather, R rounds of (K local steps + aggregation), and
        copies the result back.  Returns (params[P] f32, losses[R, M, K] f32, kept, cut)."""
        import numpy as np
        rowptr = np.ascontiguousarray(rowptr)
        is64 = 1 if rowptr.dtype == np.int64 else 0
        if rowptr.dtype not in (np.int32, np.int64):
            raise TypeError("rowptr must be int32 or int64")
        col = np.ascontiguousarray(col, dtype=np.int32)
        X = np.ascontiguousarray(X, dtype=np.float32)
        y = np.ascontiguousarray(y, dtype=np.int32)
        params0 = np.ascontiguousarray(params0, dtype=np.float32)
        gid = None if group_id is None else np.ascontiguousarray(group_id, dtype=np.int32)
        n = rowptr.size - 1
        md = model_desc(dims, lr, gemm_dtype, variant)
        out = np.empty(params0.size, dtype=np.float32)
        losses = np.empty((R, M, K), dtype=np.float32)
        kept_cut = np.empty(2, dtype=np.int64)
        vp = lambda a: ctypes.c_void_p(0) if a is None else ctypes.c_void_p(a.ctypes.data)
        st = self._lib.rtma_train_host(
            self._h, ctypes.c_int64(n), ctypes.c_int32(is64), vp(rowptr), vp(col), vp(gid), vp(X), vp(y),
            ctypes.byref(md), ctypes.c_int32(M), ctypes.c_uint64(seed), ctypes.c_int32(K), ctypes.c_int32(R),
            vp(params0), vp(out), vp(losses), vp(kept_cut), ctypes.c_void_p(_stream_handle(None)))
        self._check(st, "rtma_train_host")
        return out, losses, int(kept_cut[0]), int(kept_cut[1])
