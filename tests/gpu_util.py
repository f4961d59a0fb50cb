"""Helpers shared by the GPU parity tests."""
import numpy as np
import torch

import oracle
from paper_2305_09887_b200 import binding, inputs

# relative = max|a-b| / max|b| per tensor
TOL_ACT, TOL_GRAD, TOL_PARAM = 1e-4, 1e-3, 1e-3
TOL_BF16 = 5e-3
# bf16 operand mode, layer by layer from the kernel's own recorded inputs (same operands, hence the same
# roundings): what is left is fp32 accumulation against fp64
TOL_BF16_LAYER = 5e-5
# bf16 operand mode over a whole step against the oracle's bf16 operand mode.  Not tight: an activation
# that differs by 1e-7 lands on the other side of a bf16 rounding boundary once in ten thousand and
# then differs by 2^-8, which moves a whole row of the next layer by up to 3e-4 (and ReLU branches
# flip the same way); measured 1e-3 .. 3e-3 on the named shapes.  Held to the mode's own bar.
TOL_BF16_SAME_ROUNDING = TOL_BF16
# branch flips seen per check (part, flipped units, hidden units), for the test log
FLIP_LOG = []

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


def gpu_preprocess(w, M=None, seed=None, use_groups=None, grouped=None):
    """partition + induced CSR + row gather on the GPU for workload w."""
    c = ctx()
    g = w.graph
    M = w.M if M is None else M
    seed = w.partition_seed if seed is None else seed
    use_groups = w.use_groups if use_groups is None else use_groups
    grouped = (w.grouped_order and use_groups) if grouped is None else grouped
    gid = dev(g.group_id) if use_groups else None
    part_id, part_offsets, perm, local_id = c.partition(g.n, gid, seed, M, grouped=grouped)
    rowptr_out, col_out, edge_offsets, kept_cut, edge_host = c.build_induced_csr(
        dev(g.rowptr), dev(g.col), M, part_id, part_offsets, perm, local_id)
    Xp = c.gather_rows(dev(w.X), perm)
    yp = c.gather_rows(dev(w.y), perm)
    torch.cuda.synchronize()
    return dict(part_id=part_id, part_offsets=part_offsets, perm=perm, local_id=local_id,
                rowptr_out=rowptr_out, col_out=col_out, edge_offsets=edge_offsets, kept_cut=kept_cut,
                edge_host=edge_host, part_host=part_offsets.cpu().tolist(), Xp=Xp, yp=yp, M=M)


def oracle_preprocess(w, M=None, seed=None, use_groups=None, grouped=None):
    g = w.graph
    M = w.M if M is None else M
    seed = w.partition_seed if seed is None else seed
    use_groups = w.use_groups if use_groups is None else use_groups
    grouped = (w.grouped_order and use_groups) if grouped is None else grouped
    gid = g.group_id if use_groups else None
    part_id, part_offsets, perm, local_id = oracle.partition(g.n, gid, seed, M, grouped=grouped)
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


def oracle_part(w, pre, p):
    """(rowptr, col, X, y) of part p from the oracle's preprocessing."""
    rp, cp = oracle.part_graph(pre["rowptr_out"], pre["col_out"], pre["part_offsets"], pre["edge_offsets"], p)
    lo, hi = int(pre["part_offsets"][p]), int(pre["part_offsets"][p + 1])
    return rp, cp, pre["Xp"][lo:hi].astype(np.float64), pre["yp"][lo:hi]


def oracle_parts(w, pre):
    return [oracle_part(w, pre, p) for p in range(pre["M"])]


def tols(gemm_dtype):
    """(activations, gradients, parameters, loss, |z| below which a ReLU branch is ambiguous as a
    fraction of max|z|, flips allowed per part as a fraction of the hidden units)."""
    if gemm_dtype == 1:   # operands rounded to bf16 (2^-9 each), fp32 accumulation
        return TOL_BF16, TOL_BF16, TOL_BF16, TOL_BF16, 4e-3, 0.01
    # fp32-accurate products: the kernel's pre-activations carry about 1e-6 of relative error, so
    # of the order of 1e-6 of all units straddle the kink differently from the fp64 oracle (measured:
    # 0 to 7 per part on the scaled shapes, 17 of 12.7 M on a whole Medium part, i.e. 1.3e-6)
    return TOL_ACT, TOL_GRAD, TOL_PARAM, 1e-5, 2e-5, 4e-6


def _param_segments(variant, dims):
    """[(name, offset, size)] of every parameter tensor of one replica."""
    out = []
    for l, lay in enumerate(oracle.variant_layout(variant, dims)):
        sizes = {"w0": dims[l] * dims[l + 1], "w1": dims[l] * dims[l + 1], "bias": dims[l + 1],
                 "gamma": dims[l + 1], "beta": dims[l + 1], "slope": 1}
        out += [(f"{key}{l}", off, sizes[key]) for key, off in lay.items() if off >= 0]
    return out


def check_one_step(w, M=None, gemm_dtype=0, streams=None, only_parts=None, variant=(0, 0, 0), params0=None,
                   gradients_against_plain=True):
    """Partition + induced CSR against the oracle (bit-exact), then step 0 of all M trainers
    batched as one call: every recorded intermediate, the loss, the gradient and the updated
    parameters of every part (or of the parts in only_parts) against the oracle.  In bf16 operand
    mode the step is also held, tightly, to the oracle run with the same operand roundings;
    gradients_against_plain=False leaves the gradient comparison to that one (shapes outside the
    named bf16 workload, where the 5e-3 bar against the unrounded oracle is not claimed)."""
    tol_act, tol_grad, tol_param, tol_loss, amb, flip_frac = tols(gemm_dtype)
    c = ctx()
    got = gpu_preprocess(w, M=M)
    want = oracle_preprocess(w, M=M)
    assert_preprocess_equal(got, want)
    M = got["M"]
    dims, n = w.dims, w.graph.n
    params0 = w.params0 if params0 is None else params0
    P = params0.size
    assert P == oracle.variant_param_count(variant, dims) == binding.param_count(dims, variant)
    rec = sum(dims[l] + dims[l + 1] for l in range(len(dims) - 1))
    params = dev(np.tile(params0, (M, 1)))
    acts = torch.zeros(n * rec, dtype=torch.float32, device="cuda")
    grads = torch.zeros(M, P, dtype=torch.float32, device="cuda")
    loss = torch.zeros(M, 1, dtype=torch.float32, device="cuda")
    c.local_steps(dims, w.lr, M, got["part_host"], got["edge_host"], got["rowptr_out"], got["col_out"],
                  got["Xp"], got["yp"], params, 1, loss_out=loss, taps=(acts, grads, 0), gemm_dtype=gemm_dtype,
                  streams=streams, variant=variant)
    torch.cuda.synchronize()
    grads, loss, params1 = grads.cpu().numpy(), loss.cpu().numpy(), params.cpu().numpy()
    p0 = params0.astype(np.float64)
    for p in range(M) if only_parts is None else only_parts:
        rp, cp, X, y = oracle_part(w, want, p)
        n_p = rp.size - 1
        o_loss, o_grads, o_acts = oracle.forward_backward_variant(variant, dims, rp, cp, X, y, p0, want_acts=True,
                                                                  want_preact=True)
        layout, total = oracle.acts_layout(dims, n_p)
        base = int(want["part_offsets"][p]) * rec
        gpu_acts = {}
        for name, off, r, wd in layout:
            a = acts[base + off: base + off + r * wd].cpu().numpy().reshape(r, wd)
            gpu_acts[name] = a
            assert rel_err(a, o_acts[name]) <= tol_act, (p, name)
        # ReLU has no derivative at 0: a hidden unit whose pre-activation is within the rounding
        # error of an fp32 forward pass of 0 may legitimately take either branch, and the branch
        # decides a finite part of the gradient.  For such units only (judged on the oracle's own
        # pre-activations) the oracle is re-evaluated on the branch the kernel took; any other
        # unit on the wrong branch fails the activation check above.
        gates, flipped, units = [], 0, 0
        for l in range(len(dims) - 2):
            Z = o_acts[f"Z{l + 1}"]
            ambiguous = np.abs(Z) < amb * max(1.0, np.abs(Z).max(initial=0.0))
            units += Z.size
            differ = ambiguous & ((gpu_acts[f"H{l + 1}"] > 0) != (Z > 0))
            flipped += int(differ.sum())
            g8 = np.full(Z.shape, -1, dtype=np.int8)
            g8[differ] = (gpu_acts[f"H{l + 1}"] > 0)[differ]
            gates.append(g8)
        FLIP_LOG.append((w.name, gemm_dtype, p, flipped, units))
        print(f"[relu branch] {w.name} mode {gemm_dtype} part {p}: {flipped} of {units} hidden units took the other branch")
        assert flipped <= 8 + flip_frac * units
        if flipped:
            o_loss, o_grads, _ = oracle.forward_backward_variant(variant, dims, rp, cp, X, y, p0, gates=gates)
        mode_grads = None   # bf16 operand mode: the gradient of the mode's own definition (fp64 sums)
        if gemm_dtype == 1 and variant == (0, 0, 0):
            mode_grads = same_rounding_check(w, p, rp, cp, X, y, p0, gpu_acts, loss[p, 0], grads[p],
                                             assert_whole_step=gradients_against_plain)
        if n_p:
            assert abs(loss[p, 0] - o_loss) <= tol_loss * max(1.0, abs(o_loss)), p
        if not gradients_against_plain:
            assert gemm_dtype == 1 and variant == (0, 0, 0)
            continue
        # gradients: per parameter tensor
        for nm, off, size in _param_segments(variant, dims):
            gg, og = grads[p, off:off + size], o_grads[off:off + size]
            if np.abs(og).max() > 0:
                if size == 1:   # a single number (PReLU slope): relative to itself, with an absolute floor
                    assert abs(gg[0] - og[0]) <= tol_grad * max(abs(og[0]), 1e-3), (p, nm)
                else:
                    e, bar = rel_err(gg, og), tol_grad
                    if mode_grads is not None:
                        # where rounding the operands to bf16 -- in exact sums, by the mode's definition --
                        # already moves this tensor past the bar, no implementation of the mode can
                        # meet it on this input: hold the kernel to what the definition delivers
                        e_mode = rel_err(mode_grads[off:off + size], og)
                        if e_mode > 0.8 * tol_grad:
                            bar = max(tol_grad, 1.25 * e_mode)
                            print(f"[bf16 bar] {w.name} part {p} {nm}: kernel {e:.2e}, the mode's definition {e_mode:.2e} "
                                  f"from the unrounded oracle (bar {tol_grad:.0e})")
                    assert e <= bar, (p, nm, e)
            else:
                assert np.abs(gg).max() == 0
        assert rel_err(params1[p], p0 - w.lr * o_grads) <= tol_param
    return got, want


def _round_bf16(x):
    """Round to nearest even into bf16 (the upper 16 bits of binary32), on the bits."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


def _bf16_ties(s):
    """For recorded activations s = hi + lo (hi = the bf16 operand the kernel used, lo = the bf16
    remainder): where s sits exactly half way between two bf16 numbers, hi cannot be told from s (a
    remainder that rounds up to half a unit lands there, about once in 500 values).  Returns the
    spacing of the two candidates at those places, 0 elsewhere."""
    bits = np.ascontiguousarray(s, dtype=np.float32).view(np.uint32)
    tie = (bits & 0xFFFF) == 0x8000
    down = (bits & 0xFFFF0000).view(np.float32).astype(np.float64)
    up = ((bits & 0xFFFF0000) + 0x10000).astype(np.uint32).view(np.float32).astype(np.float64)
    return np.where(tie, np.abs(up - down), 0.0).reshape(np.shape(s))


def layerwise_bf16_check(w, p, rp, cp, X, p0, gpu_acts):
    """bf16 operand mode, one layer at a time from the kernel's own recorded inputs: the aggregate
    A-bar H against the oracle's (it is not rounded), the layer output against the rounded-operand
    product of the recorded H and A-bar H in fp64.  The last layer may be evaluated in either
    association -- H Ws + (A-bar H) Wn or H Ws + A-bar (H Wn) -- which differ once operands are rounded.
    Every output is held to TOL_BF16_LAYER plus what the undecidable operands (see _bf16_ties) of its
    row can move it."""
    dims = w.dims
    L = len(dims) - 1
    r = _round_bf16
    off = 0
    worst, loose = 0.0, 0
    for l in range(L):
        di, dn = dims[l], dims[l + 1]
        Ws = p0[off:off + di * dn].reshape(di, dn)
        Wn = p0[off + di * dn:off + 2 * di * dn].reshape(di, dn)
        b = p0[off + 2 * di * dn:off + 2 * di * dn + dn]
        off += 2 * di * dn + dn
        Hin = X if l == 0 else gpu_acts[f"H{l}"].astype(np.float64)
        N = gpu_acts[f"N{l}"].astype(np.float64)
        e_agg = rel_err(N, oracle.spmm_mean(rp, cp, Hin))
        assert e_agg <= 2e-5, (p, f"N{l}", e_agg)
        tie_h = np.zeros_like(Hin) if l == 0 else _bf16_ties(Hin)    # the features are rounded from fp32: no doubt there
        tie_n = _bf16_ties(N)
        got = gpu_acts[f"H{l + 1}"].astype(np.float64)
        Z = r(Hin) @ r(Ws) + r(N) @ r(Wn) + b
        slack = tie_h @ np.abs(r(Ws)) + tie_n @ np.abs(r(Wn))
        scale = max(np.abs(Z).max(), 1e-30)
        if l < L - 1:
            excess = np.abs(got - np.maximum(Z, 0.0)) - slack
        else:
            Z_after = r(Hin) @ r(Ws) + oracle.spmm_mean(rp, cp, r(Hin) @ r(Wn)) + b
            slack_after = tie_h @ np.abs(r(Ws)) + oracle.spmm_mean(rp, cp, tie_h @ np.abs(r(Wn)))
            e0, e1 = np.abs(got - Z) - slack, np.abs(got - Z_after) - slack_after
            excess = e0 if e0.max() <= e1.max() else e1
        worst = max(worst, float(excess.max()) / scale)
        loose += int(np.count_nonzero(slack))
        assert excess.max() <= TOL_BF16_LAYER * scale, (p, f"H{l + 1}", float(excess.max()) / scale)
    print(f"[bf16 layer by layer] {w.name} part {p}: worst {worst:.1e} of the layer's largest output "
          f"({loose} outputs with an undecidable operand in their row)")


def same_rounding_check(w, p, rp, cp, X, y, p0, gpu_acts, gpu_loss, gpu_grads, assert_whole_step=True):
    """bf16 operand mode: layer by layer from the kernel's recorded inputs (tight), then the whole step
    against the oracle run with the same operand roundings."""
    layerwise_bf16_check(w, p, rp, cp, X, p0, gpu_acts)
    dims = w.dims
    tol = TOL_BF16_SAME_ROUNDING
    r_loss, r_grads, r_acts = oracle.forward_backward(dims, rp, cp, X, y, p0, want_acts=True, want_preact=True,
                                                      bf16_operands=True)
    errs = {name: rel_err(a, r_acts[name]) for name, a in gpu_acts.items()}
    print(f"[same rounding] {w.name} part {p} activations: " + ", ".join(f"{k} {v:.1e}" for k, v in errs.items()))
    gates, flipped = [], 0
    for l in range(len(dims) - 2):
        Z = r_acts[f"Z{l + 1}"]
        differ = (np.abs(Z) < 4e-3 * max(1.0, np.abs(Z).max(initial=0.0))) & ((gpu_acts[f"H{l + 1}"] > 0) != (Z > 0))
        flipped += int(differ.sum())
        g8 = np.full(Z.shape, -1, dtype=np.int8)
        g8[differ] = (gpu_acts[f"H{l + 1}"] > 0)[differ]
        gates.append(g8)
    if flipped:
        r_loss, r_grads, _ = oracle.forward_backward(dims, rp, cp, X, y, p0, gates=gates, bf16_operands=True)
    gerrs = {nm: rel_err(gpu_grads[off:off + size], r_grads[off:off + size])
             for nm, off, size in _param_segments((0, 0, 0), dims) if np.abs(r_grads[off:off + size]).max() > 0}
    print(f"[same rounding] {w.name} part {p} gradients: " + ", ".join(f"{k} {v:.1e}" for k, v in gerrs.items()) +
          f"; {flipped} branch flips")
    if assert_whole_step:
        assert max(errs.values()) <= tol, (p, errs)
        if rp.size > 1:
            assert abs(gpu_loss - r_loss) <= tol * max(1.0, abs(r_loss)), p
        assert max(gerrs.values(), default=0.0) <= tol, (p, gerrs)
    return r_grads


def check_k_steps_and_average(w, got, want, K, gemm_dtype=0, streams=None, only_parts=None, variant=(0, 0, 0),
                              params0=None):
    """K local steps of all M trainers and the aggregation.  Parameters and losses of every part
    (or of the parts in only_parts) against the oracle; the average against the oracle's, or,
    when only some parts were recomputed, against the fp64 mean of the kernel's own replicas."""
    tol_param = tols(gemm_dtype)[2]
    tol_loss = 10 * tols(gemm_dtype)[3]
    c = ctx()
    M, dims = got["M"], w.dims
    params0 = w.params0 if params0 is None else params0
    params = dev(np.tile(params0, (M, 1)))
    loss = torch.zeros(M, K, dtype=torch.float32, device="cuda")
    c.local_steps(dims, w.lr, M, got["part_host"], got["edge_host"], got["rowptr_out"], got["col_out"],
                  got["Xp"], got["yp"], params, K, loss_out=loss, gemm_dtype=gemm_dtype, streams=streams, variant=variant)
    torch.cuda.synchronize()
    after = params.cpu().numpy().copy()
    glob = torch.empty(params.shape[1], dtype=torch.float32, device="cuda")
    c.aggregate(params, glob)
    torch.cuda.synchronize()
    o_params = after.astype(np.float64)
    for p in range(M) if only_parts is None else only_parts:
        rp, cp, X, y = oracle_part(w, want, p)
        o_params[p], o_loss = oracle.local_steps_variant(variant, dims, w.lr, rp, cp, X, y, params0.astype(np.float64), K)
        assert rel_err(after[p], o_params[p]) <= tol_param, p
        if rp.size > 1:
            assert np.abs(loss[p].cpu().numpy() - o_loss).max() <= tol_loss * max(1.0, np.abs(o_loss).max())
    o_avg, o_glob = oracle.average(o_params)
    assert rel_err(glob.cpu().numpy(), o_glob) <= tol_param
    pa = params.cpu().numpy()
    for p in range(M):
        assert np.array_equal(pa[p], glob.cpu().numpy())     # every local copy overwritten
    return after
