"""Comparison rules between the CUDA path and the oracle (test infrastructure).

Tolerances (from the target: aggregate and updated params max relative error <= 1e-5 for fp32
gradients, <= 4e-3 for bf16 gradients; scalar statistics relative error <= 1e-4), with
"relative" made well defined near zero:
  - per-element vectors: |gpu - ref| <= tol_v * max(|ref|, cond), cond being the forward-error
    scale of the sum that produced the element (sum_k w_k |x_k| for the aggregate, and so on);
  - positive sums: plain relative error <= tol_s;
  - differences (|G|^2^, <g,a>): error judged against the size of the terms (A, sqrt(A |a|^2));
  - cosine: absolute <= tol_s;
  - ratios (gns, sigma): tol_s scaled by the conditioning of the ratio, and only when the
    denominator is not itself a cancelled difference.
"""
import numpy as np

HDR = 16
TOL_S = 1e-4
TOL_V = {0: 1e-5, 1: 4e-3}


def cond_vectors(grads_f32, b, params_in, momentum_in, lr, beta):
    """Forward-error scales of g, m', theta' (float64 arrays)."""
    w = np.asarray(b, np.float64) / float(np.sum(b))
    cg = np.zeros(len(params_in), np.float64)
    for k, x in enumerate(grads_f32):
        cg += w[k] * np.abs(x.astype(np.float64))
    cm = np.abs(float(np.float32(beta)) * momentum_in.astype(np.float64)) + cg
    ct = np.abs(params_in.astype(np.float64)) + abs(float(np.float32(lr))) * cm
    return cg, cm, ct


def cond_vectors_adam(grads_f32, b, params_in, m_in, v_in, lr, beta1, beta2, eps, t, with_update=False):
    """Forward-error scales of g, m', v', theta' under the Adam update (float64 arrays). With
    with_update also |u| and the scale cu of the update u = mhat/(sqrt(vhat)+eps) itself."""
    w = np.asarray(b, np.float64) / float(np.sum(b))
    cg = np.zeros(len(params_in), np.float64)
    g = np.zeros(len(params_in), np.float64)
    for k, x in enumerate(grads_f32):
        cg += w[k] * np.abs(x.astype(np.float64))
        g += w[k] * x.astype(np.float64)
    b1, b2 = float(np.float32(beta1)), float(np.float32(beta2))
    cm = np.abs(b1 * m_in.astype(np.float64)) + (1 - b1) * cg
    cv = b2 * np.abs(v_in.astype(np.float64)) + (1 - b2) * 2 * cg * cg
    c1, c2 = 1 / (1 - b1 ** t), 1 / (1 - b2 ** t)
    m_new = b1 * m_in.astype(np.float64) + (1 - b1) * g
    v_new = b2 * v_in.astype(np.float64) + (1 - b2) * g * g
    root = np.sqrt(v_new * c2)
    den = root + float(np.float32(eps))
    u = m_new * c1 / np.maximum(den, 1e-300)
    cu = c1 * cm / np.maximum(den, 1e-300) + np.abs(u) * c2 * cv / np.maximum(2 * root * den, 1e-300)
    ct = np.abs(params_in.astype(np.float64)) + abs(float(np.float32(lr))) * (np.abs(u) + cu)
    if with_update:
        return cg, cm, cv, ct, np.abs(u), cu
    return cg, cm, cv, ct


def check_vectors_adam(dtype, gpu_vecs, ref_vecs, conds, what=""):
    tol = TOL_V[dtype]
    errs = {}
    for name, g, r, c in zip(("agg", "first_moment", "second_moment", "params"), gpu_vecs, ref_vecs, conds):
        e = vec_err(g, r, c)
        errs[name] = e
        assert e <= tol, "%s %s: max scaled error %.3e > %.1e" % (what, name, e, tol)
    return errs


def vec_err(gpu, ref, cond):
    """max over elements of |gpu-ref| / max(|ref|, cond) (0/0 counts as 0)."""
    gpu = gpu.astype(np.float64); ref = ref.astype(np.float64)
    den = np.maximum(np.abs(ref), cond)
    diff = np.abs(gpu - ref)
    with np.errstate(divide="ignore", invalid="ignore"):
        r = np.where(den > 0, diff / den, np.where(diff == 0, 0.0, np.inf))
    return float(r.max()) if r.size else 0.0


def check_vectors(dtype, gpu_vecs, ref_vecs, conds, what=""):
    tol = TOL_V[dtype]
    errs = {}
    for name, g, r, c in zip(("agg", "momentum", "params"), gpu_vecs, ref_vecs, conds):
        e = vec_err(g, r, c)
        errs[name] = e
        assert e <= tol, "%s %s: max scaled error %.3e > %.1e" % (what, name, e, tol)
    return errs


def seg_scales(cg, seg, lo=0):
    """sum_{j in s} cond_j^2 per segment, for the elements [lo, lo+len(cg)) this call covers."""
    cs = np.concatenate([[0.0], np.cumsum(cg.astype(np.float64) ** 2)])
    idx = np.clip(np.asarray(seg, np.int64) - lo, 0, len(cg))
    return cs[idx[1:]] - cs[idx[:-1]]


SMALL_SEGMENT = 64      # segments shorter than this may use the per-element floor on N_s


def check_state(gpu, ref, K, S, seg, b, what="", tol=TOL_S, seg_scale=None, adam=False):
    """Compare two out_state vectors (float32 arrays). Returns the max relative error seen.

    seg_scale[s] = sum_{j in s} cond_j^2: a segment of a few elements inherits the forward
    error of its elements (an element's g_j may be a cancelling sum), so N_s of a segment of
    fewer than SMALL_SEGMENT elements is allowed 2e-5 * seg_scale[s] on top of tol * N_s (fp32
    arithmetic on exactly widened inputs). Longer segments get the plain relative bound only."""
    gpu = gpu.astype(np.float64); ref = ref.astype(np.float64)
    seg = np.asarray(seg)
    worst = 0.0

    def rel(i, name, scale=None, t=tol):
        nonlocal worst
        s = abs(ref[i]) if scale is None else scale
        d = abs(gpu[i] - ref[i])
        if s == 0:
            assert d == 0, "%s %s: ref 0, gpu %r" % (what, name, gpu[i])
            return
        worst = max(worst, d / s)
        assert d <= t * s, "%s %s: gpu %.9g ref %.9g rel %.3e > %.1e" % (what, name, gpu[i], ref[i], d / s, t)

    B, A, trS, G2, pp = ref[0], ref[1], ref[2], ref[3], ref[7]
    q_ref = ref[HDR:HDR + K]
    Qw = float(np.dot(np.asarray(b, np.float64), q_ref))
    assert gpu[0] == ref[0], "%s B_total" % what
    if not np.all(np.isfinite(ref[:HDR + K])):
        # non-finite data: only the flag and the finiteness pattern are compared
        assert int(gpu[11]) & 1 and int(ref[11]) & 1, "%s non-finite flag" % what
        assert np.array_equal(np.isfinite(gpu[HDR:HDR + K]), np.isfinite(q_ref)), "%s q finiteness" % what
        return worst
    rel(1, "agg_sqnorm")
    if trS == 0 and K > 1:      # identical workers
        assert abs(gpu[2]) <= 1e-6 * Qw / (K - 1), "%s tr_sigma should vanish: %r" % (what, gpu[2])
    else:
        rel(2, "tr_sigma")
    rel(3, "g2_hat", scale=max(A, abs(G2)))
    rel(6, "dot_prev", scale=max(np.sqrt(A * pp), abs(ref[6])) if A * pp > 0 else None)
    rel(7, "prev_sqnorm")
    assert abs(gpu[5] - ref[5]) <= tol, "%s cos_prev gpu %.9g ref %.9g" % (what, gpu[5], ref[5])
    rel(10, "wmean_worker_sqnorm")
    if G2 >= 1e-3 * A and G2 > 0:
        rel(4, "gns", t=tol * (1 + A / G2)) if trS > 0 else None
    if A > 0 and trS > 0:
        rel(8, "sigma2_norm", t=2 * tol)
        rel(9, "sigma_norm", t=2 * tol)
    # flags: must match unless the reference sits on a threshold
    fg, fr = int(gpu[11]), int(ref[11])
    assert not fg & 16, "%s internal-error flag set (a bounded wait ran out)" % what
    assert not fg & 32, "%s range-check flag set (checked build: an index was out of range)" % what
    mask = 1 | 4 | 8
    if abs(G2) > tol * max(A, 1e-300):
        mask |= 2
    assert (fg & mask) == (fr & mask), "%s flags gpu %d ref %d" % (what, fg, fr)
    if adam:
        # mean, variance, std of ghat = g/(sqrt(vhat)+eps) over the parameters: judged against its rms
        rms2 = ref[13] + ref[12] ** 2
        assert abs(gpu[12] - ref[12]) <= tol * np.sqrt(rms2), "%s ghat mean gpu %.9g ref %.9g" % (what, gpu[12], ref[12])
        assert abs(gpu[13] - ref[13]) <= 2 * tol * rms2, "%s ghat var gpu %.9g ref %.9g" % (what, gpu[13], ref[13])
        if ref[13] > 1e-3 * rms2:
            assert abs(gpu[14] - ref[14]) <= 2 * tol * np.sqrt(rms2), "%s ghat std gpu %.9g ref %.9g" % (what, gpu[14], ref[14])
        assert gpu[15] == 0
    else:
        assert np.all(gpu[12:16] == 0)
    for k in range(K):
        rel(HDR + k, "worker_sqnorm[%d]" % k)
    for s in range(S):
        empty = seg[s] == seg[s + 1]
        iv, inn = HDR + K + s, HDR + K + S + s
        if empty:
            assert gpu[iv] == 0 and gpu[inn] == 0, "%s empty segment %d not zero" % (what, s)
            continue
        if ref[iv] == 0 and K > 1:
            assert abs(gpu[iv]) <= 1e-6 * Qw / (K - 1), "%s seg_var[%d] should vanish" % (what, s)
        else:
            rel(iv, "seg_var[%d]" % s)
        small = seg[s + 1] - seg[s] < SMALL_SEGMENT
        floor = 2e-5 * float(seg_scale[s]) if (seg_scale is not None and small) else 0.0
        if abs(gpu[inn] - ref[inn]) > floor:
            rel(inn, "seg_agg_sqnorm[%d]" % s)
    return worst


def grads_to_host(torch, grads, dtype, lo=None, hi=None):
    """Device gradient tensors -> numpy arrays in the oracle's storage format; second list
    holds the values widened to float32."""
    raw, wide = [], []
    for g in grads:
        t = g if lo is None else g[lo:hi]
        if dtype == 0:
            a = t.cpu().numpy()
            raw.append(a); wide.append(a)
        else:
            a = t.view(torch.int16).cpu().numpy().view(np.uint16)
            raw.append(a)
            wide.append((a.astype(np.uint32) << np.uint32(16)).view(np.float32))
    return raw, wide


# ---- the same scales and errors on torch tensors (any device), for problems too large for numpy ----

def cond_vectors_t(torch, grads, b, params_in, momentum_in, lr, beta):
    """cond_vectors on torch tensors: gradients as stored (fp32 or bf16 tensors, widened
    exactly), state as fp32 tensors; returns float64 tensors on the gradients' device."""
    w = np.asarray(b, np.float64) / float(np.sum(b))
    cg = torch.zeros(grads[0].numel(), dtype=torch.float64, device=grads[0].device)
    for k, x in enumerate(grads):
        cg.add_(x.abs().to(torch.float64), alpha=float(w[k]))
    cm = momentum_in.to(torch.float64).mul_(float(np.float32(beta))).abs_().add_(cg)
    ct = params_in.to(torch.float64).abs_().add_(cm, alpha=abs(float(np.float32(lr))))
    return cg, cm, ct


def cond_vectors_adam_t(torch, grads, b, params_in, m_in, v_in, lr, beta1, beta2, eps, t):
    """cond_vectors_adam (without the update's own scales) on torch tensors: gradients as stored
    (fp32 or bf16 tensors, widened exactly), state as fp32 tensors; float64 tensors on their device."""
    w = np.asarray(b, np.float64) / float(np.sum(b))
    n, dev = grads[0].numel(), grads[0].device
    cg = torch.zeros(n, dtype=torch.float64, device=dev)
    g = torch.zeros(n, dtype=torch.float64, device=dev)
    for k, x in enumerate(grads):
        x64 = x.to(torch.float64)
        g.add_(x64, alpha=float(w[k]))
        cg.add_(x64.abs_(), alpha=float(w[k]))
    b1, b2 = float(np.float32(beta1)), float(np.float32(beta2))
    m64, v64 = m_in.to(torch.float64), v_in.to(torch.float64)
    cm = (b1 * m64).abs_() + (1 - b1) * cg
    cv = b2 * v64.abs() + (1 - b2) * 2 * cg * cg
    c1, c2 = 1 / (1 - b1 ** t), 1 / (1 - b2 ** t)
    m_new = b1 * m64 + (1 - b1) * g
    v_new = b2 * v64 + (1 - b2) * g * g
    root = torch.sqrt(v_new * c2)
    den = root + float(np.float32(eps))
    tiny = torch.full_like(den, 1e-300)
    u = m_new * c1 / torch.maximum(den, tiny)
    cu = c1 * cm / torch.maximum(den, tiny) + u.abs() * c2 * cv / torch.maximum(2 * root * den, tiny)
    ct = params_in.to(torch.float64).abs_() + abs(float(np.float32(lr))) * (u.abs() + cu)
    return cg, cm, cv, ct


def seg_scales_range_t(torch, cg, seg, lo):
    """seg_scales with an offset on a torch tensor: the elements [lo, lo + len(cg)) of the problem."""
    cs = torch.cat([torch.zeros(1, dtype=torch.float64, device=cg.device), torch.cumsum(cg * cg, 0)])
    idx = torch.as_tensor(np.clip(np.asarray(seg, np.int64) - lo, 0, cg.numel()), device=cg.device)
    return (cs[idx[1:]] - cs[idx[:-1]]).cpu().numpy()


def vec_err_t(torch, gpu, ref, cond):
    """vec_err on torch tensors (fp32 values, float64 scale)."""
    ref64 = ref.to(torch.float64)
    diff = (gpu.to(torch.float64) - ref64).abs_()
    den = torch.maximum(ref64.abs_(), cond)
    r = torch.where(den > 0, diff / den, torch.where(diff == 0, torch.zeros_like(diff), torch.full_like(diff, float("inf"))))
    return float(r.max()) if r.numel() else 0.0


def seg_scales_t(torch, cg, seg):
    """seg_scales on a torch tensor; returns a numpy array."""
    cs = torch.cat([torch.zeros(1, dtype=torch.float64, device=cg.device), torch.cumsum(cg * cg, 0)])
    idx = torch.as_tensor(np.asarray(seg, np.int64), device=cg.device)
    return (cs[idx[1:]] - cs[idx[:-1]]).cpu().numpy()
