"""Parity of dmx_step_adam (through the C ABI) with the oracle's Adam mode. Needs a GPU."""
import os

import numpy as np
import pytest

from oracle.dmx_oracle import Oracle
from paper_2510_08522_b200 import workload as W
from tests import parity as PT

pytestmark = pytest.mark.gpu
NTHREADS = max(1, min(32, os.cpu_count() or 1))
LR, B1, B2, EPS = 1e-3, 0.9, 0.999, 1e-8


def _torch():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return torch


def lock_step_adam(wl, steps, v0=0.0):
    torch = _torch()
    import paper_2510_08522_b200 as D
    dp = W.DeviceProblem(wl)
    second = torch.full((wl.P,), v0, dtype=torch.float32, device="cuda")
    orc = Oracle(wl.K, wl.P, dp.seg, wl.dtype)
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    worst = {}
    for t in range(1, steps + 1):
        # Lock step: the oracle starts every step from the CUDA path's state. Adam's update is
        # sign-like where |g| is near eps, so an element whose aggregate cancels to ~0 takes a
        # legitimately different step on the two sides (its forward-error scale says so) and a
        # free-running comparison would carry that difference in theta for ever.
        hp, hm, hv, ha = (x.cpu().numpy().copy() for x in (dp.params, dp.momentum, second, dp.prev_agg))
        b = dp.fill()
        raw, wide = PT.grads_to_host(torch, dp.grads, wl.dtype)
        conds = PT.cond_vectors_adam(wide, b, hp, hm, hv, LR, B1, B2, EPS, t)
        ref = orc.step_adam(raw, b, hp, hm, hv, LR, B1, B2, EPS, t, ha, nthreads=NTHREADS)
        st = d.step_adam(dp.grads, b, dp.params, dp.momentum, second, LR, B1, B2, EPS, t, dp.prev_agg)
        torch.cuda.synchronize()
        what = "%s adam step %d" % (wl.name, t)
        e = PT.check_vectors_adam(wl.dtype, tuple(x.cpu().numpy() for x in (dp.prev_agg, dp.momentum, second, dp.params)),
                                  (ha, hm, hv, hp), conds, what)
        e["state"] = PT.check_state(st.cpu().numpy(), ref, wl.K, wl.S, dp.seg, b, what,
                                    seg_scale=PT.seg_scales(conds[0], dp.seg), adam=True)
        for k, v in e.items():
            worst[k] = max(worst.get(k, 0.0), v)
        dp.advance()
    d.close()
    return worst


ILL_CONDITIONED = 5e4      # forward-error scale of the update (in units of the update) beyond which 1e-5 of it is half a unit: sign-like


def free_run_adam(wl, steps):
    """Oracle and CUDA path each free-run the Adam step from the same initial state. g, m and v are
    held to the per-step bounds (their recurrences contract). theta is a running sum of updates
    u = mhat/(sqrt(vhat)+eps) computed with an approximate square root and reciprocal, so its bound
    is the running sum of the per-step scales lr (|u| + cu); and where an aggregate cancels to
    nearly zero while v is still small, u is sign-like (cu >> |u|: a last-bit difference in g flips
    a whole unit step): those elements, found from the ORACLE's own numbers, are left out of the
    comparison of theta from then on, counted, and must stay a small fraction."""
    torch = _torch()
    import paper_2510_08522_b200 as D
    dp = W.DeviceProblem(wl)
    second = torch.zeros(wl.P, dtype=torch.float32, device="cuda")
    orc = Oracle(wl.K, wl.P, dp.seg, wl.dtype)
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    hp, hm, hv, ha = (x.cpu().numpy().copy() for x in (dp.params, dp.momentum, second, dp.prev_agg))
    theta0 = np.abs(hp.astype(np.float64))
    run_scale = np.zeros(wl.P)
    masked = np.zeros(wl.P, dtype=bool)
    tol = PT.TOL_V[wl.dtype]
    worst = {}
    for t in range(1, steps + 1):
        b = dp.fill()
        raw, wide = PT.grads_to_host(torch, dp.grads, wl.dtype)
        cg, cm, cv, ct, au, cu = PT.cond_vectors_adam(wide, b, hp, hm, hv, LR, B1, B2, EPS, t, with_update=True)
        masked |= cu > ILL_CONDITIONED
        run_scale += abs(float(np.float32(LR))) * (au + cu)
        ref = orc.step_adam(raw, b, hp, hm, hv, LR, B1, B2, EPS, t, ha, nthreads=NTHREADS)
        st = d.step_adam(dp.grads, b, dp.params, dp.momentum, second, LR, B1, B2, EPS, t, dp.prev_agg)
        torch.cuda.synchronize()
        what = "%s adam free run step %d" % (wl.name, t)
        e = {"agg": PT.vec_err(dp.prev_agg.cpu().numpy(), ha, cg), "first_moment": PT.vec_err(dp.momentum.cpu().numpy(), hm, cm),
             "second_moment": PT.vec_err(second.cpu().numpy(), hv, cv)}
        keep = ~masked
        e["params"] = PT.vec_err(dp.params.cpu().numpy()[keep], hp[keep], (theta0 + run_scale)[keep])
        for k, v in e.items():
            assert v <= tol, "%s %s: max scaled error %.3e > %.1e" % (what, k, v, tol)
            worst[k] = max(worst.get(k, 0.0), v)
        # the statistics see the state of this step only (no accumulation): the usual bounds
        worst["state"] = max(worst.get("state", 0.0), PT.check_state(st.cpu().numpy(), ref, wl.K, wl.S, dp.seg, b, what,
                                                                     seg_scale=PT.seg_scales(cg, dp.seg), adam=True))
        dp.advance()
    d.close()
    frac = masked.mean()
    assert frac <= 2e-2, "%s: %.2e of the parameters ill-conditioned" % (wl.name, frac)
    worst["masked_fraction"] = float(frac)
    return worst


@pytest.mark.parametrize("idx,P,steps", [(0, 262_147, 6), (1, 333_337, 20), (2, 401_239, 20), (3, 290_011, 10), (4, 523_777, 10)])
def test_adam_free_running(idx, P, steps):
    print(free_run_adam(W.WORKLOADS[idx].scaled(P=P, steps=steps), steps))


@pytest.mark.parametrize("idx,P,steps", [(0, 262_147, 3), (1, 333_337, 8), (2, 401_239, 8), (3, 290_011, 4), (4, 523_777, 4)])
def test_adam_scaled_workloads_multi_step(idx, P, steps):
    print(lock_step_adam(W.WORKLOADS[idx].scaled(P=P, steps=steps), steps))


def test_adam_cfg1_full_size():
    wl = W.WORKLOADS[1]
    print(lock_step_adam(wl.scaled(P=wl.P, steps=4), 4))


@pytest.mark.parametrize("K,P", [(1, 5), (3, 1023), (5, 2049), (33, 20_011), (64, 9_973)])
def test_adam_shapes(K, P):
    wl = W.Workload("adam-K%d-P%d" % (K, P), K, P, 3, W.BF16 if K % 2 else W.F32, 2, 11, "equal", "fixed4", True)
    print(lock_step_adam(wl, 2, v0=0.25))


def test_adam_argument_errors():
    torch = _torch()
    from paper_2510_08522_b200 import binding as B
    P = 4096
    rc, h = B.dmx_create(2, P, [0, P], 0)
    assert rc == 0
    g = [torch.zeros(P, device="cuda") for _ in range(2)]
    s = [torch.zeros(P + 8, device="cuda") for _ in range(4)]
    out = torch.zeros(B.dmx_state_len(h), device="cuda")
    call = lambda **kw: B.dmx_step_adam(h, [x.data_ptr() for x in g], [1, 2], s[0].data_ptr(), s[1].data_ptr(),
                                        kw.get("v", s[2].data_ptr()), 1e-3, kw.get("b1", 0.9), kw.get("b2", 0.999),
                                        kw.get("eps", 1e-8), kw.get("t", 1), s[3].data_ptr(), out.data_ptr())
    assert call() == B.OK
    assert call(t=0) == B.ERR_ARG and call(b1=1.0) == B.ERR_ARG and call(b2=-0.5) == B.ERR_ARG and call(eps=-1.0) == B.ERR_ARG
    assert call(v=0) == B.ERR_ARG
    assert call(v=s[2].data_ptr() + 4) == B.ERR_ALIGN
    assert call(v=s[1].data_ptr()) == B.ERR_ARG          # second moment aliases the first
    torch.cuda.synchronize()
    assert B.dmx_destroy(h) == B.OK


def test_adam_full_size_streamed_cfg4():
    """One Adam step at the largest workload's full size, gradients streamed to the oracle in ranges."""
    torch = _torch()
    import paper_2510_08522_b200 as D
    wl = W.WORKLOADS[4]
    dp = W.DeviceProblem(wl)
    orc = Oracle(wl.K, wl.P, dp.seg, wl.dtype)
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    second = torch.full((wl.P,), 1e-3, dtype=torch.float32, device="cuda")
    dp.momentum.normal_(0.0, 0.01)                      # a non-trivial first moment
    b = dp.fill()
    t = 5
    ins = [x.clone() for x in (dp.params, dp.momentum, second, dp.prev_agg)]
    st = d.step_adam(dp.grads, b, dp.params, dp.momentum, second, LR, B1, B2, EPS, t, dp.prev_agg)
    torch.cuda.synchronize()
    orc.begin_adam(b, LR, B1, B2, EPS, t)
    scale = np.zeros(wl.S)
    span = 16 << 20
    tol = PT.TOL_V[wl.dtype]
    for lo in range(0, wl.P, span):
        hi = min(wl.P, lo + span)
        raw, _wide = PT.grads_to_host(torch, dp.grads, wl.dtype, lo, hi)
        hp, hm, hv, ha = (x[lo:hi].cpu().numpy() for x in ins)
        # forward-error scales and the element-wise comparison as tensor arithmetic on the device
        # (numpy needs minutes for 340 M parameters x 32 workers)
        conds = PT.cond_vectors_adam_t(torch, [g[lo:hi] for g in dp.grads], b, ins[0][lo:hi], ins[1][lo:hi], ins[2][lo:hi],
                                       LR, B1, B2, EPS, t)
        scale += PT.seg_scales_range_t(torch, conds[0], dp.seg, lo)
        orc.range_adam(lo, raw, hp, hm, hv, ha, nthreads=NTHREADS)
        for name, gpu, ref_h, cond in zip(("agg", "first_moment", "second_moment", "params"),
                                          (dp.prev_agg, dp.momentum, second, dp.params), (ha, hm, hv, hp), conds):
            e = PT.vec_err_t(torch, gpu[lo:hi], torch.from_numpy(ref_h).cuda(), cond)
            assert e <= tol, "%s adam [%d,%d) %s: max scaled error %.3e > %.1e" % (wl.name, lo, hi, name, e, tol)
        del conds
    ref = orc.end()
    PT.check_state(st.cpu().numpy(), ref, wl.K, wl.S, dp.seg, b, wl.name + " adam", seg_scale=scale, adam=True)
    d.close()
