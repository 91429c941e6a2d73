"""dmx_step_static, the entry point for callers that cannot allocate device memory (a pool or
framework allocator owns it all, or an allocation's device-wide synchronisation is not
affordable where the step runs). It must give the same step as dmx_step, to rounding: the two
differ only in the order of their sums. Checked through the C ABI on two calls in a row (the
second call finds the first call's leftovers in the shared scratch array), then on a problem of
another shape, then at the size limit.

Collected last on purpose: a failure here leaves every other test already run.
"""
import numpy as np
import pytest

from paper_2510_08522_b200 import workload as W
from tests import parity as PT

pytestmark = pytest.mark.gpu


def _setup():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2510_08522_b200 import binding as B
    return torch, B


def run_pair(wl, steps):
    """Advance two copies of the same state, one with dmx_step and one with dmx_step_static."""
    torch, B = _setup()
    dp = W.DeviceProblem(wl)
    rc, h = B.dmx_create(wl.K, wl.P, dp.seg, wl.dtype)
    assert rc == B.OK
    n = B.dmx_state_len(h)
    ref = [dp.params, dp.momentum, dp.prev_agg]
    alt = [t.clone() for t in ref]
    st_ref = torch.empty(n, dtype=torch.float32, device="cuda")
    st_alt = torch.full((n,), 7.0, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for t in range(steps):
        b = dp.fill()
        raw, wide = PT.grads_to_host(torch, dp.grads, wl.dtype)
        conds = PT.cond_vectors(wide, b, ref[0].cpu().numpy(), ref[1].cpu().numpy(), wl.lr, wl.beta)
        gp = [g.data_ptr() for g in dp.grads]
        assert B.dmx_step(h, gp, b, ref[0].data_ptr(), ref[1].data_ptr(), wl.lr, wl.beta, ref[2].data_ptr(),
                          st_ref.data_ptr(), stream) == B.OK
        assert B.dmx_step_static(wl.K, wl.P, dp.seg, wl.dtype, gp, b, alt[0].data_ptr(), alt[1].data_ptr(), wl.lr, wl.beta,
                                 alt[2].data_ptr(), st_alt.data_ptr(), stream) == B.OK
        torch.cuda.synchronize()
        what = "%s call %d" % (wl.name, t)
        # same comparison rules as the parity tests, with dmx_step's result as the reference
        PT.check_vectors(wl.dtype, (alt[2].cpu().numpy(), alt[1].cpu().numpy(), alt[0].cpu().numpy()),
                         (ref[2].cpu().numpy(), ref[1].cpu().numpy(), ref[0].cpu().numpy()), conds, what)
        PT.check_state(st_alt.cpu().numpy(), st_ref.cpu().numpy(), wl.K, wl.S, dp.seg, b, what,
                       seg_scale=PT.seg_scales(conds[0], dp.seg))
        dp.advance()
    assert B.dmx_destroy(h) == B.OK


def test_static_matches_handle_path_two_calls_in_a_row():
    run_pair(W.WORKLOADS[1].scaled(P=333_337, steps=2), 2)           # fp32, K=8, 62 segments, ragged tail


def test_static_bf16_then_other_shape_reuses_the_array():
    run_pair(W.WORKLOADS[2].scaled(P=401_239, steps=2), 2)           # bf16, K=16, 161 segments
    run_pair(W.WORKLOADS[0].scaled(P=70_001, steps=2), 2)            # fewer segments, fewer CTAs: stale cells around


def test_static_rejects_what_does_not_fit():
    torch, B = _setup()
    P = 4096
    g = [torch.zeros(P, device="cuda") for _ in range(2)]
    st = [torch.zeros(P, device="cuda") for _ in range(3)]
    S = B.STATIC_MAX_SEGMENTS + 1
    seg = [min(i, P) for i in range(S)] + [P]
    out = torch.zeros(16 + 2 + 2 * S, device="cuda")
    call = lambda seg_, b=(1, 2): B.dmx_step_static(2, P, seg_, B.F32, [t.data_ptr() for t in g], list(b), st[0].data_ptr(),
                                                    st[1].data_ptr(), 0.1, 0.9, st[2].data_ptr(), out.data_ptr())
    assert call(seg) == B.ERR_LIMIT
    assert "scratch" in B.strerror(B.ERR_LIMIT)
    assert call([0, P - 1]) == B.ERR_SEGMENTS
    assert call([0, P], b=(1, 0)) == B.ERR_BATCH
    assert call([0, P]) == B.OK
    torch.cuda.synchronize()
