"""The five workloads run as they are stated: full size AND full step count, free-running.

Oracle and CUDA path each start from the same initial state and consume the same gradient
stream; each keeps its own params, momentum and previous aggregate (fp32, as the interface
stores them) and neither is ever re-seeded from the other. The state vector is compared after
every step; the three per-parameter vectors after every step on the small workloads and after
every fifth step and the last on the two K = 32 workloads. Tolerances are those of
tests/parity.py, unchanged by the step count.

The gradients are generated on the device and streamed to the host in element ranges through
two pinned buffers (the copy of the next range overlaps the oracle's work on the current one);
the forward-error scales and the element-wise comparison run as torch tensor arithmetic on the
device, because numpy needs minutes per step at 340 M parameters x 32 workers.

With DMX_REPORT_DIR set, the per-step worst errors are written there as JSON.
"""
import json
import os

import numpy as np
import pytest

from oracle.dmx_oracle import Oracle
from paper_2510_08522_b200 import workload as W
from tests import parity as PT

pytestmark = pytest.mark.gpu

NTHREADS = max(1, min(64, os.cpu_count() or 1))
SPAN = 16 << 20           # elements per streamed range: 16 of the oracle's 2^20 blocks, one per thread


class HostStream:
    """Ranges of the K device gradient buffers, copied to pinned host memory two at a time."""

    def __init__(self, torch, grads, dtype):
        self.torch, self.grads, self.dtype = torch, grads, dtype
        K = len(grads)
        n = min(SPAN, grads[0].numel())
        self.pinned = [torch.empty((K, n), dtype=grads[0].dtype, pin_memory=True) for _ in range(2)]
        self.stream = torch.cuda.Stream()
        self.events = [torch.cuda.Event(), torch.cuda.Event()]

    def request(self, slot, lo, hi):
        torch = self.torch
        self.stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(self.stream):
            for k, g in enumerate(self.grads):
                self.pinned[slot][k, :hi - lo].copy_(g[lo:hi], non_blocking=True)
            self.events[slot].record()

    def arrays(self, slot, n):
        """numpy views of the K rows in the oracle's storage format (after the copy has landed)."""
        self.events[slot].synchronize()
        buf = self.pinned[slot]
        if self.dtype == 0:
            a = buf.numpy()
        else:
            a = buf.view(self.torch.int16).numpy().view(np.uint16)
        return [a[k, :n] for k in range(a.shape[0])]


def run_as_stated(idx, vectors_every):
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_2510_08522_b200 as D
    wl = W.WORKLOADS[idx]
    dp = W.DeviceProblem(wl)
    orc = Oracle(wl.K, wl.P, dp.seg, wl.dtype)
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    # the oracle's own state, on the host, never refreshed from the device
    h_params = dp.params.cpu().numpy().copy()
    h_mom = dp.momentum.cpu().numpy().copy()
    h_prev = dp.prev_agg.cpu().numpy().copy()
    hs = HostStream(torch, dp.grads, wl.dtype)
    spans = [(lo, min(wl.P, lo + SPAN)) for lo in range(0, wl.P, SPAN)]
    report, failures = [], []
    for t in range(wl.steps):
        b = dp.fill()
        with_vectors = t % vectors_every == 0 or t == wl.steps - 1
        # forward-error scales from the oracle's inputs of this step (device arithmetic)
        ref_m = torch.from_numpy(h_mom).cuda()
        ref_p = torch.from_numpy(h_params).cuda()
        cg, cm, ct = PT.cond_vectors_t(torch, dp.grads, b, ref_p, ref_m, wl.lr, wl.beta)
        scale = PT.seg_scales_t(torch, cg, dp.seg)
        if not with_vectors:
            del cm, ct
        del ref_m, ref_p
        # the oracle's step, range by range
        orc.begin(b, wl.lr, wl.beta)
        hs.request(0, *spans[0])
        for i, (lo, hi) in enumerate(spans):
            if i + 1 < len(spans):
                hs.request((i + 1) & 1, *spans[i + 1])
            raw = hs.arrays(i & 1, hi - lo)
            orc.range(lo, raw, h_params[lo:hi], h_mom[lo:hi], h_prev[lo:hi], nthreads=NTHREADS)
        st_ref = orc.end()
        # the CUDA path's step (the pinned copies above were ordered after fill() and are complete)
        st = d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg)
        torch.cuda.synchronize()
        what = "%s step %d" % (wl.name, t)
        row = {"step": t}
        try:
            row["state"] = PT.check_state(st.cpu().numpy(), st_ref, wl.K, wl.S, dp.seg, b, what, seg_scale=scale)
        except AssertionError as e:          # keep going: the report should show the whole run
            failures.append(str(e))
        if with_vectors:
            tol = PT.TOL_V[wl.dtype]
            for name, gpu, ref, cond in (("agg", dp.prev_agg, h_prev, cg), ("momentum", dp.momentum, h_mom, cm),
                                         ("params", dp.params, h_params, ct)):
                e = PT.vec_err_t(torch, gpu, torch.from_numpy(ref).cuda(), cond)
                row[name] = e
                if not e <= tol:
                    failures.append("%s %s: max scaled error %.3e > %.1e" % (what, name, e, tol))
            del cm, ct
        del cg
        report.append(row)
        dp.advance()
    d.close()
    out_dir = os.environ.get("DMX_REPORT_DIR")
    if out_dir:
        os.makedirs(out_dir, exist_ok=True)
        with open(os.path.join(out_dir, "stated_steps_%s.json" % wl.name), "w") as f:
            json.dump({"workload": wl.name, "steps": wl.steps, "tol_vectors": PT.TOL_V[wl.dtype], "tol_scalars": PT.TOL_S,
                       "rows": report}, f)
    worst = {k: max(r.get(k, 0.0) for r in report) for k in ("state", "agg", "momentum", "params")}
    print(wl.name, "steps", wl.steps, "worst errors", worst)
    assert not failures, "%d comparisons failed, first: %s" % (len(failures), failures[:3])
    return report


@pytest.mark.parametrize("idx,vectors_every", [(0, 1), (1, 1), (2, 1), (3, 5), (4, 5)])
def test_workload_as_stated(idx, vectors_every):
    run_as_stated(idx, vectors_every)
