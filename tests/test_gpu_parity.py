"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element, on the
same seeded inputs. Needs a GPU."""
import os

import numpy as np
import pytest

from oracle.dmx_oracle import Oracle
from paper_2510_08522_b200 import workload as W
from tests import parity as PT

pytestmark = pytest.mark.gpu

NTHREADS = max(1, min(32, os.cpu_count() or 1))


def _torch():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return torch


def _dmx():
    import paper_2510_08522_b200 as D
    return D


class Custom:
    """A hand-built problem uploaded to the device."""

    def __init__(self, grads, b, seg, dtype=0, params=None, momentum=None, prev=None, lr=0.1, beta=0.9):
        torch = _torch()
        self.K, self.P = len(grads), len(grads[0])
        self.seg = np.asarray(seg, np.int64)
        self.S = len(seg) - 1
        self.dtype, self.b, self.lr, self.beta = dtype, np.asarray(b, np.int32), lr, beta
        if dtype == 1:
            self.raw = [W.f32_to_bf16_bits(np.asarray(g, np.float32)) for g in grads]
            self.wide = [W.bf16_bits_to_f32(r) for r in self.raw]
            self.d_grads = [torch.from_numpy(r.view(np.int16)).cuda().view(torch.bfloat16) for r in self.raw]
        else:
            self.raw = [np.ascontiguousarray(g, np.float32) for g in grads]
            self.wide = self.raw
            self.d_grads = [torch.from_numpy(r).cuda() for r in self.raw]
        z = lambda a: np.zeros(self.P, np.float32) if a is None else np.array(a, np.float32)
        self.params, self.momentum, self.prev = z(params), z(momentum), z(prev)
        self.d_params = torch.from_numpy(self.params).cuda()
        self.d_momentum = torch.from_numpy(self.momentum).cuda()
        self.d_prev = torch.from_numpy(self.prev).cuda()

    def run(self, check=True, what=""):
        D = _dmx()
        cg, cm, ct = PT.cond_vectors(self.wide, self.b, self.params, self.momentum, self.lr, self.beta)
        orc = Oracle(self.K, self.P, self.seg, self.dtype)
        st_ref = orc.step(self.raw, self.b, self.params, self.momentum, self.lr, self.beta, self.prev)
        d = D.Dmx(self.K, self.P, self.seg, self.dtype)
        st = d.step(self.d_grads, self.b, self.d_params, self.d_momentum, self.lr, self.beta, self.d_prev)
        _torch().cuda.synchronize()
        st_gpu = st.cpu().numpy()
        d.check_guards()
        d.close()
        gpu = (self.d_prev.cpu().numpy(), self.d_momentum.cpu().numpy(), self.d_params.cpu().numpy())
        if check:
            PT.check_vectors(self.dtype, gpu, (self.prev, self.momentum, self.params), (cg, cm, ct), what)
            PT.check_state(st_gpu, st_ref, self.K, self.S, self.seg, self.b, what, seg_scale=PT.seg_scales(cg, self.seg))
        return st_gpu, st_ref, gpu


def rnd(seed, K, P, scale=1.0):
    r = np.random.default_rng(seed)
    mu = 0.1 * r.standard_normal(P)
    return [(mu + scale * r.standard_normal(P) / np.sqrt(32 * (k + 1))).astype(np.float32) for k in range(K)]


def free_run(wl, steps, every=1):
    """Oracle and CUDA path each free-run from the same initial state on the same gradient
    stream; compared after every step."""
    torch, D = _torch(), _dmx()
    dp = W.DeviceProblem(wl)
    orc = Oracle(wl.K, wl.P, dp.seg, wl.dtype)
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    h_params = dp.params.cpu().numpy().copy()
    h_mom = dp.momentum.cpu().numpy().copy()
    h_prev = dp.prev_agg.cpu().numpy().copy()
    worst = {}
    for t in range(steps):
        b = dp.fill()
        raw, wide = PT.grads_to_host(torch, dp.grads, wl.dtype)
        conds = PT.cond_vectors(wide, b, h_params, h_mom, wl.lr, wl.beta)
        st_ref = orc.step(raw, b, h_params, h_mom, wl.lr, wl.beta, h_prev, nthreads=NTHREADS)
        st = d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg)
        torch.cuda.synchronize()
        if t % every == 0 or t == steps - 1:
            what = "%s step %d" % (wl.name, t)
            e = PT.check_vectors(wl.dtype, (dp.prev_agg.cpu().numpy(), dp.momentum.cpu().numpy(), dp.params.cpu().numpy()),
                                 (h_prev, h_mom, h_params), conds, what)
            e["state"] = PT.check_state(st.cpu().numpy(), st_ref, wl.K, wl.S, dp.seg, b, what,
                                        seg_scale=PT.seg_scales(conds[0], dp.seg))
            for k, v in e.items():
                worst[k] = max(worst.get(k, 0.0), v)
        dp.advance()
    d.check_guards()
    d.close()
    return worst


# ---- the five workloads ------------------------------------------------------------------------

def test_cfg0_full_size():
    w = free_run(W.WORKLOADS[0], 1)
    print("cfg0 worst errors", w)


@pytest.mark.parametrize("idx,P,steps", [(1, 333_337, 6), (2, 401_239, 12), (3, 290_011, 4), (4, 523_777, 4)])
def test_scaled_workloads_multi_step(idx, P, steps):
    # same structure (K, dtype, segment-table law, batch-size schedule, drift) at a size the
    # oracle finishes in seconds; P is odd so the last tile is ragged and boundaries fall anywhere
    w = free_run(W.WORKLOADS[idx].scaled(P=P, steps=steps), steps)
    print(idx, "worst errors", w)


# The five workloads at their full sizes and full step counts, free-running, are in
# tests/test_gpu_stated_steps.py.


# ---- edge cases --------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("K,P,seg", [
    (1, 1, [0, 1]),
    (2, 5, [0, 2, 5]),
    (3, 1023, [0, 1, 2, 3, 1023]),
    (4, 1024, [0, 1024]),
    (5, 1025, [0, 1024, 1025]),
    (7, 2049, [0, 0, 7, 7, 7, 2048, 2049, 2049]),
    (8, 4100, [0, 1, 3, 6, 10, 15, 21, 28, 36, 45, 4100]),
    (9, 70_001, [0, 1021, 1022, 5119, 5120, 5121, 40_000, 70_001]),
    (17, 33_333, [0, 11_111, 22_222, 33_333]),
    (33, 20_011, [0, 20_011]),
    (64, 9_973, [0, 5000, 9_973]),
])
def test_shapes_and_boundaries(dtype, K, P, seg):
    b = [16 * (1 + (3 * k) % 7) for k in range(K)]
    c = Custom(rnd(K * 1000 + P, K, P), b, seg, dtype, params=rnd(1, 1, P)[0], momentum=rnd(2, 1, P)[0], prev=rnd(3, 1, P)[0])
    c.run(what="K=%d P=%d dtype=%d" % (K, P, dtype))


def test_boundaries_at_every_residue():
    # 40 segments whose offsets run through every residue mod 8 inside and across tiles
    P = 3 * 2048 + 5
    seg = sorted(set([0, P] + [2048 + r * 9 for r in range(8)] + [4096 - 3 + r for r in range(8)] + [5000 + 17 * r for r in range(20)]))
    for dtype in (0, 1):
        Custom(rnd(5, 6, P), [32, 64, 96, 128, 160, 192], seg, dtype, prev=rnd(6, 1, P)[0]).run(what="residues dtype=%d" % dtype)


def test_many_tiny_segments():
    P = 6000
    seg = list(range(0, 3001)) + [P]            # 3000 one-element segments, then one big one
    Custom(rnd(8, 4, P), [32, 64, 96, 128], seg, 0).run(what="tiny segments")


def test_identical_workers_give_exact_zero_spread():
    P = 50_003
    x = rnd(11, 1, P)[0]
    for dtype in (0, 1):
        c = Custom([x.copy() for _ in range(6)], [32, 64, 96, 128, 256, 48], [0, 1000, P], dtype)
        st, st_ref, gpu = c.run(what="identical dtype=%d" % dtype)
        assert st[2] == 0 and np.all(st[PT.HDR + 6:PT.HDR + 8] == 0)        # tr_sigma and V_s exactly 0
        assert np.array_equal(gpu[0], c.wide[0])                           # g = g_k exactly
        assert st[4] == 0


def test_equal_batches_plain_mean():
    P, K = 10_007, 8
    c = Custom(rnd(13, K, P), [48] * K, [0, P], 0)
    st, st_ref, gpu = c.run(what="equal b")
    mean = np.mean(np.stack(c.wide).astype(np.float64), axis=0)
    assert np.allclose(gpu[0], mean, rtol=1e-5, atol=1e-7)


def test_worker_permutation_invariance():
    P, K = 30_011, 5
    g = rnd(17, K, P)
    b = [32, 64, 96, 128, 256]
    prev = rnd(18, 1, P)[0]
    st0, _, v0 = Custom(g, b, [0, 500, P], 0, prev=prev).run()
    perm = [3, 0, 4, 1, 2]
    st1, _, v1 = Custom([g[i] for i in perm], [b[i] for i in perm], [0, 500, P], 0, prev=prev).run()
    assert np.allclose(v0[0], v1[0], rtol=1e-5, atol=1e-7)
    assert np.allclose(st0[:PT.HDR], st1[:PT.HDR], rtol=1e-5)
    assert np.allclose(st0[PT.HDR:PT.HDR + K][perm], st1[PT.HDR:PT.HDR + K], rtol=1e-6)


def test_nonfinite_inputs_set_flag():
    P = 5000
    g = rnd(19, 3, P)
    g[1][1234] = np.inf
    c = Custom(g, [32, 64, 96], [0, P], 0)
    st, st_ref, gpu = c.run(check=False)
    PT.check_state(st, st_ref, c.K, c.S, c.seg, c.b, "inf")      # flag and finiteness pattern only
    assert int(st[11]) & 1 and not np.isfinite(st[PT.HDR + 1]) and np.isfinite(st[PT.HDR + 0])
    assert not np.isfinite(gpu[0][1234]) and np.all(np.isfinite(np.delete(gpu[0], 1234)))


def test_first_step_flags_and_negative_g2():
    c = Custom([[1.0, -1.0] * 8, [-1.0, 1.0] * 8], [8, 8], [0, 16], 0)
    st, st_ref, _ = c.run(what="opposed")
    assert int(st[11]) & 2 and int(st[11]) & 4 and st[4] == 0 and st[3] < 0


# ---- determinism, reuse, resume ------------------------------------------------------------------

def test_bitwise_reproducible_and_handle_reuse():
    torch, D = _torch(), _dmx()
    wl = W.WORKLOADS[2].scaled(P=777_777, steps=3)
    outs = []
    for rep in range(2):
        dp = W.DeviceProblem(wl)
        d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
        sts = []
        for t in range(3):
            b = dp.fill()
            sts.append(d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg).clone())
            dp.advance()
        torch.cuda.synchronize()
        outs.append((torch.stack(sts).cpu().numpy(), dp.params.cpu().numpy(), dp.momentum.cpu().numpy()))
        d.close()
    for a, b_ in zip(outs[0], outs[1]):
        assert np.array_equal(a, b_)


def test_resume_after_destroy_is_bitwise_identical():
    torch, D = _torch(), _dmx()
    wl = W.WORKLOADS[1].scaled(P=200_003, steps=4)

    def run(split):
        dp = W.DeviceProblem(wl)
        d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
        for t in range(4):
            if split and t == 2:           # all mutable state is the caller's: a new handle continues
                d.close()
                d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
            b = dp.fill()
            st = d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg)
            dp.advance()
        torch.cuda.synchronize()
        d.close()
        return st.cpu().numpy(), dp.params.cpu().numpy()

    a, b_ = run(False), run(True)
    assert np.array_equal(a[0], b_[0]) and np.array_equal(a[1], b_[1])


def test_non_default_stream():
    torch, D = _torch(), _dmx()
    c = Custom(rnd(23, 4, 100_003), [32, 64, 96, 128], [0, 100_003], 0)
    s = torch.cuda.Stream()
    d = D.Dmx(c.K, c.P, c.seg, 0)
    with torch.cuda.stream(s):
        st = d.step(c.d_grads, c.b, c.d_params, c.d_momentum, c.lr, c.beta, c.d_prev)
    s.synchronize()
    orc = Oracle(c.K, c.P, c.seg, 0)
    st_ref = orc.step(c.raw, c.b, c.params, c.momentum, c.lr, c.beta, c.prev)
    PT.check_state(st.cpu().numpy(), st_ref, c.K, c.S, c.seg, c.b, "stream")
    d.close()


# ---- argument errors: rejected on the host, nothing launched ---------------------------------------

def test_argument_errors_return_codes():
    torch, D = _torch(), _dmx()
    from paper_2510_08522_b200 import binding as Bn
    P = 4096
    rc, h = Bn.dmx_create(2, P, [0, P], 0)
    assert rc == 0
    g = [torch.zeros(P + 8, device="cuda") for _ in range(2)]
    st = [torch.zeros(P + 8, device="cuda") for _ in range(3)]
    out = torch.zeros(Bn.dmx_state_len(h) + 4, device="cuda")
    ptr = lambda t, off=0: t.data_ptr() + off
    ok = lambda **kw: Bn.dmx_step(h, kw.get("g", [ptr(g[0]), ptr(g[1])]), kw.get("b", [1, 2]), kw.get("p", ptr(st[0])),
                                  kw.get("m", ptr(st[1])), 0.1, 0.9, kw.get("a", ptr(st[2])), kw.get("o", ptr(out)))
    assert ok() == 0
    assert ok(b=[1, 0]) == Bn.ERR_BATCH
    assert ok(g=[ptr(g[0], 4), ptr(g[1])]) == Bn.ERR_ALIGN
    assert ok(p=ptr(st[0], 8)) == Bn.ERR_ALIGN
    assert ok(o=ptr(out, 2)) == Bn.ERR_ALIGN
    assert ok(p=ptr(st[1])) == Bn.ERR_ARG                      # params aliases momentum
    assert ok(a=ptr(g[0])) == Bn.ERR_ARG                       # prev_agg aliases a gradient
    assert ok(p=ptr(st[1], 16)) == Bn.ERR_ARG                  # partial overlap
    assert ok(g=[0, ptr(g[1])]) == Bn.ERR_ARG
    assert Bn.dmx_step(None, [1], [1], 16, 32, 0.1, 0.9, 48, 64) == Bn.ERR_HANDLE
    torch.cuda.synchronize()
    assert Bn.dmx_destroy(h) == 0
    assert Bn.dmx_destroy(None) == 0
