"""dmx_step_static, the entry point for callers that cannot allocate device memory (a pool or
framework allocator owns it all, or an allocation's device-wide synchronisation is not
affordable where the step runs). It must give the same step as dmx_step, to rounding: the two
differ only in the order of their sums. Checked through the C ABI on two calls in a row (the
second call finds the first call's leftovers in the shared scratch array), then on a problem of
another shape, then at the size limit; and against the CPU oracle itself on the shapes its
kernel table and its segment search have to get right (one worker, more than 32 workers, empty
segments, a boundary exactly on a tile edge, 512 segments on a full grid, and a 32-worker bf16
problem of 32 Mi parameters, where every thread's partial sums run over its CTA's whole range).

Collected last on purpose: a failure here leaves every other test already run.
"""
import numpy as np
import pytest

from oracle.dmx_oracle import Oracle
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


def static_against_oracle(K, P, seg, dtype, b, calls=2, seed=0, on_device=False):
    """dmx_step_static and the oracle free-run from the same state over `calls` steps."""
    torch, B = _setup()
    gen = torch.Generator(device="cuda").manual_seed(seed)
    gdt = torch.float32 if dtype == 0 else torch.bfloat16
    seg = np.asarray(seg, np.int64)
    S = len(seg) - 1
    mu = 0.1 * torch.randn(P, device="cuda", generator=gen)
    st = [0.05 * torch.randn(P, device="cuda", generator=gen), torch.zeros(P, device="cuda"), torch.zeros(P, device="cuda")]
    h = [t.cpu().numpy().copy() for t in st]
    out = torch.full((16 + K + 2 * S,), 7.0, device="cuda")
    orc = Oracle(K, P, seg, dtype)
    for call in range(calls):
        grads = [(mu + torch.randn(P, device="cuda", generator=gen) / float(np.sqrt(b[k]))).to(gdt) for k in range(K)]
        raw, wide = PT.grads_to_host(torch, grads, dtype)
        what = "static K=%d P=%d S=%d dtype=%d call %d" % (K, P, S, dtype, call)
        if on_device:
            cg, cm, ct = PT.cond_vectors_t(torch, grads, b, torch.from_numpy(h[0]).cuda(), torch.from_numpy(h[1]).cuda(), 0.1, 0.9)
            scale = PT.seg_scales_t(torch, cg, seg)
        else:
            cg, cm, ct = PT.cond_vectors(wide, b, h[0], h[1], 0.1, 0.9)
            scale = PT.seg_scales(cg, seg)
        del wide
        st_ref = orc.step(raw, b, h[0], h[1], 0.1, 0.9, h[2], nthreads=16)
        assert B.dmx_step_static(K, P, seg, dtype, [g.data_ptr() for g in grads], b, st[0].data_ptr(), st[1].data_ptr(), 0.1, 0.9,
                                 st[2].data_ptr(), out.data_ptr(), torch.cuda.current_stream().cuda_stream) == B.OK
        torch.cuda.synchronize()
        if on_device:
            for name, gpu, ref, cond in (("agg", st[2], h[2], cg), ("momentum", st[1], h[1], cm), ("params", st[0], h[0], ct)):
                e = PT.vec_err_t(torch, gpu, torch.from_numpy(ref).cuda(), cond)
                assert e <= PT.TOL_V[dtype], "%s %s: max scaled error %.3e" % (what, name, e)
        else:
            PT.check_vectors(dtype, (st[2].cpu().numpy(), st[1].cpu().numpy(), st[0].cpu().numpy()), (h[2], h[1], h[0]), (cg, cm, ct), what)
        PT.check_state(out.cpu().numpy(), st_ref, K, S, seg, b, what, seg_scale=scale)
        del grads, raw


@pytest.mark.parametrize("dtype", [0, 1])
def test_static_against_the_oracle_on_the_shapes_its_kernel_table_covers(dtype):
    tile = 1024 if dtype == 0 else 2048          # elements per tile of the static path's kernel
    static_against_oracle(1, 5 * tile + 3, [0, 7, 5 * tile + 3], dtype, [48], seed=1)                       # one worker: no spread
    static_against_oracle(40, 3 * tile + 1, [0, tile, 3 * tile + 1], dtype, [16 * (1 + k % 5) for k in range(40)], seed=2)  # 64-slot kernel
    P = 200 * tile + 5
    seg = [0, 0, 3, 3, 3, tile, 2 * tile, 2 * tile, 7 * tile + 1, 150 * tile, 150 * tile, P, P]               # empty segments, boundaries on tile edges
    static_against_oracle(5, P, seg, dtype, [32, 64, 96, 128, 160], seed=3)


def test_static_at_the_limit_that_just_fits():
    # 512 segments on a full grid: the per-CTA segment cells take 148 x 512 x 8 bytes of the 1 MiB array
    torch, B = _setup()
    P = 400 * 1024 + 77
    rng = np.random.default_rng(5)
    seg = np.concatenate([[0], np.sort(rng.integers(0, P + 1, B.STATIC_MAX_SEGMENTS - 1)), [P]])
    static_against_oracle(6, P, seg, 0, [32, 64, 96, 128, 160, 192], seed=4)


def test_static_k32_bf16_at_32_mi_parameters():
    # the sizes the library is for: each thread's fp32 partials (q_k, c, pp, the segment sums) run over about nine
    # thousand elements per worker here, and the 1e-4 bound on the scalars has to hold all the same
    wl = W.WORKLOADS[4].scaled(P=(32 << 20) + 13)
    static_against_oracle(wl.K, wl.P, wl.segment_table(), wl.dtype, [int(v) for v in wl.batch_sizes(0)], calls=2, seed=6, on_device=True)
