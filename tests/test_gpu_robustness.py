"""Failure paths of the library, shown without ever faulting, trapping or hanging a GPU:
allocation failure injected on the host, calls on destroyed handles, a bounded wait that is made
to run out on a barrier nothing completes (no copy in flight), guard words beside the scratch,
the wrong-device check, and the checked build (range tests of every table and scratch index)."""
import os
import subprocess
import sys

import numpy as np
import pytest

from paper_2510_08522_b200 import workload as W

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _env():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_2510_08522_b200 as D
    from paper_2510_08522_b200 import binding as Bn
    return torch, D, Bn


def test_every_allocation_of_create_can_fail_cleanly(monkeypatch):
    torch, D, Bn = _env()
    seg = [0, 1000, 70_001]
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    n = 1
    while True:
        monkeypatch.setenv("DMX_TEST_FAIL_ALLOC", str(n))
        rc, h = Bn.dmx_create(5, 70_001, seg, Bn.F32)
        if rc == Bn.OK:
            break
        assert rc == Bn.ERR_NOMEM and not h, (n, rc)
        assert Bn.dmx_last_cuda_error() in (0, 2)               # 2 = cudaErrorMemoryAllocation (device buffers)
        n += 1
        assert n < 64
    assert n >= 16                                               # the handle and its 15+ device buffers
    assert Bn.dmx_check_guards(h) == Bn.OK
    assert Bn.dmx_destroy(h) == Bn.OK
    monkeypatch.delenv("DMX_TEST_FAIL_ALLOC")
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free0 - (4 << 20)     # nothing leaked by the failed creates
    # the window-statistics handle honours the same knob
    for k in (1, 2, 3, 4):
        monkeypatch.setenv("DMX_TEST_FAIL_ALLOC", str(k))
        rc, a = Bn.dmx_agg_create(40, 3)
        assert rc == Bn.ERR_NOMEM and not a
    monkeypatch.setenv("DMX_TEST_FAIL_ALLOC", "5")
    rc, a = Bn.dmx_agg_create(40, 3)
    assert rc == Bn.OK
    assert Bn.dmx_agg_destroy(a) == Bn.OK


def test_destroyed_handles_are_refused():
    torch, D, Bn = _env()
    P = 4096
    rc, h = Bn.dmx_create(2, P, [0, P], Bn.F32)
    assert rc == Bn.OK
    g = [torch.zeros(P, device="cuda") for _ in range(2)]
    st = [torch.zeros(P, device="cuda") for _ in range(3)]
    out = torch.zeros(Bn.dmx_state_len(h), device="cuda")
    step = lambda: Bn.dmx_step(h, [x.data_ptr() for x in g], [1, 2], st[0].data_ptr(), st[1].data_ptr(), 0.1, 0.9,
                               st[2].data_ptr(), out.data_ptr())
    assert step() == Bn.OK
    torch.cuda.synchronize()
    assert Bn.dmx_destroy(h) == Bn.OK
    assert Bn.dmx_destroy(h) == Bn.ERR_HANDLE                    # a second destroy touches nothing
    assert step() == Bn.ERR_HANDLE
    assert Bn.dmx_state_len(h) == Bn.ERR_HANDLE and Bn.dmx_check_guards(h) == Bn.ERR_HANDLE
    rc, a = Bn.dmx_agg_create(20, 2)
    assert rc == Bn.OK and Bn.dmx_agg_destroy(a) == Bn.OK
    assert Bn.dmx_agg_destroy(a) == Bn.ERR_HANDLE
    assert Bn.dmx_agg_push(a, out.data_ptr(), out.data_ptr())[0] == Bn.ERR_HANDLE
    assert Bn.dmx_step(a, [g[0].data_ptr()], [1], st[0].data_ptr(), st[1].data_ptr(), 0.1, 0.9, st[2].data_ptr(),
                       out.data_ptr()) == Bn.ERR_HANDLE        # a handle of the other kind is not a step handle


@pytest.mark.parametrize("idx,P", [(1, 300_007), (4, 2_000_003)])
def test_a_wait_that_runs_out_is_reported_and_cleared(idx, P):
    torch, D, Bn = _env()
    wl = W.WORKLOADS[idx].scaled(P=P, S=7)
    dp = W.DeviceProblem(wl)
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    b = dp.fill()
    st0 = d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg).cpu().numpy()
    assert not int(st0[Bn.ST_FLAGS]) & Bn.FLAG_INTERNAL
    times = {}
    for polls in (1 << 10, 1 << 14, 1 << 18):
        rc, timed_out, ms = Bn.dmx_selftest_wait(d._h, polls)
        assert rc == Bn.OK and timed_out == 1, (polls, rc, timed_out)
        times[polls] = ms
        # the next step carries the flag, its numbers are those of an undisturbed step, and the flag is gone after it
        st1 = d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg).cpu().numpy()
        assert int(st1[Bn.ST_FLAGS]) & Bn.FLAG_INTERNAL
        assert np.array_equal(st1[Bn.ST_HDR:Bn.ST_HDR + wl.K], st0[Bn.ST_HDR:Bn.ST_HDR + wl.K])
        st2 = d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg).cpu().numpy()
        assert not int(st2[Bn.ST_FLAGS]) & Bn.FLAG_INTERNAL
    per_poll_us = times[1 << 18] / (1 << 18) * 1e3
    print("bounded wait: %s ms; %.3f us per poll" % (times, per_poll_us))
    assert times[1 << 18] < 5000.0                               # 2^18 polls is the fused pass's own budget: seconds, not minutes
    d.check_guards()
    d.close()


def test_guard_words_stay_intact_over_the_shapes_that_stress_the_scratch():
    torch, D, Bn = _env()
    rng = np.random.default_rng(7)
    for K, P, S, dtype in ((3, 5, 2, 0), (4, 6000, 3001, 0), (9, 70_001, 7, 1), (16, 1_500_013, 161, 1), (33, 200_011, 40, 0)):
        cuts = np.sort(rng.integers(0, P + 1, S - 1)) if S > 2 else np.array([P // 2] * (S - 1))
        seg = np.concatenate([[0], cuts, [P]]).astype(np.int64)
        d = D.Dmx(K, P, seg, dtype)
        gdt = torch.float32 if dtype == 0 else torch.bfloat16
        grads = [torch.randn(P, device="cuda").to(gdt) for _ in range(K)]
        st = [torch.randn(P, device="cuda") for _ in range(3)]
        for _ in range(2):
            d.step(grads, [8 * (k + 1) for k in range(K)], st[0], st[1], 0.1, 0.9, st[2])
        torch.cuda.synchronize()
        d.check_guards()
        d.close()


def test_a_step_on_another_device_is_refused_on_the_host():
    torch, D, Bn = _env()
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two visible devices; the check itself is host code (cudaGetDevice against the handle's device)")
    P = 4096
    rc, h = Bn.dmx_create(2, P, [0, P], Bn.F32)
    g = [torch.zeros(P, device="cuda:0") for _ in range(2)]
    st = [torch.zeros(P, device="cuda:0") for _ in range(4)]
    with torch.cuda.device(1):
        assert Bn.dmx_step(h, [x.data_ptr() for x in g], [1, 2], st[0].data_ptr(), st[1].data_ptr(), 0.1, 0.9,
                           st[2].data_ptr(), st[3].data_ptr()) == Bn.ERR_HANDLE
    assert Bn.dmx_destroy(h) == Bn.OK


def test_checked_build_finds_nothing_out_of_range():
    """The shape, boundary, tiny-segment and random-problem parity tests once more against the
    checked build (DMX_CHECKED_BUILD=1, own process): parity holds, DMX_FLAG_BOUNDS never appears
    (tests/parity.py rejects any flag bit it does not expect), guard words stay intact."""
    env = dict(os.environ, DMX_CHECKED_BUILD="1")
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
           os.path.join(ROOT, "tests", "test_gpu_parity.py"), os.path.join(ROOT, "tests", "test_gpu_more.py"),
           "-k", "shapes_and_boundaries or every_residue or tiny_segments or scaled_workloads or random_problems or identical"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
