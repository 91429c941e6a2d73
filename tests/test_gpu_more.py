"""More GPU cases through the C ABI: the plain-load kernel (DMX_KERNEL=direct) against the
oracle, the scheduling knobs (results must not depend on them beyond rounding), and a problem
of more than 2^32 elements checked by closed forms."""
import os

import numpy as np
import pytest

from oracle.dmx_oracle import Oracle
from paper_2510_08522_b200 import workload as W
from tests import parity as PT
from tests.test_gpu_parity import Custom, _dmx, _torch, free_run, rnd

pytestmark = pytest.mark.gpu


class env:
    def __init__(self, **kv):
        self.kv = kv

    def __enter__(self):
        self.old = {k: os.environ.get(k) for k in self.kv}
        os.environ.update({k: str(v) for k, v in self.kv.items()})

    def __exit__(self, *a):
        for k, v in self.old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v


@pytest.mark.parametrize("idx,P,steps", [(0, 262_147, 2), (1, 333_337, 3), (2, 401_239, 3), (3, 290_011, 2), (4, 523_777, 2)])
def test_plain_load_kernel_matches_oracle(idx, P, steps):
    with env(DMX_KERNEL="direct"):
        free_run(W.WORKLOADS[idx].scaled(P=P, steps=steps), steps)


@pytest.mark.parametrize("dtype", [0, 1])
def test_plain_load_kernel_shapes(dtype):
    with env(DMX_KERNEL="direct"):
        for K, P, seg in [(1, 5, [0, 5]), (3, 2049, [0, 1, 1, 700, 2049]), (33, 20_011, [0, 9, 10_000, 20_011]),
                          (64, 9_973, [0, 9_973])]:
            Custom(rnd(K + P, K, P), [32 * (1 + k % 5) for k in range(K)], seg, dtype).run(what="direct K=%d P=%d" % (K, P))


@pytest.mark.parametrize("knobs", [dict(DMX_TILE_GROUP=1, DMX_CHUNK_TILES=1), dict(DMX_TILE_GROUP=3, DMX_CHUNK_TILES=7),
                                   dict(DMX_TILE_GROUP=8, DMX_CHUNK_TILES=64), dict(DMX_CTAS_PER_SM=1, DMX_CHUNK_TILES=4)])
def test_scheduling_knobs_do_not_change_results_beyond_rounding(knobs):
    # many chunks per CTA, odd group sizes, segment boundaries at every residue: the work list and
    # the slot bookkeeping must stay consistent for any cut
    K, P = 6, 1_300_003
    seg = [0] + sorted(set(int(v) for v in np.random.default_rng(5).integers(1, P, 40))) + [P]
    with env(**knobs):
        for dtype in (0, 1):
            Custom(rnd(17, K, P), [16, 48, 32, 256, 64, 1024], seg, dtype).run(what="knobs %r" % (knobs,))


def test_more_than_2_to_32_elements_closed_forms():
    """Index arithmetic beyond 32 bits. Two workers share one constant bf16 gradient buffer
    (identical workers: g = x exactly, no spread), so every output has a closed form:
    A = q_k = P c^2, m' = beta m + c, theta' = theta - lr m'; slices of the per-element
    outputs are compared at the ends and around the 2^31 and 2^32 element marks."""
    torch, D = _torch(), _dmx()
    P = (1 << 32) + 1_234_567
    free, _ = torch.cuda.mem_get_info()
    if free < P * 14 + (4 << 30):
        pytest.skip("needs about 64 GB of free device memory")
    c = 0.0078125                                    # 2^-7: exact in bf16, P c^2 exact in fp64
    g = torch.full((P,), c, dtype=torch.bfloat16, device="cuda")
    gen = torch.Generator(device="cuda").manual_seed(1)
    params = torch.empty(P, dtype=torch.float32, device="cuda").normal_(0, 0.05, generator=gen)
    mom = torch.empty(P, dtype=torch.float32, device="cuda").normal_(0, 0.01, generator=gen)
    prev = torch.full((P,), 2 * c, dtype=torch.float32, device="cuda")
    seg = [0, 1 << 31, (1 << 32) - 3, (1 << 32) + 5, P]
    marks = [0, (1 << 31) - 4096, (1 << 32) - 4096, P - 8192]
    before = [(params[a:a + 8192].cpu().numpy().astype(np.float64), mom[a:a + 8192].cpu().numpy().astype(np.float64)) for a in marks]
    sum_m0 = float(torch.sum(mom, dtype=torch.float64))
    d = D.Dmx(2, P, seg, W.BF16)
    lr, beta = np.float32(0.1), np.float32(0.9)
    st = d.step([g, g], [32, 96], params, mom, float(lr), float(beta), prev)
    torch.cuda.synchronize()
    st = st.cpu().numpy().astype(np.float64)
    d.close()
    A = P * c * c
    assert st[0] == 128 and st[11] == 0
    assert abs(st[1] - A) <= 1e-4 * A and st[2] == 0.0 and abs(st[3] - A) <= 1e-4 * A and st[4] == 0.0
    assert abs(st[5] - 1.0) <= 1e-4 and abs(st[6] - 2 * A) <= 2e-4 * A and abs(st[7] - 4 * A) <= 4e-4 * A
    assert np.allclose(st[16:18], A, rtol=1e-4)
    sizes = np.diff(np.array(seg, dtype=np.float64))
    assert np.all(st[18:22] == 0.0) and np.allclose(st[22:26], sizes * c * c, rtol=1e-4)
    for a, (p0, m0) in zip(marks, before):
        m1 = float(beta) * m0 + c
        p1 = p0 - float(lr) * m1
        assert np.array_equal(prev[a:a + 8192].cpu().numpy(), np.full(8192, c, np.float32))
        assert np.allclose(mom[a:a + 8192].cpu().numpy(), m1, rtol=1e-6, atol=1e-9)
        assert np.allclose(params[a:a + 8192].cpu().numpy(), p1, rtol=1e-6, atol=1e-9)
    # nothing outside the sampled slices was skipped or done twice: the updated momentum's total
    # matches its closed form
    sum_m1 = float(torch.sum(mom, dtype=torch.float64))
    assert abs(sum_m1 - (float(beta) * sum_m0 + P * c)) <= 1e-6 * P * c
    del g, params, prev, mom
    torch.cuda.empty_cache()


def test_step_captured_in_a_cuda_graph_replays_bitwise():
    """A step is two launches and nothing else (no allocation, no copy, no synchronisation), so
    it can be captured in a CUDA graph; replays must give what eager steps give, bit for bit."""
    torch, D = _torch(), _dmx()
    wl = W.WORKLOADS[2].scaled(P=2_000_003, steps=4)
    dp = W.DeviceProblem(wl)
    b = dp.fill()
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    out = torch.empty(d.state_len, dtype=torch.float32, device="cuda")
    p0, m0, a0 = dp.params.clone(), dp.momentum.clone(), dp.prev_agg.clone()
    eager = []
    for _ in range(3):                       # the same gradients three times: the state still evolves
        d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg, out)
        torch.cuda.synchronize()
        eager.append((out.clone(), dp.params.clone(), dp.momentum.clone(), dp.prev_agg.clone()))
    dp.params.copy_(p0); dp.momentum.copy_(m0); dp.prev_agg.copy_(a0)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg, out, stream=side.cuda_stream)
    torch.cuda.synchronize()
    # capture enqueues nothing: the state is still the initial one
    assert torch.equal(dp.params, p0)
    for i in range(3):
        graph.replay()
        torch.cuda.synchronize()
        st, p, m, a = eager[i]
        assert torch.equal(out, st) and torch.equal(dp.params, p) and torch.equal(dp.momentum, m) and torch.equal(dp.prev_agg, a), i
    # and the handle still works eagerly after the replays
    d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg, out)
    torch.cuda.synchronize()
    assert int(out[11].item()) & 16 == 0
    d.close()


@pytest.mark.parametrize("idx", [3, 4])
def test_full_size_step_is_bitwise_reproducible_under_the_dynamic_schedule(idx):
    """At full size every CTA draws dozens of chunks and which CTA gets which varies from run to
    run; the results must not."""
    torch, D = _torch(), _dmx()
    wl = W.WORKLOADS[idx]
    dp = W.DeviceProblem(wl)
    b = dp.fill()
    dp.prev_agg.normal_(0, 0.05)                     # a non-trivial previous aggregate
    p0, m0, a0 = dp.params.clone(), dp.momentum.clone(), dp.prev_agg.clone()
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    runs = []
    for _ in range(3):
        dp.params.copy_(p0); dp.momentum.copy_(m0); dp.prev_agg.copy_(a0)
        st = d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg)
        torch.cuda.synchronize()
        runs.append((st.clone(), dp.params.clone(), dp.momentum.clone(), dp.prev_agg.clone()))
        if len(runs) > 1:
            for x, y in zip(runs[0], runs[-1]):
                assert torch.equal(x, y)
            runs.pop()
    assert int(runs[0][0][11].item()) & 16 == 0
    d.close()


def test_gpu_matches_the_stored_seeded_golden():
    """The CUDA path against stored expected values (tests/golden/seeded_small_k3.json, written by
    the oracle from exact arithmetic)."""
    import json
    torch, D = _torch(), _dmx()
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "seeded_small_k3.json")) as f:
        g = json.load(f)
    dev = "cuda"
    grads = [torch.tensor(x, dtype=torch.float32, device=dev) for x in g["grads"]]
    params, mom, prev = (torch.tensor(g[k], dtype=torch.float32, device=dev) for k in ("params", "momentum", "prev_agg"))
    d = D.Dmx(g["K"], g["P"], g["seg_offsets"], 0)
    st = d.step(grads, g["batch_sizes"], params, mom, g["lr"], g["beta"], prev)
    torch.cuda.synchronize()
    d.close()
    exp = g["expect"]
    # integer-valued inputs with B = 8: the aggregate and the update are exact in fp32 too
    assert prev.cpu().tolist() == exp["agg"] and mom.cpu().tolist() == exp["momentum"] and params.cpu().tolist() == exp["params"]
    assert np.allclose(st.cpu().numpy(), np.array(exp["state"]), rtol=1e-6, atol=1e-6)


@pytest.mark.parametrize("dtype", [0, 1])
def test_step_from_host_gradients_equals_the_device_step(dtype):
    """dmx_step_host: gradients in pinned host memory, staged by the call; same result, bit for bit,
    as dmx_step on the same values, and the state vector arrives in host memory."""
    torch, D = _torch(), _dmx()
    from paper_2510_08522_b200 import binding as B
    K, P = 5, 300_007
    seg = [0, 1000, 150_000, P]
    rng = np.random.default_rng(21)
    gdt = torch.float32 if dtype == 0 else torch.bfloat16
    host = [torch.from_numpy(rng.normal(size=P).astype(np.float32)).to(gdt).pin_memory() for _ in range(K)]
    b = [32, 64, 16, 128, 256]
    p0 = torch.from_numpy(rng.normal(scale=0.05, size=P).astype(np.float32)).cuda()
    m0 = torch.from_numpy(rng.normal(scale=0.01, size=P).astype(np.float32)).cuda()
    a0 = torch.from_numpy(rng.normal(scale=0.1, size=P).astype(np.float32)).cuda()
    d = D.Dmx(K, P, seg, dtype)
    # reference: copy by hand, then the device step
    dev = [h.cuda() for h in host]
    p1, m1, a1 = p0.clone(), m0.clone(), a0.clone()
    st_ref = d.step(dev, b, p1, m1, 0.1, 0.9, a1).clone()
    # the host form
    staging = [torch.empty(P, dtype=gdt, device="cuda") for _ in range(K)]
    p2, m2, a2 = p0.clone(), m0.clone(), a0.clone()
    out_dev = torch.empty(d.state_len, dtype=torch.float32, device="cuda")
    out_host = torch.zeros(d.state_len, dtype=torch.float32).pin_memory()
    d.step_host(host, staging, b, p2, m2, 0.1, 0.9, a2, out_dev, out_host)       # synchronous
    assert torch.equal(out_host, st_ref.cpu()) and torch.equal(out_dev, st_ref)
    assert torch.equal(p1, p2) and torch.equal(m1, m2) and torch.equal(a1, a2)
    for s, h in zip(staging, host):
        assert torch.equal(s.cpu(), h)
    # argument errors come back as codes
    hp = [h.data_ptr() for h in host]
    sp = [s.data_ptr() for s in staging]
    args = (b, p2.data_ptr(), m2.data_ptr(), 0.1, 0.9, a2.data_ptr(), out_dev.data_ptr(), out_host.data_ptr())
    assert B.dmx_step_host(d._h, hp, [sp[0] + 2] + sp[1:], *args) == B.ERR_ALIGN
    assert B.dmx_step_host(d._h, hp, sp, b, p2.data_ptr(), m2.data_ptr(), 0.1, 0.9, a2.data_ptr(), out_dev.data_ptr(), 0) == B.ERR_ARG
    assert B.dmx_step_host(None, hp, sp, *args) == B.ERR_HANDLE
    d.close()


def test_profiling_hooks():
    torch, D = _torch(), _dmx()
    from paper_2510_08522_b200 import binding as B
    c = Custom(rnd(3, 4, 50_000), [32, 64, 96, 128], [0, 50_000])
    d = D.Dmx(c.K, c.P, c.seg, 0)
    assert d.launches_per_step in (1, 2) and B.dmx_launches_per_step(None) == B.ERR_HANDLE
    assert B.dmx_get_profile(d._h)[0] == B.ERR_ARG            # profiling is off
    d.set_profiling(True)
    assert B.dmx_get_profile(d._h)[0] == B.ERR_ARG            # on, but no step recorded yet
    st_on = d.step(c.d_grads, c.b, c.d_params, c.d_momentum, 0.1, 0.9, c.d_prev).clone()
    fused_ms, fin_ms = d.profile()
    assert 0.0 < fused_ms < 50.0 and 0.0 <= fin_ms < 50.0      # a one-launch step has no second kernel to time
    d.set_profiling(False)
    assert B.dmx_get_profile(d._h)[0] == B.ERR_ARG
    # timing on or off does not change results: rerun the same step from the same state without it
    c2 = Custom(rnd(3, 4, 50_000), [32, 64, 96, 128], [0, 50_000])
    st_off = d.step(c2.d_grads, c2.b, c2.d_params, c2.d_momentum, 0.1, 0.9, c2.d_prev)
    torch.cuda.synchronize()
    assert torch.equal(st_on, st_off) and torch.equal(c.d_params, c2.d_params)
    assert B.dmx_set_profiling(None, 1) == B.ERR_HANDLE and B.dmx_last_cuda_error() == 0
    d.close()


@pytest.mark.parametrize("seed", [11, 12])
def test_random_problems_match_the_oracle(seed):
    """Seeded random problems: K from 1 to 64 around the kernel table's capacities, P around the
    tile sizes and up to a few hundred tiles, random segment tables, both gradient types, both
    updates, sometimes with odd scheduling knobs."""
    torch, D = _torch(), _dmx()
    rng = np.random.default_rng(seed)
    for case in range(60):
        K = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 15, 16, 17, 31, 32, 33, 48, 64]))
        P = int(rng.choice([1, 7, 895, 896, 897, 1792, 1793, int(rng.integers(1, 5000)), int(rng.integers(5000, 400_000))]))
        dtype = int(rng.integers(0, 2))
        S = int(rng.choice([1, 2, 3, 17, 200])) if P > 1 else 1
        seg = [0] + sorted(int(v) for v in rng.integers(0, P + 1, S - 1)) + [P]
        b = [int(v) for v in rng.choice([1, 16, 32, 33, 64, 100, 256, 1024], K)]
        knobs = {}
        if rng.random() < 0.3:
            knobs = dict(DMX_CHUNK_TILES=int(rng.choice([1, 2, 5, 8, 33])), DMX_TILE_GROUP=int(rng.choice([1, 2, 3, 4])))
        adam = rng.random() < 0.3
        mu = 0.1 * rng.standard_normal(P)
        g32 = [(mu + rng.standard_normal(P) / np.sqrt(b[k])).astype(np.float32) for k in range(K)]
        what = "case %d: K=%d P=%d dtype=%d S=%d adam=%s knobs=%s" % (case, K, P, dtype, S, adam, knobs)
        with env(**knobs):
            c = Custom(g32, b, seg, dtype, params=0.05 * rng.standard_normal(P), momentum=0.01 * rng.standard_normal(P),
                       prev=0.1 * rng.standard_normal(P))
            if not adam:
                st, _, _ = c.run(what=what)
                assert int(st[11]) & 16 == 0, what
                continue
            h2 = np.abs(0.01 * rng.standard_normal(P)).astype(np.float32)
            d2 = torch.from_numpy(h2.copy()).cuda()
            conds = PT.cond_vectors_adam(c.wide, c.b, c.params, c.momentum, h2, 1e-3, 0.9, 0.999, 1e-8, 3)
            st_ref = Oracle(K, P, c.seg, dtype).step_adam(c.raw, c.b, c.params, c.momentum, h2, 1e-3, 0.9, 0.999, 1e-8, 3, c.prev)
            d = D.Dmx(K, P, c.seg, dtype)
            st = d.step_adam(c.d_grads, c.b, c.d_params, c.d_momentum, d2, 1e-3, 0.9, 0.999, 1e-8, 3, c.d_prev)
            torch.cuda.synchronize()
            d.check_guards()
            d.close()
            PT.check_state(st.cpu().numpy(), st_ref, K, S, c.seg, c.b, what, seg_scale=PT.seg_scales(conds[0], c.seg), adam=True)
            PT.check_vectors_adam(dtype, (c.d_prev.cpu().numpy(), c.d_momentum.cpu().numpy(), d2.cpu().numpy(), c.d_params.cpu().numpy()),
                                  (c.prev, c.momentum, h2, c.params), conds, what)
            assert int(st[11].item()) & 16 == 0, what
