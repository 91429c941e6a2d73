"""The controller's decision step: pins of the CPU oracle (no GPU), then GPU parity through the C ABI.

The paper fixes the action set {-100,-25,0,+25,+100}, the clamp to [32, 1024] and the reward
formula (Sections "Action space and batch size adjustment" and "Reward function design"); those
are pinned by hand-computed values. The policy network and the state layout are this library's
definitions; the network is pinned against torch.nn layers, the layout by one-hot probes.
"""
import numpy as np
import pytest

from oracle import dmx_ctl_oracle as O

HDR = 16


def make_window(K, S, rng, **over):
    """A plausible window vector (means, then deviations) of a K-worker, S-segment state."""
    n = HDR + K + 2 * S
    mean = np.zeros(n)
    std = np.zeros(n)
    mean[0] = over.get("B", 128.0 * K)
    mean[4] = over.get("gns", 900.0)
    mean[5] = over.get("cos", 0.3)
    mean[8] = over.get("sig2", 0.04)
    mean[9] = over.get("sig", 0.2)
    q = rng.uniform(0.5, 2.0, K)
    mean[HDR:HDR + K] = q
    mean[10] = over.get("wq", float(q.mean()))
    std[5], std[9] = 0.05, 0.01
    std[HDR:HDR + K] = 0.1
    return np.concatenate([mean, std]).astype(np.float32), n


def test_action_table_and_clamp_by_hand():
    # one feature (M=1), H=1, weights zero except the output bias: the bias picks the action
    K, S = 5, 1
    rng = np.random.default_rng(0)
    win, n = make_window(K, S, rng)
    aux = np.zeros((K, 1))
    F, H = O.n_features(1), 1
    batch = [40, 1000, 512, 32, 1024]
    for a_idx, delta in enumerate([-100, -25, 0, 25, 100]):
        w = np.zeros(H * F + H + H * H + H + 5 * H + 5)
        w[-5 + a_idx] = 1.0
        d = O.decide(win, n, aux, batch, w, H, cols=(-1, -1, -1))
        assert list(d["action"]) == [a_idx] * K
        want = [min(max(b + delta, 32), 1024) for b in batch]
        assert list(d["next_batch"]) == want
    # the values the text's rule gives, typed out: x <- max(min(x + a, 1024), 32)
    w = np.zeros(H * F + H + H * H + H + 5 * H + 5)
    w[-5] = 1.0
    assert list(O.decide(win, n, aux, batch, w, H, cols=(-1, -1, -1))["next_batch"]) == [32, 900, 412, 32, 924]
    w[-5] = 0.0
    w[-1] = 1.0
    assert list(O.decide(win, n, aux, batch, w, H, cols=(-1, -1, -1))["next_batch"]) == [140, 1024, 612, 132, 1024]


def test_reward_by_hand():
    # r = Abar + alpha max(0, dA) - beta T - delta (log2 x - 5) - eta (sigma2 + sigma)
    K, S = 3, 2
    rng = np.random.default_rng(1)
    win, n = make_window(K, S, rng, sig2=0.25, sig=0.5)
    aux = np.array([[0.50, 0.10, 2.0], [0.75, -0.20, 1.0], [0.25, 0.00, 4.0]])
    batch = [32, 1024, 128]
    r = O.reward(win, n, aux, batch, (0, 1, 2), alpha=2.0, beta_t=0.125, delta=0.5, eta=0.0)
    # worker 0: 0.5 + 0.2 - 0.25 - 0            = 0.45
    # worker 1: 0.75 + 0  - 0.125 - 0.5*5       = -1.875
    # worker 2: 0.25 + 0  - 0.5   - 0.5*2       = -1.25
    assert np.allclose(r, [0.45, -1.875, -1.25], rtol=0, atol=1e-12)
    r2 = O.reward(win, n, aux, batch, (0, 1, 2), alpha=2.0, beta_t=0.125, delta=0.5, eta=4.0)
    assert np.allclose(r2, np.array([0.45, -1.875, -1.25]) - 4.0 * 0.75, rtol=0, atol=1e-12)
    # absent columns drop their terms; the regulariser is 0 at the minimum batch of 32
    r3 = O.reward(win, n, aux, [32, 32, 32], (-1, -1, -1), alpha=2.0, beta_t=1.0, delta=3.0, eta=0.0)
    assert np.all(r3 == 0.0)
    # swapping the gain's sign must matter only through max(0, .)
    aux_neg = aux.copy()
    aux_neg[:, 1] = -np.abs(aux[:, 1])
    r4 = O.reward(win, n, aux_neg, batch, (0, 1, 2), alpha=2.0, beta_t=0.125, delta=0.5, eta=0.0)
    assert np.allclose(r4, [0.25, -1.875, -1.25], rtol=0, atol=1e-12)


def test_mlp_matches_torch_layers_in_fp64():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(2)
    K, F, H = 7, 13, 24
    f = rng.normal(size=(K, F))
    w = rng.normal(scale=0.4, size=H * F + H + H * H + H + 5 * H + 5)
    W1, c1, W2, c2, W3, c3 = O.unpack_weights(w, F, H)
    net = torch.nn.Sequential(torch.nn.Linear(F, H), torch.nn.Tanh(), torch.nn.Linear(H, H), torch.nn.Tanh(),
                              torch.nn.Linear(H, 5)).double()
    with torch.no_grad():
        for lin, (W, c) in zip((net[0], net[2], net[4]), ((W1, c1), (W2, c2), (W3, c3))):
            lin.weight.copy_(torch.from_numpy(W.copy()))
            lin.bias.copy_(torch.from_numpy(c.copy()))
        ref = net(torch.from_numpy(f)).numpy()
    z = O.logits(f, w, H)
    assert np.allclose(z, ref, rtol=1e-12, atol=1e-13)
    # a transposed first layer would not survive this (F != H), nor a dropped bias
    assert not np.allclose(O.logits(f, np.concatenate([w[:H * F], 0 * c1, w[H * F + H:]]), H), ref, atol=1e-3)


def test_feature_layout_by_probes():
    K, S, M = 4, 3, 2
    rng = np.random.default_rng(3)
    win, n = make_window(K, S, rng, B=4 * 64.0, gns=3 * 256.0, cos=0.5, sig2=0.09, sig=0.3, wq=2.0)
    aux = np.arange(K * M, dtype=np.float64).reshape(K, M) + 10
    batch = [32, 64, 128, 32]
    f = O.features(win, n, aux, batch)
    assert f.shape == (K, M + 9)
    assert np.array_equal(f[:, :M], aux)
    assert np.allclose(f[:, M], [0, 1, 2, 0])                          # log2 x - 5
    assert np.allclose(f[:, M + 1], [0.5, 1.0, 2.0, 0.5])              # x K / Bbar, Bbar = 256
    assert np.allclose(f[:, M + 2], win[HDR:HDR + K].astype(np.float64) / 2.0)
    g = M + 3
    assert np.allclose(f[:, g + 0], np.float32(0.3)) and np.allclose(f[:, g + 1], np.float32(0.09))
    assert np.allclose(f[:, g + 2], np.float32(0.01))
    assert np.allclose(f[:, g + 3], 0.5) and np.allclose(f[:, g + 4], np.float32(0.05))
    assert np.allclose(f[:, g + 5], 2.0)                               # log2(1 + 768/256)
    # a negative noise-scale estimate counts as 0; an all-zero window divides by nothing
    win2, _ = make_window(K, S, rng, gns=-5.0)
    assert np.all(O.features(win2, n, aux, batch)[:, g + 5] == 0.0)
    z = O.features(np.zeros(2 * n, np.float32), n, aux, batch)
    assert np.all(np.isfinite(z)) and np.all(z[:, M + 1:M + 3] == 0.0)


def test_sampling_follows_softmax():
    rng = np.random.default_rng(4)
    z = np.tile(np.array([[0.3, -1.0, 2.0, 0.0, 1.2]]), (20000, 1))
    u = rng.random(20000)
    a = O.choose(z, u)
    p = np.exp(z[0] - z[0].max())
    p /= p.sum()
    freq = np.bincount(a, minlength=5) / len(a)
    assert np.all(np.abs(freq - p) < 4 * np.sqrt(p * (1 - p) / len(a)) + 1e-3)
    # the ends of the unit interval: u = 0 takes the first action, u just below 1 the last
    assert O.choose(z[:1], [0.0])[0] == 0 and O.choose(z[:1], [1.0 - 1e-12])[0] == 4
    # greedy: ties go to the lowest index
    assert O.choose(np.array([[1.0, 3.0, 3.0, 0.0, 3.0]]))[0] == 1


# ------------------------------------------------------------------------------------------
# GPU parity through the C ABI

def _gpu_decide(torch, D, win, n, aux, batch, w, H, cols, coef, rng_u, b_min=32, b_max=1024):
    dev = "cuda:0"
    K, M = aux.shape
    t_win = torch.from_numpy(np.asarray(win, np.float32)).to(dev)
    t_aux = torch.from_numpy(np.asarray(aux, np.float32)).to(dev).contiguous()
    t_b = torch.tensor(list(batch), dtype=torch.int32, device=dev)
    t_w = torch.from_numpy(np.asarray(w, np.float32)).to(dev)
    t_u = None if rng_u is None else torch.from_numpy(np.asarray(rng_u, np.float32)).to(dev)
    out = D.ctl_decide(K, M, H, n, t_win, t_aux, t_b, t_w, cols, coef, b_min, b_max, t_u)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def _check(d_gpu, d_ref, z_margin=1e-5):
    assert np.allclose(d_gpu["features"], d_ref["features"], rtol=1e-6, atol=1e-7)
    assert np.allclose(d_gpu["logits"], d_ref["logits"], rtol=1e-5, atol=1e-6)
    assert np.allclose(d_gpu["reward"], d_ref["reward"], rtol=1e-5, atol=1e-6)
    # the decision is unique unless the two best logits sit within rounding of each other
    zs = np.sort(d_ref["logits"], axis=1)
    sure = (zs[:, -1] - zs[:, -2]) > z_margin
    assert sure.mean() > 0.9
    return sure


@pytest.mark.gpu
@pytest.mark.parametrize("K,S,M,H", [(4, 4, 3, 16), (32, 390, 8, 64), (64, 7, 0, 256), (1, 1, 32, 1), (16, 161, 5, 33)])
def test_gpu_greedy_matches_oracle(K, S, M, H):
    import torch
    import paper_2510_08522_b200 as D
    rng = np.random.default_rng(100 + K)
    win, n = make_window(K, S, rng)
    aux = rng.normal(size=(K, M)).astype(np.float32)
    batch = rng.integers(1, 33, K) * 32
    F = O.n_features(M)
    w = rng.normal(scale=1.0 / np.sqrt(max(F, H)), size=H * F + H + H * H + H + 5 * H + 5).astype(np.float32)
    cols = (0, 1, 2) if M >= 3 else (-1, -1, -1)
    coef = (1.5, 0.01, 0.05, 0.3)
    ref = O.decide(win, n, aux, batch, w, H, cols, *coef)
    got = _gpu_decide(torch, D, win, n, aux, batch, w, H, cols, coef, None)
    sure = _check(got, ref)
    assert np.array_equal(got["action"][sure], ref["action"][sure])
    assert np.array_equal(got["next_batch"][sure], ref["next_batch"][sure])
    # always: the device's decision is the argmax of its own emitted logits, and the update obeys the clamp
    assert np.array_equal(got["action"], np.argmax(got["logits"], axis=1))
    assert np.array_equal(got["next_batch"], np.clip(batch + O.ACTIONS[got["action"]], 32, 1024))


@pytest.mark.gpu
def test_gpu_sampling_matches_oracle():
    import torch
    import paper_2510_08522_b200 as D
    rng = np.random.default_rng(7)
    K, S, M, H = 64, 5, 4, 32
    win, n = make_window(K, S, rng)
    aux = rng.normal(size=(K, M)).astype(np.float32)
    batch = rng.integers(1, 33, K) * 32
    F = O.n_features(M)
    w = rng.normal(scale=0.5, size=H * F + H + H * H + H + 5 * H + 5).astype(np.float32)
    hits = np.zeros(5, int)
    for rep in range(4):
        u = rng.random(K).astype(np.float32)
        ref = O.decide(win, n, aux, batch, w, H, (0, 1, 2), 1.0, 0.1, 0.1, 0.0, uniforms=u)
        got = _gpu_decide(torch, D, win, n, aux, batch, w, H, (0, 1, 2), (1.0, 0.1, 0.1, 0.0), u)
        _check(got, ref)
        # unique unless u sits within rounding of a cumulative probability
        z = ref["logits"].astype(np.float32).astype(np.float64)
        p = np.exp(z - z.max(axis=1, keepdims=True))
        c = np.cumsum(p / p.sum(axis=1, keepdims=True), axis=1)
        sure = np.min(np.abs(c - u[:, None].astype(np.float64)), axis=1) > 1e-6
        assert sure.mean() > 0.95
        assert np.array_equal(got["action"][sure], ref["action"][sure])
        assert np.array_equal(got["next_batch"][sure], ref["next_batch"][sure])
        hits += np.bincount(got["action"], minlength=5)
    assert (hits > 0).sum() >= 3          # the sampler really spreads over the actions


@pytest.mark.gpu
def test_gpu_closed_loop_with_window_and_steps():
    """Steps -> window statistics -> decision, all on the device; the oracle chain beside it."""
    import torch
    import paper_2510_08522_b200 as D
    from oracle.dmx_oracle import Oracle, window_stats
    from paper_2510_08522_b200 import workload as W
    from tests import parity as PT
    wl = W.WORKLOADS[1].scaled(P=200_003, steps=6)
    dp = W.DeviceProblem(wl, "cuda:0")
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    orc = Oracle(wl.K, wl.P, dp.seg, wl.dtype)
    k = 3
    rc, agg = D.dmx_agg_create(d.state_len, k)
    assert rc == 0
    window = torch.zeros(2 * d.state_len, dtype=torch.float32, device="cuda:0")
    hp, hm, hv = dp.params.cpu().numpy().copy(), dp.momentum.cpu().numpy().copy(), dp.prev_agg.cpu().numpy().copy()
    rng = np.random.default_rng(11)
    M, H = 3, 16
    F = O.n_features(M)
    w = rng.normal(scale=0.5, size=H * F + H + H * H + H + 5 * H + 5).astype(np.float32)
    batch = np.array(dp.batch_sizes(), dtype=np.int64)
    ref_states = []
    stream = torch.cuda.current_stream().cuda_stream
    for t in range(6):
        dp.fill()
        raw, _ = PT.grads_to_host(torch, dp.grads, wl.dtype)
        ref_states.append(orc.step(raw, batch.astype(np.int32), hp, hm, wl.lr, wl.beta, hv))
        st = d.step(dp.grads, [int(b) for b in batch], dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg)
        rc, emitted = D.dmx_agg_push(agg, st.data_ptr(), window.data_ptr(), stream)
        assert rc == 0 and emitted == (1 if t % k == k - 1 else 0)
        if emitted:
            aux = rng.normal(size=(wl.K, M)).astype(np.float32)
            ref_win = window_stats(np.stack(ref_states))
            ref_states = []
            ref = O.decide(ref_win, d.state_len, aux, batch, w, H, (0, 1, 2), 1.0, 0.1, 0.05, 0.2)
            got = _gpu_decide(torch, D, window.cpu().numpy(), d.state_len, aux, batch, w, H, (0, 1, 2),
                              (1.0, 0.1, 0.05, 0.2), None)
            assert np.allclose(got["features"], ref["features"], rtol=2e-4, atol=1e-6)   # scalar statistics: 1e-4
            assert np.allclose(got["logits"], ref["logits"], rtol=1e-3, atol=1e-3)
            assert np.allclose(got["reward"], ref["reward"], rtol=1e-4, atol=1e-5)
            batch = got["next_batch"].astype(np.int64)       # the device's decision drives the next cycle
            assert batch.min() >= 32 and batch.max() <= 1024
        dp.advance()
    D.dmx_agg_destroy(agg)
    d.close()


@pytest.mark.gpu
def test_gpu_ctl_argument_errors():
    import torch
    import paper_2510_08522_b200 as D
    from paper_2510_08522_b200 import binding as B
    z = torch.zeros(4096, dtype=torch.float32, device="cuda:0")
    zi = torch.zeros(64, dtype=torch.int32, device="cuda:0")
    p = z.data_ptr()
    ok = dict(K=4, M=2, H=8, state_len=HDR + 4 + 2, window=p, aux=p, batch=zi.data_ptr(), weights=p, cols=(0, 1, -1),
              coef=(1.0, 0.0, 0.0, 0.0), b_min=32, b_max=1024, uniforms=0, next_batch=zi.data_ptr(), action=zi.data_ptr(),
              reward=p, logits=p, features=p)

    def call(**kw):
        a = dict(ok)
        a.update(kw)
        return B.dmx_ctl_decide(**a)

    assert call(K=0) == B.ERR_ARG and call(K=65) == B.ERR_ARG
    assert call(M=-1) == B.ERR_ARG and call(M=33) == B.ERR_ARG
    assert call(H=0) == B.ERR_ARG and call(H=257) == B.ERR_ARG
    assert call(state_len=HDR + 3) == B.ERR_ARG           # shorter than header + K
    assert call(cols=(0, 2, -1)) == B.ERR_ARG             # column beyond M
    assert call(b_min=0) == B.ERR_ARG and call(b_min=64, b_max=32) == B.ERR_ARG
    assert call(window=0) == B.ERR_ARG and call(next_batch=0) == B.ERR_ARG
    assert call(M=0, aux=0, cols=(-1, -1, -1)) == B.OK    # no caller metrics: aux may be null
    assert call() == B.OK
    torch.cuda.synchronize()


@pytest.mark.gpu
@pytest.mark.parametrize("adam", [False, True])
def test_gpu_closed_loop_module_runs(adam):
    """The packaged loop (steps -> window -> decision -> batch sizes) keeps its invariants."""
    from paper_2510_08522_b200 import closed_loop
    recs = closed_loop.run(workload=2, P=300_011, cycles=4, k=3, hidden=16, adam=adam, sample=True, seed=3)
    assert len(recs) == 4
    for i, r in enumerate(recs):
        assert r["batch"].min() >= 32 and r["batch"].max() <= 1024
        assert np.all((r["action"] >= 0) & (r["action"] <= 4)) and np.all(np.isfinite(r["reward"]))
        assert r["gns"] > 0 and -1.0 <= r["cos"] <= 1.0 and r["sigma_norm"] > 0
        assert r["flags"] & 16 == 0
        if i:
            step = r["batch"].astype(np.int64) - recs[i - 1]["batch"]
            want = np.clip(recs[i - 1]["batch"] + O.ACTIONS[recs[i - 1]["action"]], 32, 1024) - recs[i - 1]["batch"]
            assert np.array_equal(step, want)
