"""Window statistics of the state vector over k steps: oracle pins (CPU) and GPU parity."""
import numpy as np
import pytest

from oracle.dmx_oracle import OracleError, window_stats


def make(k, n, seed=0):
    r = np.random.default_rng(seed)
    s = (r.standard_normal((k, n)) * np.logspace(-3, 3, n)).astype(np.float32)
    s[:, 11] = r.integers(0, 16, k).astype(np.float32)
    return s


def test_against_numpy_mean_and_std():
    s = make(7, 40)
    out = window_stats(s)
    keep = np.arange(40) != 11
    assert np.allclose(out[:40][keep], s.astype(np.float64).mean(axis=0)[keep], rtol=1e-6, atol=1e-12)
    assert np.allclose(out[40:][keep], s.astype(np.float64).std(axis=0)[keep], rtol=1e-6, atol=1e-12)
    assert out[11] == float(np.bitwise_or.reduce(s[:, 11].astype(np.int64))) and out[40 + 11] == 0


def test_closed_forms():
    k, n = 9, 16
    s = np.tile(np.arange(1, k + 1, dtype=np.float32)[:, None], (1, n))        # 1..k in every entry
    s[:, 11] = [1, 0, 4, 0, 0, 8, 0, 0, 0]
    out = window_stats(s)
    keep = np.arange(n) != 11
    assert np.allclose(out[:n][keep], (k + 1) / 2) and np.allclose(out[n:][keep], np.sqrt((k * k - 1) / 12.0), rtol=1e-6)
    assert out[11] == 13
    c = np.full((5, n), 3.25, np.float32); c[:, 11] = 2
    out = window_stats(c)
    assert np.all(out[:n][keep] == 3.25) and np.all(out[n:] == 0) and out[11] == 2
    one = window_stats(make(1, 20))                                              # k = 1: the vector itself
    assert np.array_equal(one[:20], make(1, 20)[0]) and np.all(one[20:] == 0)
    with pytest.raises(OracleError):
        window_stats(np.zeros((3, 5), np.float32))


@pytest.mark.gpu
def test_gpu_window_matches_oracle_over_several_windows():
    import torch
    assert torch.cuda.is_available()
    from paper_2510_08522_b200 import binding as B
    n, k = 16 + 8 + 2 * 62, 5
    rc, a = B.dmx_agg_create(n, k)
    assert rc == B.OK
    s = make(3 * k + 2, n, seed=3)
    d = torch.from_numpy(s).cuda()
    out = torch.full((2 * n,), -7.0, device="cuda")
    for t in range(s.shape[0]):
        rc, emitted = B.dmx_agg_push(a, d[t].data_ptr(), out.data_ptr())
        assert rc == B.OK and emitted == int((t + 1) % k == 0)
        torch.cuda.synchronize()
        if emitted:
            ref = window_stats(s[t + 1 - k:t + 1])
            got = out.cpu().numpy()
            assert np.allclose(got[:n], ref[:n], rtol=2e-6, atol=0), t
            scale = np.maximum(ref[n:], 1e-6 * np.abs(ref[:n]))
            assert np.all(np.abs(got[n:] - ref[n:]) <= 1e-5 * scale), t
            assert got[11] == ref[11] and got[n + 11] == 0
        elif t < k:
            assert torch.all(out == -7.0)                 # untouched before the first window closes
    assert B.dmx_agg_push(None, d[0].data_ptr(), out.data_ptr())[0] == B.ERR_HANDLE
    assert B.dmx_agg_push(a, 0, out.data_ptr())[0] == B.ERR_ARG
    assert B.dmx_agg_destroy(a) == B.OK and B.dmx_agg_destroy(None) == B.OK
    assert B.dmx_agg_create(11, 3)[0] == B.ERR_ARG and B.dmx_agg_create(20, 0)[0] == B.ERR_ARG


@pytest.mark.gpu
def test_gpu_window_on_real_steps():
    import torch
    import paper_2510_08522_b200 as D
    from paper_2510_08522_b200 import binding as B
    from paper_2510_08522_b200 import workload as W
    wl = W.WORKLOADS[1].scaled(P=120_011, steps=6)
    dp = W.DeviceProblem(wl)
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    rc, a = B.dmx_agg_create(d.state_len, 3)
    assert rc == B.OK
    out = torch.zeros(2 * d.state_len, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    states = []
    for t in range(6):
        b = dp.fill()
        st = d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg)
        rc, emitted = B.dmx_agg_push(a, st.data_ptr(), out.data_ptr(), stream)      # same stream, after the step
        assert rc == B.OK
        states.append(st.cpu().numpy())
        if emitted:
            ref = window_stats(np.stack(states[-3:]))
            got = out.cpu().numpy()
            n = d.state_len
            assert np.allclose(got[:n], ref[:n], rtol=2e-6)
            assert np.all(np.abs(got[n:] - ref[n:]) <= 1e-5 * np.maximum(ref[n:], 1e-6 * np.abs(ref[:n])))
        dp.advance()
    B.dmx_agg_destroy(a)
    d.close()
