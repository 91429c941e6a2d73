"""Pins of the oracle's Adam mode: the library optimizer in fp64, closed forms, invariances."""
import math

import numpy as np
import pytest
import torch

from oracle.dmx_oracle import F32, ST, Oracle, OracleError

HDR = ST["HDR"]


def grads_exact(seed, K, P):
    r = np.random.default_rng(seed)
    return [r.integers(-16, 17, P).astype(np.float32) / 8 for _ in range(K)]


def test_against_torch_adam_in_fp64():
    # equal batch sizes and dyadic gradients: the aggregate is exact, so the only difference to
    # torch.optim.Adam (fp64 state) is the oracle's fp32 storage of theta, m, v between steps
    K, P, steps = 4, 257, 12
    lr, b1, b2, eps = 0.01, 0.9, 0.999, 1e-8
    o = Oracle(K, P, [0, 100, P], F32)
    r = np.random.default_rng(0)
    theta0 = r.standard_normal(P).astype(np.float32)
    params = theta0.copy(); m = np.zeros(P, np.float32); v = np.zeros(P, np.float32); prev = np.zeros(P, np.float32)
    tp = torch.nn.Parameter(torch.tensor(theta0, dtype=torch.float64))
    opt = torch.optim.Adam([tp], lr=float(np.float32(lr)), betas=(float(np.float32(b1)), float(np.float32(b2))),
                           eps=float(np.float32(eps)))
    for t in range(1, steps + 1):
        g = grads_exact(t, K, P)
        o.step_adam(g, [32] * K, params, m, v, lr, b1, b2, eps, t, prev)
        tp.grad = torch.tensor(np.mean(np.stack(g).astype(np.float64), axis=0))
        opt.step()
        st = opt.state[tp]
        assert np.allclose(params, tp.detach().numpy(), rtol=2e-6, atol=2e-7), t
        assert np.allclose(m, st["exp_avg"].numpy(), rtol=2e-6, atol=1e-8), t
        assert np.allclose(v, st["exp_avg_sq"].numpy(), rtol=2e-6, atol=1e-10), t
        assert np.array_equal(prev, np.mean(np.stack(g).astype(np.float64), axis=0).astype(np.float32))


def test_constant_gradient_closed_form():
    # m_t = c (1 - b1^t), v_t = c^2 (1 - b2^t): the corrected estimates are c and c^2 at every
    # step, so theta_t = theta_0 - t lr c / (|c| + eps)
    P, c, lr, eps = 5, -0.75, 0.125, 0.25
    o = Oracle(2, P, [0, P], F32)
    params = np.full(P, 2.0, np.float32); m = np.zeros(P, np.float32); v = np.zeros(P, np.float32); prev = np.zeros(P, np.float32)
    g = [np.full(P, c, np.float32)] * 2
    for t in range(1, 9):
        st = o.step_adam(g, [3, 5], params, m, v, lr, 0.9, 0.999, eps, t, prev)
        assert np.allclose(params, 2.0 - t * lr * c / (abs(c) + eps), rtol=1e-6)
        assert np.allclose(m, c * (1 - np.float32(0.9) ** t), rtol=1e-6)
        assert np.allclose(v, c * c * (1 - float(np.float32(0.999)) ** t), rtol=1e-5)
        ghat = c / (abs(c) + eps)
        assert math.isclose(st[12], ghat, rel_tol=1e-6) and abs(st[13]) < 1e-9 and st[14] < 1e-4 and st[15] == 0


def test_first_step_is_sign_like_and_scale_invariant():
    P = 64
    g = grads_exact(3, 3, P)
    b = [32, 64, 96]
    o = Oracle(3, P, [0, P], F32)
    outs = []
    for alpha in (1.0, 8.0):
        params = np.ones(P, np.float32); m = np.zeros(P, np.float32); v = np.zeros(P, np.float32); prev = np.zeros(P, np.float32)
        o.step_adam([alpha * x for x in g], b, params, m, v, 0.5, 0.9, 0.999, 0.0, 1, prev)
        outs.append((params.copy(), prev.copy()))
    agg = outs[0][1]
    expect = np.where(agg != 0, 1.0 - 0.5 * np.sign(agg), np.nan)
    ok = agg != 0
    assert np.allclose(outs[0][0][ok], expect[ok], rtol=1e-6)        # eps = 0, t = 1: update = lr * sign(g)
    assert np.allclose(outs[0][0][ok], outs[1][0][ok], rtol=1e-6)    # gradients x8: same step


def test_bias_correction_uses_t():
    P = 8
    g = grads_exact(5, 2, P)
    o = Oracle(2, P, [0, P], F32)
    res = {}
    for t in (1, 7):
        params = np.zeros(P, np.float32); m = np.zeros(P, np.float32); v = np.zeros(P, np.float32); prev = np.zeros(P, np.float32)
        o.step_adam(g, [1, 1], params, m, v, 1.0, 0.5, 0.75, 0.0, t, prev)
        res[t] = params.copy()
    # from zero state: mhat = (1-b1) g / (1-b1^t), vhat = (1-b2) g^2 / (1-b2^t)
    gg = (g[0].astype(np.float64) + g[1]) / 2
    for t in (1, 7):
        mh = 0.5 * gg / (1 - 0.5 ** t); vh = 0.25 * gg * gg / (1 - 0.75 ** t)
        ok = gg != 0
        assert np.allclose(res[t][ok], (-mh / np.sqrt(vh))[ok], rtol=1e-6)


def test_gradient_statistics_do_not_depend_on_the_optimizer():
    K, P = 4, 999
    r = np.random.default_rng(9)
    g = [r.standard_normal(P).astype(np.float32) for _ in range(K)]
    b = [32, 64, 96, 128]
    seg = [0, 10, 500, P]
    prev0 = r.standard_normal(P).astype(np.float32)
    o = Oracle(K, P, seg, F32)
    st_sgd = o.step(g, b, np.zeros(P, np.float32), np.zeros(P, np.float32), 0.1, 0.9, prev0.copy())
    v = np.full(P, 0.5, np.float32)
    st_adam = o.step_adam(g, b, np.zeros(P, np.float32), np.zeros(P, np.float32), v, 0.1, 0.9, 0.999, 1e-8, 3, prev0.copy())
    assert np.array_equal(st_sgd[:12], st_adam[:12]) and np.array_equal(st_sgd[16:], st_adam[16:])
    assert np.all(st_sgd[12:16] == 0) and st_adam[13] > 0
    # the normalised-gradient statistics against their definition in numpy fp64
    G = np.stack(g).astype(np.float64); w = np.array(b) / sum(b)
    gg = w @ G
    vh = (float(np.float32(0.999)) * 0.5 + (1 - float(np.float32(0.999))) * gg * gg) / (1 - float(np.float32(0.999)) ** 3)
    gh = gg / (np.sqrt(vh) + float(np.float32(1e-8)))
    assert math.isclose(st_adam[12], gh.mean(), rel_tol=1e-5, abs_tol=1e-7)
    assert math.isclose(st_adam[13], gh.var(), rel_tol=1e-5)
    assert math.isclose(st_adam[14], gh.std(), rel_tol=1e-5)


def test_adam_argument_errors():
    o = Oracle(2, 4, [0, 4], F32)
    z = lambda: np.zeros(4, np.float32)
    g = [z(), z()]
    for kw in (dict(t=0), dict(b1=1.0), dict(b2=-0.1), dict(eps=-1.0)):
        a = dict(t=1, b1=0.9, b2=0.999, eps=1e-8); a.update(kw)
        with pytest.raises(OracleError):
            o.step_adam(g, [1, 1], z(), z(), z(), 0.1, a["b1"], a["b2"], a["eps"], a["t"], z())
