"""Pins of the CPU oracle against things that are not the oracle: a hand-computed example,
exact rational brute force, closed forms, invariants and statistical expectations.
The paper prints no numeric value for any gradient statistic, so the mathematics is the pin.
"""
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle.dmx_oracle import BF16, F32, ST, Oracle, OracleError
from paper_2510_08522_b200 import workload as W

HDR = ST["HDR"]


def run(grads, b, seg, params=None, momentum=None, prev=None, lr=0.1, beta=0.9, dtype=F32, nthreads=1):
    K, P = len(grads), len(grads[0])
    want = np.float32 if dtype == F32 else np.uint16
    grads = [np.ascontiguousarray(g, dtype=want) for g in grads]
    z = lambda a: np.zeros(P, np.float32) if a is None else np.array(a, dtype=np.float32)
    params, momentum, prev = z(params), z(momentum), z(prev)
    o = Oracle(K, P, seg, dtype)
    st = o.step(grads, b, params, momentum, lr, beta, prev, nthreads=nthreads)
    return dict(st=st, params=params, momentum=momentum, agg=prev, K=K, S=len(seg) - 1,
                q=st[HDR:HDR + K], V=st[HDR + K:HDR + K + len(seg) - 1], N=st[HDR + K + len(seg) - 1:])


def rnd(seed, K, P, scale=1.0):
    r = np.random.default_rng(seed)
    return [(scale * r.standard_normal(P)).astype(np.float32) for _ in range(K)]


# ---- 0. hand-computed example ------------------------------------------------------------------

def test_hand_example():
    path = os.path.join(os.path.dirname(__file__), "golden", "hand_example_k2.json")
    ex = json.load(open(path))
    r = run(ex["grads"], ex["batch_sizes"], ex["seg_offsets"], ex["params"], ex["momentum"],
            ex["prev_agg"], ex["lr"], ex["beta"])
    e, st = ex["expect"], r["st"]
    assert list(r["agg"]) == e["agg"]
    assert list(r["momentum"]) == e["momentum"]
    assert list(r["params"]) == e["params"]
    for name, key in [("B", "B"), ("A", "A"), ("TRS", "tr_sigma"), ("G2", "G2"), ("GNS", "gns"),
                      ("DOT", "dot"), ("PP", "prev_sqnorm"), ("WQ", "wmean_sqnorm"), ("FLAGS", "flags")]:
        assert st[ST[name]] == e[key], name
    for name, key in [("COS", "cos"), ("SIG2", "sigma2_norm"), ("SIG", "sigma_norm")]:
        assert st[ST[name]] == np.float32(e[key]), name
    assert list(r["q"]) == e["worker_sqnorm"]
    assert list(r["V"]) == e["seg_var"]
    assert list(r["N"]) == e["seg_agg_sqnorm"]
    assert list(st[12:16]) == [0, 0, 0, 0]


# ---- 1. exact rational brute force on tiny problems ----------------------------------------------

def brute(grads, b, seg, params, momentum, prev, lr, beta):
    """The step in exact rational arithmetic, written from the second route to the spread:
    sum_k b_k |x_k|^2 - B |g|^2 per element instead of the centred sum."""
    K, P, S = len(grads), len(grads[0]), len(seg) - 1
    F = Fraction
    x = [[F(float(v)) for v in g] for g in grads]
    B = sum(b)
    g = [sum(F(b[k]) * x[k][j] for k in range(K)) / B for j in range(P)]
    spread = [sum(F(b[k]) * x[k][j] ** 2 for k in range(K)) - B * g[j] ** 2 for j in range(P)]
    out = {}
    out["g"] = g
    out["m"] = [F(float(np.float32(beta))) * F(float(momentum[j])) + g[j] for j in range(P)]
    out["theta"] = [F(float(params[j])) - F(float(np.float32(lr))) * out["m"][j] for j in range(P)]
    out["q"] = [sum(v * v for v in x[k]) for k in range(K)]
    out["A"] = sum(v * v for v in g)
    out["D"] = sum(spread)
    out["V"] = [sum(spread[seg[s]:seg[s + 1]]) / max(K - 1, 1) for s in range(S)]
    out["N"] = [sum(v * v for v in g[seg[s]:seg[s + 1]]) for s in range(S)]
    out["trS"] = out["D"] / (K - 1) if K > 1 else F(0)
    out["G2"] = out["A"] - out["trS"] / B
    out["dot"] = sum(g[j] * F(float(prev[j])) for j in range(P))
    out["pp"] = sum(F(float(v)) ** 2 for v in prev)
    out["wq"] = sum(F(b[k]) * out["q"][k] for k in range(K)) / B
    return out


@pytest.mark.parametrize("seed,K,P,seg", [
    (0, 2, 1, [0, 1]),
    (1, 3, 7, [0, 3, 3, 7]),
    (2, 4, 16, [0, 5, 6, 16]),
    (3, 4, 13, [0, 0, 13]),
    (4, 1, 5, [0, 2, 5]),
    (5, 4, 9, [0, 9, 9]),
])
def test_brute_force_rationals(seed, K, P, seg):
    r = np.random.default_rng(seed)
    grads = [r.integers(-8, 9, P).astype(np.float32) / 4 for _ in range(K)]
    b = [int(v) for v in r.choice([1, 2, 3, 4, 8, 16, 5], K)]
    params = r.integers(-8, 9, P).astype(np.float32) / 8
    mom = r.integers(-8, 9, P).astype(np.float32) / 8
    prev = r.integers(-8, 9, P).astype(np.float32) / 8
    ref = brute(grads, b, seg, params, mom, prev, 0.25, 0.5)
    got = run(grads, b, seg, params, mom, prev, 0.25, 0.5)
    st = got["st"]
    f32 = lambda fr: np.float32(float(fr))
    # vectors: the oracle's fp64 result rounded to fp32 must be the correctly rounded exact value
    assert [f32(v) for v in ref["g"]] == list(got["agg"])
    assert [f32(v) for v in ref["m"]] == list(got["momentum"])
    assert [f32(v) for v in ref["theta"]] == list(got["params"])
    close = lambda a, fr: math.isclose(float(a), float(fr), rel_tol=3e-7, abs_tol=1e-12)
    assert close(st[ST["B"]], sum(b))
    assert close(st[ST["A"]], ref["A"])
    assert close(st[ST["TRS"]], ref["trS"])
    assert math.isclose(float(st[ST["G2"]]), float(ref["G2"]), rel_tol=3e-7, abs_tol=3e-7 * float(ref["A"]))
    assert close(st[ST["DOT"]], ref["dot"])
    assert close(st[ST["PP"]], ref["pp"])
    assert close(st[ST["WQ"]], ref["wq"])
    for k in range(K):
        assert close(got["q"][k], ref["q"][k])
    for s in range(len(seg) - 1):
        assert close(got["V"][s], ref["V"][s]), s
        assert close(got["N"][s], ref["N"][s]), s
        if seg[s] == seg[s + 1]:
            assert got["V"][s] == 0 and got["N"][s] == 0
    if ref["G2"] > 0:
        assert close(st[ST["GNS"]], ref["trS"] / ref["G2"])
    else:
        assert st[ST["GNS"]] == 0 and int(st[ST["FLAGS"]]) & 2
    if K == 1:
        assert int(st[ST["FLAGS"]]) & 8 and st[ST["TRS"]] == 0 and st[ST["G2"]] == st[ST["A"]]
    if ref["A"] > 0 and ref["pp"] > 0:
        assert close(st[ST["COS"]], float(ref["dot"]) / math.sqrt(float(ref["A"] * ref["pp"])))
    if ref["A"] > 0:
        assert close(st[ST["SIG2"]], ref["trS"] / (sum(b) * ref["A"]))
        assert close(st[ST["SIG"]], math.sqrt(float(ref["trS"] / (sum(b) * ref["A"]))))


# ---- 2. closed forms ---------------------------------------------------------------------------

def test_identical_workers():
    x = rnd(7, 1, 1000)[0]
    r = run([x.copy() for _ in range(5)], [32, 64, 96, 128, 17], [0, 400, 1000])
    st = r["st"]
    assert np.array_equal(r["agg"], x)                       # g = g_k
    A = float(np.sum(x.astype(np.float64) ** 2))
    assert st[ST["TRS"]] <= 1e-24 * A * 5 and np.all(r["V"] <= 1e-24 * A)
    assert math.isclose(st[ST["A"]], A, rel_tol=2e-7)
    assert math.isclose(st[ST["G2"]], A, rel_tol=2e-7)
    assert np.allclose(r["q"], A, rtol=2e-7)
    assert st[ST["GNS"]] <= 1e-20


def test_equal_batches_reduce_to_plain_mean_and_two_batch_estimator():
    K, P, bsz = 6, 777, 48
    g = rnd(11, K, P)
    r = run(g, [bsz] * K, [0, P])
    G = np.stack(g).astype(np.float64)
    mean = G.mean(axis=0)
    assert np.array_equal(r["agg"], mean.astype(np.float32))
    small = (G ** 2).sum(axis=1).mean()        # mean |g_k|^2 : batch b
    big = (mean ** 2).sum()                    # |g|^2        : batch K b
    # two-batch-size estimators (McCandlish et al. 2018, appendix A): B_small = b, B_big = K b
    tr_two = (small - big) / (1.0 / bsz - 1.0 / (K * bsz))
    g2_two = (K * bsz * big - bsz * small) / (K * bsz - bsz)
    assert math.isclose(r["st"][ST["TRS"]], tr_two, rel_tol=1e-6)
    assert math.isclose(r["st"][ST["G2"]], g2_two, rel_tol=1e-6, abs_tol=1e-6 * big)
    assert math.isclose(r["st"][ST["TRS"]], bsz / (K - 1) * ((G ** 2).sum() - K * big), rel_tol=1e-6)


@pytest.mark.parametrize("b1,b2,x1,x2", [(1, 1, 3.0, 1.0), (32, 96, 0.5, -1.25), (7, 5, 2.0, 2.0)])
def test_two_groups_pooled_variance(b1, b2, x1, x2):
    r = run([[x1], [x2]], [b1, b2], [0, 1])
    expect = b1 * b2 / (b1 + b2) * (x1 - x2) ** 2
    assert math.isclose(r["st"][ST["TRS"]], expect, rel_tol=2e-7, abs_tol=0)
    assert math.isclose(r["agg"][0], (b1 * x1 + b2 * x2) / (b1 + b2), rel_tol=2e-7)


def test_momentum_closed_form():
    # constant gradient c, m_0 = 0: m_n = c (1-beta^n)/(1-beta),
    # theta_n = theta_0 - lr c [ n/(1-beta) - beta (1-beta^n)/(1-beta)^2 ]
    c, lr, beta, n = 0.75, 0.125, 0.5, 12
    P = 3
    o = Oracle(2, P, np.array([0, P]), F32)
    params = np.full(P, 2.0, np.float32); mom = np.zeros(P, np.float32); prev = np.zeros(P, np.float32)
    g = [np.full(P, c, np.float32), np.full(P, c, np.float32)]
    for _ in range(n):
        o.step(g, [3, 5], params, mom, lr, beta, prev)
    m_n = c * (1 - beta ** n) / (1 - beta)
    th_n = 2.0 - lr * c * (n / (1 - beta) - beta * (1 - beta ** n) / (1 - beta) ** 2)
    assert np.allclose(mom, m_n, rtol=1e-6) and np.allclose(params, th_n, rtol=1e-6)
    assert np.array_equal(prev, g[0])
    # first step with m = 0 gives m = g and theta = theta_0 - lr g exactly
    params = np.full(P, 2.0, np.float32); mom = np.zeros(P, np.float32); prev = np.zeros(P, np.float32)
    o.step(g, [3, 5], params, mom, lr, beta, prev)
    assert np.all(mom == np.float32(c)) and np.all(params == np.float32(2.0 - lr * c))


def test_lr_beta_are_the_fp32_values():
    # lr = 0.1f is not 0.1: theta' must be the rounding of theta - (double)0.1f * m'
    P = 4
    x = rnd(5, 2, P)
    r = run(x, [1, 1], [0, P], params=[1, 2, 3, 4], momentum=[1, 1, 1, 1], lr=0.1, beta=0.9)
    g = (x[0].astype(np.float64) + x[1]) / 2
    m = float(np.float32(0.9)) * 1.0 + g
    th = np.array([1, 2, 3, 4], np.float64) - float(np.float32(0.1)) * m
    assert np.array_equal(r["momentum"], m.astype(np.float32))
    assert np.array_equal(r["params"], th.astype(np.float32))


# ---- 3. invariants -----------------------------------------------------------------------------

def test_worker_permutation():
    K, P = 5, 2000
    g = rnd(3, K, P)
    b = [32, 64, 96, 128, 256]
    seg = [0, 100, 1500, 2000]
    r0 = run(g, b, seg, prev=rnd(4, 1, P)[0])
    perm = [3, 0, 4, 1, 2]
    r1 = run([g[i] for i in perm], [b[i] for i in perm], seg, prev=rnd(4, 1, P)[0])
    assert np.array_equal(r0["agg"], r1["agg"])
    assert np.allclose(r0["st"][:HDR], r1["st"][:HDR], rtol=1e-6, atol=0)
    assert np.allclose(r0["q"][perm], r1["q"], rtol=1e-7)
    assert np.allclose(r0["V"], r1["V"], rtol=1e-6) and np.allclose(r0["N"], r1["N"], rtol=1e-6)


def test_sums_and_two_routes():
    K, P = 7, 5000
    g = rnd(21, K, P)
    b = [16, 32, 48, 64, 80, 96, 1024]
    r = run(g, b, [0, 1, 1, 2500, 4999, 5000])
    st = r["st"]
    B = sum(b)
    assert st[ST["B"]] == B
    assert math.isclose(r["V"].astype(np.float64).sum(), st[ST["TRS"]], rel_tol=1e-6)
    assert math.isclose(r["N"].astype(np.float64).sum(), st[ST["A"]], rel_tol=1e-6)
    Qw = float(np.dot(np.array(b, np.float64), r["q"].astype(np.float64)))
    assert math.isclose(st[ST["WQ"]], Qw / B, rel_tol=1e-6)
    D = st[ST["TRS"]] * (K - 1)
    assert abs(D - (Qw - B * st[ST["A"]])) <= 1e-6 * Qw        # D = Qw - B A
    assert math.isclose(st[ST["G2"]], st[ST["A"]] - st[ST["TRS"]] / B, rel_tol=1e-5, abs_tol=1e-6 * st[ST["A"]])
    # per-element vectors against the definition evaluated by numpy in fp64
    G = np.stack(g).astype(np.float64)
    w = np.array(b, np.float64) / B
    assert np.array_equal(r["agg"], (w @ G).astype(np.float32)) or np.allclose(r["agg"], w @ G, rtol=1e-6, atol=1e-9)
    assert np.allclose(r["q"], (G ** 2).sum(axis=1), rtol=1e-6)


def test_scaling_laws():
    K, P = 4, 3000
    g = rnd(9, K, P)
    b = np.array([32, 64, 96, 128])
    seg = [0, 1000, 3000]
    prev = rnd(10, 1, P)[0]
    r = run(g, b, seg, prev=prev)
    r2 = run(g, 4 * b, seg, prev=prev)                      # all batch sizes x4
    assert np.array_equal(r["agg"], r2["agg"])
    for nm in ("A", "COS", "DOT", "PP", "WQ"):
        assert math.isclose(r["st"][ST[nm]], r2["st"][ST[nm]], rel_tol=1e-6)
    assert math.isclose(4 * r["st"][ST["TRS"]], r2["st"][ST["TRS"]], rel_tol=1e-6)
    assert np.allclose(4 * r["V"], r2["V"], rtol=1e-6)
    assert math.isclose(r["st"][ST["SIG2"]], r2["st"][ST["SIG2"]], rel_tol=1e-5)
    r3 = run([2 * x for x in g], b, seg, prev=prev)            # all gradients x2
    assert np.array_equal(2 * r["agg"], r3["agg"])
    for nm in ("A", "TRS", "G2", "WQ"):
        assert math.isclose(4 * r["st"][ST[nm]], r3["st"][ST[nm]], rel_tol=1e-6)
    for nm in ("GNS", "COS", "SIG2", "SIG"):
        assert math.isclose(r["st"][ST[nm]], r3["st"][ST[nm]], rel_tol=1e-5)


def test_segment_refinement():
    K, P = 3, 4000
    g = rnd(13, K, P)
    b = [32, 64, 128]
    r = run(g, b, [0, 1500, 4000])
    r2 = run(g, b, [0, 700, 1500, 1501, 4000])
    assert np.allclose(r["st"][:HDR + K], r2["st"][:HDR + K], rtol=1e-7)
    assert math.isclose(r["V"][0], r2["V"][0] + r2["V"][1], rel_tol=1e-6)
    assert math.isclose(r["V"][1], r2["V"][2] + r2["V"][3], rel_tol=1e-6)
    assert math.isclose(r["N"][0], r2["N"][0] + r2["N"][1], rel_tol=1e-6)
    assert math.isclose(r["N"][1], r2["N"][2] + r2["N"][3], rel_tol=1e-6)


def test_cosine_against_self_and_negation_and_first_step():
    K, P = 3, 1000
    g = rnd(17, K, P)
    b = [32, 32, 64]
    r = run(g, b, [0, P])
    assert r["st"][ST["COS"]] == 0 and int(r["st"][ST["FLAGS"]]) & 4          # zero prev_agg
    agg = r["agg"].copy()
    assert math.isclose(run(g, b, [0, P], prev=agg)["st"][ST["COS"]], 1.0, rel_tol=1e-6)
    assert math.isclose(run(g, b, [0, P], prev=-agg)["st"][ST["COS"]], -1.0, rel_tol=1e-6)
    # orthogonal prev_agg: P=2, g = (1, 0), prev = (0, 5)
    r = run([[1.0, 0.0], [1.0, 0.0]], [1, 1], [0, 2], prev=[0.0, 5.0])
    assert r["st"][ST["COS"]] == 0 and r["st"][ST["PP"]] == 25 and not int(r["st"][ST["FLAGS"]]) & 4


def test_negative_g2_is_reported_raw_with_flag():
    # two workers pointing in opposite directions: A = 0 < tr/B
    r = run([[1.0, -1.0], [-1.0, 1.0]], [8, 8], [0, 2])
    st = r["st"]
    assert st[ST["A"]] == 0 and st[ST["TRS"]] == 8 * 8 / 16 * 8 and st[ST["G2"]] == -st[ST["TRS"]] / 16
    assert st[ST["GNS"]] == 0 and int(st[ST["FLAGS"]]) & 2 and int(st[ST["FLAGS"]]) & 4
    assert st[ST["SIG2"]] == 0 and st[ST["SIG"]] == 0


def test_nonfinite_inputs_flagged_not_trapped():
    g = rnd(1, 2, 8)
    g[1][3] = np.inf
    r = run(g, [1, 1], [0, 8])
    assert int(r["st"][ST["FLAGS"]]) & 1
    assert not np.isfinite(r["q"][1]) and np.isfinite(r["q"][0])
    assert not np.isfinite(r["agg"][3]) and np.all(np.isfinite(np.delete(r["agg"], 3)))


def test_bf16_inputs_are_widened_exactly():
    K, P = 3, 515
    gf = rnd(23, K, P)
    bits = [W.f32_to_bf16_bits(x) for x in gf]
    widened = [W.bf16_bits_to_f32(v) for v in bits]
    b = [16, 48, 512]
    r16 = run(bits, b, [0, 100, P], dtype=BF16, prev=gf[0])
    r32 = run(widened, b, [0, 100, P], dtype=F32, prev=gf[0])
    assert np.array_equal(r16["st"], r32["st"]) and np.array_equal(r16["agg"], r32["agg"])
    # bf16 rounding itself: nearest-even on the 16 dropped bits
    assert W.f32_to_bf16_bits(np.array([1.0, 1.00390625, 1.01171875], np.float32)).tolist() == [0x3F80, 0x3F80, 0x3F82]


def test_thread_count_and_streaming_do_not_change_the_result():
    K, P = 3, (2 << 20) + 12345
    g = rnd(29, K, P)
    b = [32, 64, 96]
    seg = [0, 1 << 20, (1 << 20) + 7, P]
    prev = rnd(30, 1, P)[0]
    r1 = run(g, b, seg, prev=prev, nthreads=1)
    r4 = run(g, b, seg, prev=prev, nthreads=4)
    assert np.array_equal(r1["st"], r4["st"]) and np.array_equal(r1["params"], r4["params"])
    o = Oracle(K, P, np.array(seg), F32)
    params = np.zeros(P, np.float32); mom = np.zeros(P, np.float32); pv = prev.copy()
    o.begin(b, 0.1, 0.9)
    cuts = [0, 1 << 20, P]
    for a, e in zip(cuts[:-1], cuts[1:]):
        o.range(a, [x[a:e].copy() for x in g], params[a:e], mom[a:e], pv[a:e], nthreads=2)
    st = o.end()
    assert np.array_equal(st, r1["st"]) and np.array_equal(params, r1["params"]) and np.array_equal(pv, r1["agg"])


def test_argument_errors():
    with pytest.raises(OracleError):
        Oracle(0, 4, [0, 4])
    with pytest.raises(OracleError):
        Oracle(2, 4, [0, 3])
    with pytest.raises(OracleError):
        Oracle(2, 4, [0, 3, 2, 4])
    with pytest.raises(OracleError):
        run(rnd(0, 2, 4), [1, 0], [0, 4])


# ---- 4. statistical pins under the workload generator --------------------------------------------

def test_unbiasedness_under_the_generator():
    # equal noise scale: E tr = P, E |G|^2^ = |mu|^2, E q_k = |mu|^2 + P/b_k
    wl = W.WORKLOADS[0].scaled(P=1 << 18)
    hp = W.HostProblem(wl)
    grads, b = hp.grads()
    r = run(grads, b, hp.seg)
    st, P, K = r["st"], wl.P, wl.K
    mu2 = float(np.sum(hp.mu.astype(np.float64) ** 2))
    assert abs(mu2 / P - 0.01) < 5 * 0.01 * math.sqrt(2.0 / P)
    rel_sd = math.sqrt(2.0 / ((K - 1) * P))
    assert abs(st[ST["TRS"]] / P - 1.0) < 5 * rel_sd
    B = int(b.sum())
    # var(|g|^2) ~ 4 |mu|^2/B + 2P/B^2 ; var of tr/B adds a little: use a generous 6 sigma
    sd_g2 = math.sqrt(4 * mu2 / B + 2 * P / B ** 2 + (rel_sd * P / B) ** 2)
    assert abs(st[ST["G2"]] - mu2) < 6 * sd_g2
    for k in range(K):
        sd = math.sqrt(4 * mu2 / b[k] + 2 * P / b[k] ** 2)
        assert abs(r["q"][k] - (mu2 + P / b[k])) < 6 * sd
    assert abs(st[ST["GNS"]] - P / mu2) < 0.05 * P / mu2          # ~100
    assert np.allclose(r["V"], P / 4, rtol=0.02)


def test_unbiasedness_with_per_worker_noise_scales():
    # worker k has per-sample covariance sigma_k^2 I: E tr^ = P sum_k sigma_k^2 (1 - w_k) / (K-1)
    wl = W.WORKLOADS[4].scaled(P=1 << 16)
    hp = W.HostProblem(wl)
    grads, b = hp.grads()
    r = run(grads, b, hp.seg, dtype=BF16)
    sig = wl.sigma()
    w = b / b.sum()
    expect = wl.P * float(np.sum(sig ** 2 * (1 - w))) / (wl.K - 1)
    assert abs(r["st"][ST["TRS"]] / expect - 1.0) < 0.02
    assert 0.5 <= sig.min() and sig.max() <= 2.0 and 16 <= b.min() and b.max() <= 1024


def _seeded_golden():
    import json
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "seeded_small_k3.json")) as f:
        return json.load(f)


def test_seeded_golden_is_what_the_oracle_computes_and_its_exact_parts_check_by_hand():
    """The stored fixture (written by tests/golden/make_seeded_golden.py) still equals the oracle's
    output, and the parts of it that are exact rationals are recomputed here with Python
    fractions from the definitions."""
    from fractions import Fraction as Fr
    d = _seeded_golden()
    K, P, seg, b = d["K"], d["P"], d["seg_offsets"], d["batch_sizes"]
    grads = [np.array(g, np.float32) for g in d["grads"]]
    params, mom, prev = (np.array(d[k], np.float32) for k in ("params", "momentum", "prev_agg"))
    prev_in = prev.copy()
    st = Oracle(K, P, seg, 0).step(grads, b, params, mom, d["lr"], d["beta"], prev)
    assert [float(v) for v in st] == d["expect"]["state"]
    assert prev.tolist() == d["expect"]["agg"] and mom.tolist() == d["expect"]["momentum"] and params.tolist() == d["expect"]["params"]
    B = sum(b)
    g = [sum(Fr(b[k]) * Fr(float(grads[k][j])) for k in range(K)) / B for j in range(P)]
    assert [float(x) for x in g] == d["expect"]["agg"]
    A = sum(x * x for x in g)
    D = sum(Fr(b[k]) * (Fr(float(grads[k][j])) - g[j]) ** 2 for k in range(K) for j in range(P))
    assert float(A) == d["expect"]["state"][1] and float(D / (K - 1)) == d["expect"]["state"][2]
    assert float(A - D / (K - 1) / B) == d["expect"]["state"][3]
    assert float(sum(g[j] * Fr(float(prev_in[j])) for j in range(P))) == d["expect"]["state"][6]
    S = len(seg) - 1
    for s in range(S):
        Vs = sum(Fr(b[k]) * (Fr(float(grads[k][j])) - g[j]) ** 2 for k in range(K) for j in range(seg[s], seg[s + 1])) / (K - 1)
        assert float(Vs) == d["expect"]["state"][16 + K + s]
        assert float(sum(g[j] ** 2 for j in range(seg[s], seg[s + 1]))) == d["expect"]["state"][16 + K + S + s]
