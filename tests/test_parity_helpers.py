"""The torch forms of the comparison helpers (used where numpy is too slow) equal the numpy forms,
and the per-element floor on N_s applies to short segments only. CPU only."""
import numpy as np
import pytest
import torch

from tests import parity as PT


def _problem(seed=3, K=5, P=4099):
    r = np.random.default_rng(seed)
    grads = [r.standard_normal(P).astype(np.float32) for _ in range(K)]
    b = r.integers(1, 200, K)
    params, mom = r.standard_normal(P).astype(np.float32), r.standard_normal(P).astype(np.float32)
    return grads, b, params, mom


def test_torch_scales_equal_numpy_scales():
    grads, b, params, mom = _problem()
    ref = PT.cond_vectors(grads, b, params, mom, 0.1, 0.9)
    got = PT.cond_vectors_t(torch, [torch.from_numpy(g) for g in grads], b, torch.from_numpy(params), torch.from_numpy(mom), 0.1, 0.9)
    for a, t in zip(ref, got):
        assert np.allclose(a, t.numpy(), rtol=1e-14, atol=0)
    seg = [0, 1, 1, 7, 4000, 4099]
    assert np.allclose(PT.seg_scales(ref[0], seg), PT.seg_scales_t(torch, got[0], seg), rtol=1e-10)


def test_torch_adam_scales_equal_numpy_scales():
    grads, b, params, mom = _problem(seed=6)
    v = np.abs(_problem(seed=7)[2]) * 1e-2
    ref = PT.cond_vectors_adam(grads, b, params, mom, v, 1e-3, 0.9, 0.999, 1e-8, 5)
    got = PT.cond_vectors_adam_t(torch, [torch.from_numpy(g) for g in grads], b, torch.from_numpy(params), torch.from_numpy(mom),
                                 torch.from_numpy(v), 1e-3, 0.9, 0.999, 1e-8, 5)
    for a, t in zip(ref, got):
        assert np.allclose(a, t.numpy(), rtol=1e-12, atol=0)
    seg = [0, 1, 1, 7, 4000, 4099]
    for lo, hi in ((0, 4099), (5, 3000), (3999, 4099)):
        assert np.allclose(PT.seg_scales(ref[0][lo:hi], seg, lo), PT.seg_scales_range_t(torch, got[0][lo:hi], seg, lo), rtol=1e-10)


def test_torch_scales_widen_bf16_exactly():
    grads, b, params, mom = _problem(seed=4)
    gb = [torch.from_numpy(g).to(torch.bfloat16) for g in grads]
    wide = [g.to(torch.float32).numpy() for g in gb]
    ref = PT.cond_vectors(wide, b, params, mom, 0.1, 0.9)
    got = PT.cond_vectors_t(torch, gb, b, torch.from_numpy(params), torch.from_numpy(mom), 0.1, 0.9)
    assert np.allclose(ref[0], got[0].numpy(), rtol=1e-14, atol=0)


def test_torch_error_equals_numpy_error():
    r = np.random.default_rng(5)
    ref = r.standard_normal(1000).astype(np.float32)
    gpu = (ref + 1e-6 * r.standard_normal(1000)).astype(np.float32)
    cond = np.abs(r.standard_normal(1000))
    ref[10] = 0; cond[10] = 0; gpu[10] = 0                      # 0/0 counts as no error
    e = PT.vec_err(gpu, ref, cond)
    assert e == pytest.approx(PT.vec_err_t(torch, torch.from_numpy(gpu), torch.from_numpy(ref), torch.from_numpy(cond)), rel=1e-12)
    gpu[10] = 1e-30                                             # anything against an exact zero is an error
    assert PT.vec_err(gpu, ref, cond) == float("inf")
    assert PT.vec_err_t(torch, torch.from_numpy(gpu), torch.from_numpy(ref), torch.from_numpy(cond)) == float("inf")


def test_floor_on_segment_norm_is_for_short_segments_only():
    K, S = 2, 2
    seg = [0, 8, 8 + PT.SMALL_SEGMENT]
    ref = np.zeros(PT.HDR + K + 2 * S, np.float32)
    ref[0], ref[1], ref[2], ref[3], ref[7] = 3, 2.0, 1.0, 2.0 - 1.0 / 3, 1.0
    ref[4] = ref[2] / ref[3]; ref[8] = ref[2] / (ref[0] * ref[1]); ref[9] = np.sqrt(ref[8]); ref[10] = 1.0
    ref[PT.HDR:PT.HDR + K] = 1.0
    ref[PT.HDR + K:PT.HDR + K + S] = 0.5
    ref[PT.HDR + K + S:] = 1.0
    scale = np.array([100.0, 100.0])
    gpu = ref.copy()
    gpu[PT.HDR + K + S] *= 1 + 5e-4                  # short segment: inside 2e-5 * scale
    PT.check_state(gpu, ref, K, S, seg, [1, 2], seg_scale=scale)
    gpu = ref.copy()
    gpu[PT.HDR + K + S + 1] *= 1 + 5e-4              # long segment: the plain relative bound applies
    with pytest.raises(AssertionError):
        PT.check_state(gpu, ref, K, S, seg, [1, 2], seg_scale=scale)
