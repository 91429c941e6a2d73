"""Thin ctypes binding of the C ABI in include/dmx.h: same names, argument marshalling only.

Every step of the path runs in the CUDA library. There is no CPU fallback: if the shared
object is missing or fails to load, importing callers get an error.
"""
from __future__ import annotations

import ctypes
import os

from . import build as _build

F32, BF16 = 0, 1
OK = 0
ERR_ARG, ERR_SEGMENTS, ERR_BATCH, ERR_ALIGN, ERR_NOMEM, ERR_CUDA, ERR_HANDLE, ERR_LIMIT, ERR_GUARD = -1, -2, -3, -4, -5, -6, -7, -8, -9
STATIC_MAX_SEGMENTS, STATIC_SCRATCH_BYTES = 512, 1 << 20
ST_B_TOTAL, ST_AGG_SQNORM, ST_TR_SIGMA, ST_G2, ST_GNS, ST_COS_PREV, ST_DOT_PREV, ST_PREV_SQNORM = range(8)
ST_SIGMA2_NORM, ST_SIGMA_NORM, ST_WMEAN_SQNORM, ST_FLAGS = 8, 9, 10, 11
ST_HDR = 16
FLAG_NONFINITE, FLAG_G2_NONPOS, FLAG_COS_UNDEF, FLAG_SINGLE, FLAG_INTERNAL, FLAG_BOUNDS = 1, 2, 4, 8, 16, 32

EXPORTS = ("dmx_create", "dmx_state_len", "dmx_step", "dmx_step_adam", "dmx_step_host", "dmx_step_static", "dmx_set_profiling", "dmx_get_profile",
           "dmx_launches_per_step", "dmx_destroy", "dmx_strerror", "dmx_last_cuda_error", "dmx_agg_create",
           "dmx_agg_push", "dmx_agg_destroy", "dmx_ctl_num_features", "dmx_ctl_num_weights", "dmx_ctl_decide", "dmx_plan_chunks",
           "dmx_shard_range", "dmx_shard_segments", "dmx_partials_len", "dmx_step_partial", "dmx_step_adam_partial",
           "dmx_finalize_partials", "dmx_check_guards", "dmx_selftest_wait", "dmx_scratch_info")
CTL_ACTIONS = (-100, -25, 0, 25, 100)

_lib = None


class DmxError(RuntimeError):
    def __init__(self, code, where=""):
        self.code = code
        super().__init__("%s: %s (%d)" % (where or "dmx", strerror(code), code))


def lib():
    """Load lib/libdmx.so (built in-tree by `python -m paper_2510_08522_b200.build`). With the
    environment variable DMX_CHECKED_BUILD=1 the checked build lib/libdmx_checked.so is loaded
    instead (`python -m paper_2510_08522_b200.build --checked`): same ABI, every table and scratch
    index range-tested on the device."""
    global _lib
    if _lib is None:
        path = _build.lib_path("libdmx_checked.so" if os.environ.get("DMX_CHECKED_BUILD") == "1" else "libdmx.so")
        if not os.path.exists(path):
            raise RuntimeError("CUDA library %s is not built; run `python -m paper_2510_08522_b200.build`" % path)
        L = ctypes.CDLL(path)
        vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float
        L.dmx_create.argtypes = [i32, i64, vp, i32, i32, ctypes.POINTER(vp)]
        L.dmx_create.restype = i32
        L.dmx_state_len.argtypes = [vp]
        L.dmx_state_len.restype = i32
        L.dmx_step.argtypes = [vp, vp, vp, vp, vp, f32, f32, vp, vp, vp]
        L.dmx_step.restype = i32
        L.dmx_step_host.argtypes = [vp, vp, vp, vp, vp, vp, f32, f32, vp, vp, vp, vp]
        L.dmx_step_host.restype = i32
        L.dmx_step_adam.argtypes = [vp, vp, vp, vp, vp, vp, f32, f32, f32, f32, i64, vp, vp, vp]
        L.dmx_step_adam.restype = i32
        L.dmx_step_static.argtypes = [i32, i64, vp, i32, i32, vp, vp, vp, vp, f32, f32, vp, vp, vp]
        L.dmx_step_static.restype = i32
        L.dmx_agg_create.argtypes = [i32, i32, ctypes.POINTER(vp)]
        L.dmx_agg_create.restype = i32
        L.dmx_agg_push.argtypes = [vp, vp, vp, ctypes.POINTER(i32), vp]
        L.dmx_agg_push.restype = i32
        L.dmx_agg_destroy.argtypes = [vp]
        L.dmx_agg_destroy.restype = i32
        L.dmx_ctl_num_features.argtypes = [i32]
        L.dmx_ctl_num_features.restype = i32
        L.dmx_ctl_num_weights.argtypes = [i32, i32]
        L.dmx_ctl_num_weights.restype = i64
        L.dmx_ctl_decide.argtypes = [i32, i32, i32, i32, vp, vp, vp, vp, i32, i32, i32, f32, f32, f32, f32, i32, i32,
                                     vp, vp, vp, vp, vp, vp, vp]
        L.dmx_ctl_decide.restype = i32
        L.dmx_plan_chunks.argtypes = [i64, i32, i32, i32, i32, vp, vp, vp, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.dmx_plan_chunks.restype = i32
        L.dmx_shard_range.argtypes = [i64, i32, i32, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.dmx_shard_range.restype = i32
        L.dmx_shard_segments.argtypes = [vp, i32, i64, i64, vp]
        L.dmx_shard_segments.restype = i32
        L.dmx_partials_len.argtypes = [vp]
        L.dmx_partials_len.restype = i32
        L.dmx_step_partial.argtypes = [vp, vp, vp, vp, vp, f32, f32, vp, vp, vp]
        L.dmx_step_partial.restype = i32
        L.dmx_step_adam_partial.argtypes = [vp, vp, vp, vp, vp, vp, f32, f32, f32, f32, i64, vp, vp, vp]
        L.dmx_step_adam_partial.restype = i32
        L.dmx_finalize_partials.argtypes = [i32, i32, vp, vp, i32, i64, vp, vp]
        L.dmx_finalize_partials.restype = i32
        L.dmx_set_profiling.argtypes = [vp, i32]
        L.dmx_set_profiling.restype = i32
        L.dmx_get_profile.argtypes = [vp, ctypes.POINTER(f32), ctypes.POINTER(f32)]
        L.dmx_get_profile.restype = i32
        L.dmx_launches_per_step.argtypes = [vp]
        L.dmx_launches_per_step.restype = i32
        L.dmx_scratch_info.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.dmx_scratch_info.restype = i32
        L.dmx_check_guards.argtypes = [vp]
        L.dmx_check_guards.restype = i32
        L.dmx_selftest_wait.argtypes = [vp, ctypes.c_uint32, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_double), vp]
        L.dmx_selftest_wait.restype = i32
        L.dmx_destroy.argtypes = [vp]
        L.dmx_destroy.restype = i32
        L.dmx_strerror.argtypes = [i32]
        L.dmx_strerror.restype = ctypes.c_char_p
        L.dmx_last_cuda_error.argtypes = []
        L.dmx_last_cuda_error.restype = i32
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().dmx_strerror(int(code)).decode()


def dmx_create(K, P, seg_offsets, grad_dtype=F32):
    """-> (code, handle). seg_offsets: sequence of S+1 ints (host)."""
    seg = (ctypes.c_int64 * len(seg_offsets))(*[int(v) for v in seg_offsets])
    h = ctypes.c_void_p()
    rc = lib().dmx_create(int(K), int(P), seg, len(seg_offsets) - 1, int(grad_dtype), ctypes.byref(h))
    return rc, h


def dmx_state_len(h) -> int:
    return lib().dmx_state_len(h)


def dmx_step(h, grad_ptrs, batch_sizes, params, momentum, lr, beta, prev_agg, out_state, stream=0) -> int:
    """All buffer arguments are raw device addresses (ints); grad_ptrs / batch_sizes are
    host sequences of length K."""
    K = len(grad_ptrs)
    gp = (ctypes.c_void_p * K)(*[int(p) for p in grad_ptrs])
    bs = (ctypes.c_int32 * K)(*[int(b) for b in batch_sizes])
    return lib().dmx_step(h, gp, bs, int(params), int(momentum), float(lr), float(beta), int(prev_agg),
                          int(out_state), int(stream) if stream else None)


def dmx_step_host(h, host_grad_ptrs, staging_ptrs, batch_sizes, params, momentum, lr, beta, prev_agg,
                  out_state_dev, out_state_host, stream=0) -> int:
    """Gradients in host memory (raw host addresses), staged into caller-owned device buffers;
    synchronous: out_state_host (raw host address) is filled on return."""
    K = len(host_grad_ptrs)
    hp = (ctypes.c_void_p * K)(*[int(p) for p in host_grad_ptrs])
    sp = (ctypes.c_void_p * K)(*[int(p) for p in staging_ptrs])
    bs = (ctypes.c_int32 * K)(*[int(b) for b in batch_sizes])
    return lib().dmx_step_host(h, hp, sp, bs, int(params), int(momentum), float(lr), float(beta), int(prev_agg),
                               int(out_state_dev), int(out_state_host), int(stream) if stream else None)


def dmx_step_adam(h, grad_ptrs, batch_sizes, params, first_moment, second_moment, lr, beta1, beta2, eps, t, prev_agg,
                  out_state, stream=0) -> int:
    """The step with the Adam update; t is the 1-based step count. Raw device addresses as dmx_step."""
    K = len(grad_ptrs)
    gp = (ctypes.c_void_p * K)(*[int(p) for p in grad_ptrs])
    bs = (ctypes.c_int32 * K)(*[int(b) for b in batch_sizes])
    return lib().dmx_step_adam(h, gp, bs, int(params), int(first_moment), int(second_moment), float(lr), float(beta1),
                               float(beta2), float(eps), int(t), int(prev_agg), int(out_state),
                               int(stream) if stream else None)


def dmx_step_static(K, P, seg_offsets, grad_dtype, grad_ptrs, batch_sizes, params, momentum, lr, beta, prev_agg,
                    out_state, stream=0) -> int:
    """The step without a handle and without any allocation (fixed scratch inside the library;
    one call at a time per GPU). Buffer arguments are raw device addresses."""
    seg = (ctypes.c_int64 * len(seg_offsets))(*[int(v) for v in seg_offsets])
    K = int(K)
    gp = (ctypes.c_void_p * K)(*[int(p) for p in grad_ptrs])
    bs = (ctypes.c_int32 * K)(*[int(b) for b in batch_sizes])
    return lib().dmx_step_static(K, int(P), seg, len(seg_offsets) - 1, int(grad_dtype), gp, bs, int(params),
                                 int(momentum), float(lr), float(beta), int(prev_agg), int(out_state),
                                 int(stream) if stream else None)


def dmx_agg_create(state_len, k):
    """-> (code, handle) of a k-step window over state vectors of length state_len."""
    a = ctypes.c_void_p()
    rc = lib().dmx_agg_create(int(state_len), int(k), ctypes.byref(a))
    return rc, a


def dmx_agg_push(a, out_state, window_out, stream=0):
    """-> (code, emitted). Raw device addresses; window_out has 2*state_len floats (mean, then std)."""
    e = ctypes.c_int(0)
    rc = lib().dmx_agg_push(a, int(out_state), int(window_out), ctypes.byref(e), int(stream) if stream else None)
    return rc, e.value


def dmx_agg_destroy(a) -> int:
    return lib().dmx_agg_destroy(a)


def dmx_ctl_num_features(M) -> int:
    return lib().dmx_ctl_num_features(int(M))


def dmx_ctl_num_weights(M, H) -> int:
    return lib().dmx_ctl_num_weights(int(M), int(H))


def dmx_ctl_decide(K, M, H, state_len, window, aux, batch, weights, cols, coef, b_min, b_max, uniforms, next_batch,
                   action, reward, logits, features, stream=0) -> int:
    """The controller's decision for all K workers. Buffer arguments are raw device addresses (0 = NULL);
    cols = (col_acc, col_gain, col_titer); coef = (alpha, beta_t, delta, eta)."""
    def p(x):
        return int(x) if x else None
    return lib().dmx_ctl_decide(int(K), int(M), int(H), int(state_len), p(window), p(aux), p(batch), p(weights),
                                int(cols[0]), int(cols[1]), int(cols[2]), float(coef[0]), float(coef[1]),
                                float(coef[2]), float(coef[3]), int(b_min), int(b_max), p(uniforms), p(next_batch),
                                p(action), p(reward), p(logits), p(features), p(stream))


def ctl_decide(K, M, H, state_len, window, aux, batch, weights, cols=(-1, -1, -1), coef=(1.0, 0.0, 0.0, 0.0),
               b_min=32, b_max=1024, uniforms=None, stream=None):
    """Torch convenience over dmx_ctl_decide: device tensors in, a dict of new device tensors out
    (next_batch, action: int32 [K]; reward: [K]; logits: [K, 5]; features: [K, F])."""
    import torch
    dev = window.device
    F = dmx_ctl_num_features(M)
    if F < 0 or weights.numel() != dmx_ctl_num_weights(M, H) or window.numel() != 2 * state_len or batch.numel() != K:
        raise DmxError(ERR_ARG, "dmx_ctl_decide")
    if (M > 0 and aux.numel() != K * M) or (uniforms is not None and uniforms.numel() != K):
        raise DmxError(ERR_ARG, "dmx_ctl_decide")
    for t, dt in ((window, torch.float32), (batch, torch.int32), (weights, torch.float32)):
        if t.dtype != dt or not t.is_cuda or not t.is_contiguous():
            raise DmxError(ERR_ARG, "dmx_ctl_decide (tensor)")
    out = dict(next_batch=torch.empty(K, dtype=torch.int32, device=dev), action=torch.empty(K, dtype=torch.int32, device=dev),
               reward=torch.empty(K, dtype=torch.float32, device=dev),
               logits=torch.empty((K, len(CTL_ACTIONS)), dtype=torch.float32, device=dev),
               features=torch.empty((K, F), dtype=torch.float32, device=dev))
    if stream is None:
        stream = torch.cuda.current_stream(dev).cuda_stream
    rc = dmx_ctl_decide(K, M, H, state_len, window.data_ptr(), aux.data_ptr() if M > 0 else 0, batch.data_ptr(),
                        weights.data_ptr(), cols, coef, b_min, b_max, uniforms.data_ptr() if uniforms is not None else 0,
                        out["next_batch"].data_ptr(), out["action"].data_ptr(), out["reward"].data_ptr(),
                        out["logits"].data_ptr(), out["features"].data_ptr(), stream)
    if rc != OK:
        raise DmxError(rc, "dmx_ctl_decide")
    return out


def dmx_shard_range(P, nshards, shard):
    """-> (code, lo, hi): the parameter range of one shard (host only)."""
    lo, hi = ctypes.c_int64(0), ctypes.c_int64(0)
    rc = lib().dmx_shard_range(int(P), int(nshards), int(shard), ctypes.byref(lo), ctypes.byref(hi))
    return rc, lo.value, hi.value


def dmx_shard_segments(seg_offsets, lo, hi):
    """-> (code, shard_offsets): the problem's segment table clipped to [lo, hi) and shifted (host only)."""
    n = len(seg_offsets)
    seg = (ctypes.c_int64 * n)(*[int(v) for v in seg_offsets])
    out = (ctypes.c_int64 * n)()
    rc = lib().dmx_shard_segments(seg, n - 1, int(lo), int(hi), out)
    return rc, list(out)


def dmx_partials_len(h) -> int:
    return lib().dmx_partials_len(h)


def dmx_step_partial(h, grad_ptrs, batch_sizes, params, momentum, lr, beta, prev_agg, partials, stream=0) -> int:
    """dmx_step on a parameter shard: raw fp64 sums to `partials` (device address) instead of a state vector."""
    K = len(grad_ptrs)
    gp = (ctypes.c_void_p * K)(*[int(p) for p in grad_ptrs])
    bs = (ctypes.c_int32 * K)(*[int(b) for b in batch_sizes])
    return lib().dmx_step_partial(h, gp, bs, int(params), int(momentum), float(lr), float(beta), int(prev_agg),
                                  int(partials) if partials else None, int(stream) if stream else None)


def dmx_step_adam_partial(h, grad_ptrs, batch_sizes, params, first_moment, second_moment, lr, beta1, beta2, eps, t,
                          prev_agg, partials, stream=0) -> int:
    K = len(grad_ptrs)
    gp = (ctypes.c_void_p * K)(*[int(p) for p in grad_ptrs])
    bs = (ctypes.c_int32 * K)(*[int(b) for b in batch_sizes])
    return lib().dmx_step_adam_partial(h, gp, bs, int(params), int(first_moment), int(second_moment), float(lr),
                                       float(beta1), float(beta2), float(eps), int(t), int(prev_agg),
                                       int(partials) if partials else None, int(stream) if stream else None)


def dmx_finalize_partials(K, S, batch_sizes, partials, adam, P_total, out_state, stream=0) -> int:
    """The state vector from the shards' summed partials (device addresses)."""
    bs = (ctypes.c_int32 * len(batch_sizes))(*[int(b) for b in batch_sizes])
    return lib().dmx_finalize_partials(int(K), int(S), bs, int(partials) if partials else None, int(bool(adam)),
                                       int(P_total), int(out_state) if out_state else None,
                                       int(stream) if stream else None)


def dmx_plan_chunks(P, K, grad_dtype, tile_elems, resident_ctas):
    """-> (code_or_count, first_tile, num_tiles, group_stride, group_tiles, grid): the fused pass's work
    list as dmx_create would build it (host only; lists of ints)."""
    R, G = ctypes.c_int(0), ctypes.c_int(0)
    n = lib().dmx_plan_chunks(int(P), int(K), int(grad_dtype), int(tile_elems), int(resident_ctas), None, None, None, 0,
                              ctypes.byref(R), ctypes.byref(G))
    if n < 0:
        return n, [], [], [], 0, 0
    a, b, c = (ctypes.c_int32 * n)(), (ctypes.c_int32 * n)(), (ctypes.c_int32 * n)()
    n = lib().dmx_plan_chunks(int(P), int(K), int(grad_dtype), int(tile_elems), int(resident_ctas), a, b, c, n,
                              ctypes.byref(R), ctypes.byref(G))
    return n, list(a), list(b), list(c), R.value, G.value


def dmx_set_profiling(h, on) -> int:
    return lib().dmx_set_profiling(h, int(bool(on)))


def dmx_get_profile(h):
    """-> (code, fused_ms, finalize_ms) of the handle's last step."""
    a, b = ctypes.c_float(), ctypes.c_float()
    rc = lib().dmx_get_profile(h, ctypes.byref(a), ctypes.byref(b))
    return rc, a.value, b.value


def dmx_launches_per_step(h) -> int:
    return lib().dmx_launches_per_step(h)


def dmx_scratch_info(h):
    """-> (code, grid, nchunks, nslots) of the handle's launch plan."""
    g, c, n = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0)
    rc = lib().dmx_scratch_info(h, ctypes.byref(g), ctypes.byref(c), ctypes.byref(n))
    return rc, g.value, c.value, n.value


def dmx_check_guards(h) -> int:
    return lib().dmx_check_guards(h)


def dmx_selftest_wait(h, polls, stream=0):
    """-> (code, timed_out, waited_ms): one warp waits `polls` polls on a barrier nothing completes."""
    t, ms = ctypes.c_int(0), ctypes.c_double(0.0)
    rc = lib().dmx_selftest_wait(h, int(polls), ctypes.byref(t), ctypes.byref(ms), int(stream) if stream else None)
    return rc, t.value, ms.value


def dmx_destroy(h) -> int:
    return lib().dmx_destroy(h)


def dmx_last_cuda_error() -> int:
    return lib().dmx_last_cuda_error()


class Dmx:
    """Convenience owner of a handle for torch callers: tensors in, raw pointers through the C ABI."""

    def __init__(self, K, P, seg_offsets, grad_dtype=F32):
        import torch
        self._torch = torch
        self.K, self.P, self.S, self.dtype = int(K), int(P), len(seg_offsets) - 1, int(grad_dtype)
        rc, self._h = dmx_create(K, P, seg_offsets, grad_dtype)
        if rc != OK:
            self._h = None
            raise DmxError(rc, "dmx_create")
        self.state_len = dmx_state_len(self._h)

    def step(self, grads, batch_sizes, params, momentum, lr, beta, prev_agg, out_state=None, stream=None):
        torch = self._torch
        want = torch.float32 if self.dtype == F32 else torch.bfloat16
        if len(grads) != self.K or len(batch_sizes) != self.K:
            raise DmxError(ERR_ARG, "dmx_step")
        for g in grads:
            if g.dtype != want or not g.is_cuda or not g.is_contiguous() or g.numel() != self.P:
                raise DmxError(ERR_ARG, "dmx_step (gradient tensor)")
        for t in (params, momentum, prev_agg):
            if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous() or t.numel() != self.P:
                raise DmxError(ERR_ARG, "dmx_step (state tensor)")
        if out_state is None:
            out_state = torch.empty(self.state_len, dtype=torch.float32, device=params.device)
        elif out_state.dtype != torch.float32 or out_state.numel() != self.state_len or not out_state.is_cuda:
            raise DmxError(ERR_ARG, "dmx_step (out_state)")
        if stream is None:
            stream = torch.cuda.current_stream(params.device).cuda_stream
        rc = dmx_step(self._h, [g.data_ptr() for g in grads], batch_sizes, params.data_ptr(), momentum.data_ptr(),
                      lr, beta, prev_agg.data_ptr(), out_state.data_ptr(), stream)
        if rc != OK:
            raise DmxError(rc, "dmx_step")
        return out_state

    def step_adam(self, grads, batch_sizes, params, first_moment, second_moment, lr, beta1, beta2, eps, t, prev_agg,
                  out_state=None, stream=None):
        torch = self._torch
        want = torch.float32 if self.dtype == F32 else torch.bfloat16
        if len(grads) != self.K or len(batch_sizes) != self.K:
            raise DmxError(ERR_ARG, "dmx_step_adam")
        for g in grads:
            if g.dtype != want or not g.is_cuda or not g.is_contiguous() or g.numel() != self.P:
                raise DmxError(ERR_ARG, "dmx_step_adam (gradient tensor)")
        for x in (params, first_moment, second_moment, prev_agg):
            if x.dtype != torch.float32 or not x.is_cuda or not x.is_contiguous() or x.numel() != self.P:
                raise DmxError(ERR_ARG, "dmx_step_adam (state tensor)")
        if out_state is None:
            out_state = torch.empty(self.state_len, dtype=torch.float32, device=params.device)
        if stream is None:
            stream = torch.cuda.current_stream(params.device).cuda_stream
        rc = dmx_step_adam(self._h, [g.data_ptr() for g in grads], batch_sizes, params.data_ptr(),
                           first_moment.data_ptr(), second_moment.data_ptr(), lr, beta1, beta2, eps, t,
                           prev_agg.data_ptr(), out_state.data_ptr(), stream)
        if rc != OK:
            raise DmxError(rc, "dmx_step_adam")
        return out_state

    def step_host(self, host_grads, staging, batch_sizes, params, momentum, lr, beta, prev_agg, out_state_dev,
                  out_state_host, stream=None):
        """host_grads: K pinned CPU tensors; staging: K device tensors; out_state_host: pinned CPU tensor."""
        torch = self._torch
        if stream is None:
            stream = torch.cuda.current_stream(params.device).cuda_stream
        rc = dmx_step_host(self._h, [g.data_ptr() for g in host_grads], [g.data_ptr() for g in staging], batch_sizes,
                           params.data_ptr(), momentum.data_ptr(), lr, beta, prev_agg.data_ptr(),
                           out_state_dev.data_ptr(), out_state_host.data_ptr(), stream)
        if rc != OK:
            raise DmxError(rc, "dmx_step_host")
        return out_state_host

    def set_profiling(self, on=True):
        rc = dmx_set_profiling(self._h, on)
        if rc != OK:
            raise DmxError(rc, "dmx_set_profiling")

    def profile(self):
        rc, a, b = dmx_get_profile(self._h)
        if rc != OK:
            raise DmxError(rc, "dmx_get_profile")
        return a, b

    @property
    def launches_per_step(self):
        return dmx_launches_per_step(self._h)

    def check_guards(self):
        rc = dmx_check_guards(self._h)
        if rc != OK:
            raise DmxError(rc, "dmx_check_guards")

    def close(self):
        if getattr(self, "_h", None):
            dmx_destroy(self._h)
            self._h = None

    __del__ = close


class ShardedDmx:
    """One parameter shard of a problem (shard `shard` of `nshards`), for torch callers.

    `step_partial` runs the fused pass on views [lo:hi) of the full-length tensors and returns the
    shard's raw sums (a float64 device tensor); the caller adds the shards' tensors (an all-reduce
    when the shards live on different GPUs, see dist_util.allreduce_sum) and calls `finalize`.
    """

    def __init__(self, K, P, seg_offsets, grad_dtype, nshards, shard):
        import torch
        self._torch = torch
        self.K, self.P, self.S, self.dtype = int(K), int(P), len(seg_offsets) - 1, int(grad_dtype)
        rc, self.lo, self.hi = dmx_shard_range(P, nshards, shard)
        if rc != OK:
            raise DmxError(rc, "dmx_shard_range")
        self.state_len = ST_HDR + self.K + 2 * self.S
        self.partials_len = self.K + 5 + 2 * self.S
        self._h = None
        if self.hi > self.lo:
            rc, seg = dmx_shard_segments(seg_offsets, self.lo, self.hi)
            if rc != OK:
                raise DmxError(rc, "dmx_shard_segments")
            rc, self._h = dmx_create(K, self.hi - self.lo, seg, grad_dtype)
            if rc != OK:
                self._h = None
                raise DmxError(rc, "dmx_create")

    def step_partial(self, grads, batch_sizes, params, momentum, lr, beta, prev_agg, adam=None, stream=None, local=False):
        """adam: None for SGD with momentum, else (second_moment, beta2, eps, t) with beta = beta1.
        local=False: every tensor has the whole problem's length and the shard works on [lo:hi);
        local=True: every tensor holds the shard's range only (hi - lo elements, element lo first)."""
        torch = self._torch
        part = torch.zeros(self.partials_len, dtype=torch.float64, device=params.device)
        if self._h is None:                      # an empty shard contributes zeros
            return part
        if stream is None:
            stream = torch.cuda.current_stream(params.device).cuda_stream
        esz = 2 if self.dtype == BF16 else 4
        lo = 0 if local else self.lo
        need = (self.hi - self.lo) if local else self.P
        for x in list(grads) + [params, momentum, prev_agg]:
            if x.numel() < need or not x.is_contiguous():
                raise DmxError(ERR_ARG, "dmx_step_partial (tensor length)")
        gp = [g.data_ptr() + lo * esz for g in grads]
        off = lo * 4
        if adam is None:
            rc = dmx_step_partial(self._h, gp, batch_sizes, params.data_ptr() + off, momentum.data_ptr() + off, lr, beta,
                                  prev_agg.data_ptr() + off, part.data_ptr(), stream)
        else:
            second, beta2, eps, t = adam
            rc = dmx_step_adam_partial(self._h, gp, batch_sizes, params.data_ptr() + off, momentum.data_ptr() + off,
                                       second.data_ptr() + off, lr, beta, beta2, eps, t, prev_agg.data_ptr() + off,
                                       part.data_ptr(), stream)
        if rc != OK:
            raise DmxError(rc, "dmx_step_partial")
        return part

    def finalize(self, batch_sizes, partials_sum, adam=False, out_state=None, stream=None):
        torch = self._torch
        if out_state is None:
            out_state = torch.empty(self.state_len, dtype=torch.float32, device=partials_sum.device)
        if stream is None:
            stream = torch.cuda.current_stream(partials_sum.device).cuda_stream
        rc = dmx_finalize_partials(self.K, self.S, batch_sizes, partials_sum.data_ptr(), adam, self.P,
                                   out_state.data_ptr(), stream)
        if rc != OK:
            raise DmxError(rc, "dmx_finalize_partials")
        return out_state

    def close(self):
        if getattr(self, "_h", None):
            dmx_destroy(self._h)
            self._h = None

    __del__ = close
