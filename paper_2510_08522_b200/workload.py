"""Seeded synthetic workloads: the only module the CUDA path's tests and the oracle's tests share.

It holds no arithmetic of the gradient step itself: only a counter-based random generator
(Philox4x32-10, from its published definition: Salmon, Moraes, Dror, Shaw, "Parallel random
numbers: as easy as 1, 2, 3", SC'11), the recipes that turn it into gradients, segment tables
and batch-size schedules, and the bf16 storage conversions.

The five workloads stand in for the gradient traffic of the models the paper trains (VGG and
ResNet variants on CIFAR, Section "Workloads and Datasets") and for a BERT-large sized model,
by size and structure only: no dataset, weights or real gradients are involved.

    mu_j            ~ N(0, 0.01)                  common signal (variance 0.01, std 0.1)
    x_kj            = round_dtype(mu_j + sigma_k * z_kj / sqrt(b_k)),  z ~ N(0,1) i.i.d.
    mu              <- mu + N(0, 1e-3) per element per step (workloads with drift)
    theta_0         ~ N(0, 0.05^2),  m_0 = 0,  prev_agg_0 = 0

Random numbers are addressed, not drawn in sequence: the four normals of elements 4i..4i+3 of
stream (tag, c2, c3) come from Philox counter (i lo, i hi, c2, c3) under key (seed, tag), so
any slice regenerates on its own and the GPU fill kernels and this host twin agree on the
integers (the float transforms agree to rounding).
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

F32, BF16 = 0, 1

TAG_MU, TAG_DRIFT, TAG_NOISE, TAG_THETA, TAG_HOST = 1, 2, 3, 4, 5

MU_STD = 0.1                    # sqrt(0.01)
DRIFT_STD = math.sqrt(1e-3)
THETA_STD = 0.05

_M0, _M1 = 0xD2511F53, 0xCD9E8D57
_W0, _W1 = 0x9E3779B9, 0xBB67AE85
_MASK = 0xFFFFFFFF


def philox4x32(c0, c1, c2, c3, k0, k1):
    """Philox4x32-10 on numpy uint64 arrays holding 32-bit words; returns four such arrays."""
    c0 = np.asarray(c0, dtype=np.uint64); c1 = np.asarray(c1, dtype=np.uint64)
    c2 = np.asarray(c2, dtype=np.uint64); c3 = np.asarray(c3, dtype=np.uint64)
    c0, c1, c2, c3 = np.broadcast_arrays(c0, c1, c2, c3)
    k0 = int(k0) & _MASK
    k1 = int(k1) & _MASK
    m = np.uint64(_MASK)
    sh = np.uint64(32)
    for _ in range(10):
        p0 = np.uint64(_M0) * c0
        p1 = np.uint64(_M1) * c2
        hi0, lo0 = p0 >> sh, p0 & m
        hi1, lo1 = p1 >> sh, p1 & m
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
        k0 = (k0 + _W0) & _MASK
        k1 = (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def normals(seed, tag, c2, c3, j0, n):
    """Standard normals (float64) of elements [j0, j0+n) of stream (tag, c2, c3)."""
    i0, i1 = j0 // 4, (j0 + n + 3) // 4
    idx = np.arange(i0, i1, dtype=np.uint64)
    r = philox4x32(idx & np.uint64(_MASK), idx >> np.uint64(32), c2, c3, seed, tag)
    u = [(x.astype(np.float64) + 0.5) * 2.0 ** -32 for x in r]
    rad0 = np.sqrt(-2.0 * np.log(u[0]))
    rad1 = np.sqrt(-2.0 * np.log(u[2]))
    z = np.empty((i1 - i0, 4), dtype=np.float64)
    z[:, 0] = rad0 * np.cos(2.0 * np.pi * u[1])
    z[:, 1] = rad0 * np.sin(2.0 * np.pi * u[1])
    z[:, 2] = rad1 * np.cos(2.0 * np.pi * u[3])
    z[:, 3] = rad1 * np.sin(2.0 * np.pi * u[3])
    z = z.reshape(-1)
    return z[j0 - 4 * i0: j0 - 4 * i0 + n]


def host_words(seed, purpose, n, c3=0):
    """n uint32 words for host-side draws (tables, batch sizes), word i of (purpose, c3)."""
    idx = np.arange((n + 3) // 4, dtype=np.uint64)
    r = philox4x32(idx, 0, purpose, c3, seed, TAG_HOST)
    return np.stack(r, axis=1).reshape(-1)[:n].astype(np.uint64)


def f32_to_bf16_bits(x):
    """fp32 -> bf16 bit patterns (uint16), round to nearest even; finite inputs."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    return ((u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f32(b):
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# ---------------------------------------------------------------------------------------------
# segment tables


def equal_segments(P, S):
    return np.array([P * s // S for s in range(S + 1)], dtype=np.int64)


def _lognormal_sizes(total, n, seed, purpose):
    """n sizes >= 1 summing to `total`, proportional to exp(1.5 * N(0,1)); the remainder goes
    to the largest. Sizes are not rounded to any multiple, so boundaries fall at every
    residue mod 4 and mod 8, like a real layer table with its bias and norm vectors."""
    z = normals(seed, TAG_HOST, purpose, 1, 0, n)
    ell = np.exp(1.5 * z)
    sizes = np.maximum(1, np.floor(total * ell / ell.sum())).astype(np.int64)
    sizes[np.argmax(sizes)] += total - sizes.sum()
    assert sizes.min() >= 1 and sizes.sum() == total
    return sizes


def lognormal_segments(P, S, seed):
    return np.concatenate([[0], np.cumsum(_lognormal_sizes(P, S, seed, 10))]).astype(np.int64)


def two_heavy_segments(P, S, seed, heavy=((26, 0.65), (28, 0.15))):
    """S segments; the listed ones hold the given fractions of P (together 80 %), the others
    share the rest log-normally (a VGG-like table: two huge dense layers)."""
    sizes = np.zeros(S, dtype=np.int64)
    taken = 0
    for idx, frac in heavy:
        sizes[idx] = int(P * frac)
        taken += sizes[idx]
    rest = [s for s in range(S) if s not in dict(heavy)]
    sizes[rest] = _lognormal_sizes(P - taken, len(rest), seed, 11)
    return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)


# ---------------------------------------------------------------------------------------------
# workloads


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    K: int
    P: int
    S: int
    dtype: int
    steps: int
    seed: int
    segments: str           # "equal" | "lognormal" | "two_heavy"
    batches: str            # "fixed4" | "once32" | "redraw16" | "tiers" | "walk32"
    drift: bool
    sigma_spread: bool = False
    lr: float = 0.1
    beta: float = 0.9

    @property
    def elem_bytes(self):
        return 4 if self.dtype == F32 else 2

    @property
    def bytes_per_step(self):
        """Algorithmic HBM bytes of one step: every gradient element read once; params,
        momentum and prev_agg each read once and written once."""
        return self.P * (self.K * self.elem_bytes + 24)

    def scaled(self, P, steps=None, S=None):
        """Same structure at another size (parity tests at sizes the oracle finishes fast)."""
        return dataclasses.replace(self, name="%s@P=%d" % (self.name, P), P=int(P),
                                   steps=self.steps if steps is None else steps,
                                   S=self.S if S is None else S)

    def segment_table(self):
        if self.segments == "equal":
            return equal_segments(self.P, self.S)
        if self.segments == "lognormal":
            return lognormal_segments(self.P, self.S, self.seed)
        if self.segments == "two_heavy":
            return two_heavy_segments(self.P, self.S, self.seed)
        raise ValueError(self.segments)

    def sigma(self):
        """Per-worker noise scale sigma_k (1 unless the workload spreads it over U(0.5, 2))."""
        if not self.sigma_spread:
            return np.ones(self.K, dtype=np.float64)
        w = host_words(self.seed, 20, self.K).astype(np.float64)
        return 0.5 + 1.5 * (w + 0.5) * 2.0 ** -32

    def batch_sizes(self, step):
        K = self.K
        if self.batches == "fixed4":
            base = np.array([32, 64, 96, 128], dtype=np.int64)
            return np.resize(base, K).astype(np.int32)
        if self.batches == "once32":          # uniform over {32, 64, ..., 256}, drawn once
            return (32 * (1 + host_words(self.seed, 21, K) % 8)).astype(np.int32)
        if self.batches == "redraw16":        # multiples of 16 in [16, 512], redrawn every 10 steps
            return (16 * (1 + host_words(self.seed, 22, K, c3=step // 10) % 32)).astype(np.int32)
        if self.batches == "tiers":           # four tiers, K/4 workers each
            tiers = np.array([32, 64, 128, 256], dtype=np.int64)
            return tiers[(np.arange(K) * 4) // K].astype(np.int32)
        if self.batches == "walk32":          # +-32 every step within [16, 1024]
            b = (32 * (1 + host_words(self.seed, 23, K) % 32)).astype(np.int64)
            for t in range(1, step + 1):
                coin = host_words(self.seed, 24, K, c3=t) & np.uint64(1)
                b = np.clip(b + np.where(coin == 1, 32, -32), 16, 1024)
            return b.astype(np.int32)
        raise ValueError(self.batches)

    def grad_scale(self, step):
        """scale_k = sigma_k / sqrt(b_k), as the fp32 values the fill kernels receive."""
        return (self.sigma() / np.sqrt(self.batch_sizes(step).astype(np.float64))).astype(np.float32)


WORKLOADS = [
    Workload("cfg0-K4-1M-f32", 4, 1_048_576, 4, F32, 1, 0, "equal", "fixed4", False),
    Workload("cfg1-K8-resnet18-f32", 8, 11_689_512, 62, F32, 100, 1, "lognormal", "once32", True),
    Workload("cfg2-K16-resnet50-bf16", 16, 25_557_032, 161, BF16, 200, 2, "lognormal", "redraw16", True),
    Workload("cfg3-K32-vgg16-f32", 32, 138_357_544, 32, F32, 50, 3, "two_heavy", "tiers", True),
    Workload("cfg4-K32-bertlarge-bf16", 32, 340_000_000, 390, BF16, 50, 4, "lognormal", "walk32", True,
             sigma_spread=True),
]


# ---------------------------------------------------------------------------------------------
# host twin of the fill kernels (small sizes; float transforms agree with the GPU to rounding)


class HostProblem:
    """A workload materialised in numpy, one step at a time. Arrays are what `dmx_step`
    and the oracle consume: float32 (or bf16 bit patterns as uint16) gradients, float32 state."""

    def __init__(self, wl: Workload):
        self.wl = wl
        self.seg = wl.segment_table()
        P = wl.P
        self.mu = (MU_STD * normals(wl.seed, TAG_MU, 0, 0, 0, P)).astype(np.float32)
        self.params0 = (THETA_STD * normals(wl.seed, TAG_THETA, 0, 0, 0, P)).astype(np.float32)
        self.step_index = 0

    def grads(self):
        """Gradients of the current step (list of K arrays) and its batch sizes."""
        wl, t = self.wl, self.step_index
        b = wl.batch_sizes(t)
        scale = wl.grad_scale(t)
        out = []
        for k in range(wl.K):
            z = normals(wl.seed, TAG_NOISE, k, t, 0, wl.P).astype(np.float32)
            x = (self.mu + scale[k] * z).astype(np.float32)
            out.append(f32_to_bf16_bits(x) if wl.dtype == BF16 else x)
        return out, b

    def advance(self):
        self.step_index += 1
        if self.wl.drift:
            d = (DRIFT_STD * normals(self.wl.seed, TAG_DRIFT, 0, self.step_index, 0, self.wl.P))
            self.mu = (self.mu + d.astype(np.float32)).astype(np.float32)


# ---------------------------------------------------------------------------------------------
# device side: the same recipes through the fill kernels of lib/libdmx_gen.so


_gen = None


def gen_lib():
    global _gen
    if _gen is None:
        import ctypes
        import os
        from . import build as _build
        path = _build.lib_path("libdmx_gen.so")
        if not os.path.exists(path):
            raise RuntimeError("%s is not built; run `python -m paper_2510_08522_b200.build`" % path)
        L = ctypes.CDLL(path)
        vp, i32, i64, u32, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint32, ctypes.c_float
        L.dmxgen_normal_fill.argtypes = [vp, i64, u32, u32, u32, u32, f32, f32, vp]
        L.dmxgen_normal_add.argtypes = [vp, i64, u32, u32, u32, u32, f32, vp]
        L.dmxgen_grad_fill.argtypes = [vp, i32, vp, i64, u32, u32, u32, u32, f32, vp]
        L.dmxgen_read_probe.argtypes = [vp, i32, i64, vp, vp]
        L.dmxgen_probe_sink_words.argtypes = []
        for f in (L.dmxgen_normal_fill, L.dmxgen_normal_add, L.dmxgen_grad_fill, L.dmxgen_read_probe, L.dmxgen_probe_sink_words):
            f.restype = i32
        _gen = L
    return _gen


class DeviceProblem:
    """A workload resident on one GPU: K gradient buffers, mu, and the fp32 state
    (params, momentum, prev_agg). `fill()` writes the current step's gradients with the fill
    kernels; `advance()` moves to the next step (drift of mu). torch is used for memory only."""

    def __init__(self, wl: Workload, device="cuda:0"):
        import torch
        self.torch = torch
        self.wl = wl
        self.device = torch.device(device)
        self.seg = wl.segment_table()
        P, dev = wl.P, self.device
        gdt = torch.float32 if wl.dtype == F32 else torch.bfloat16
        self.grads = [torch.empty(P, dtype=gdt, device=dev) for _ in range(wl.K)]
        self.mu = torch.empty(P, dtype=torch.float32, device=dev)
        self.params = torch.empty(P, dtype=torch.float32, device=dev)
        self.momentum = torch.zeros(P, dtype=torch.float32, device=dev)
        self.prev_agg = torch.zeros(P, dtype=torch.float32, device=dev)
        self.step_index = 0
        self.reset()

    def _stream(self):
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def _chk(self, rc, what):
        if rc != 0:
            raise RuntimeError("%s failed with %d" % (what, rc))

    def reset(self):
        wl, L = self.wl, gen_lib()
        with self.torch.cuda.device(self.device):
            self._chk(L.dmxgen_normal_fill(self.mu.data_ptr(), wl.P, wl.seed, TAG_MU, 0, 0, 0.0, MU_STD, self._stream()), "mu fill")
            self._chk(L.dmxgen_normal_fill(self.params.data_ptr(), wl.P, wl.seed, TAG_THETA, 0, 0, 0.0, THETA_STD, self._stream()), "theta fill")
        self.momentum.zero_()
        self.prev_agg.zero_()
        self.step_index = 0

    def batch_sizes(self):
        return self.wl.batch_sizes(self.step_index)

    def fill(self, batch=None):
        """Write the gradients of the current step; returns its batch sizes. `batch` replaces
        the workload's own schedule (a controller in the loop): worker k's noise then has scale
        sigma_k / sqrt(batch[k])."""
        wl, L = self.wl, gen_lib()
        if batch is None:
            scale = wl.grad_scale(self.step_index)
        else:
            batch = np.asarray(batch, dtype=np.int32)
            scale = (wl.sigma() / np.sqrt(batch.astype(np.float64))).astype(np.float32)
        with self.torch.cuda.device(self.device):
            for k, g in enumerate(self.grads):
                self._chk(L.dmxgen_grad_fill(g.data_ptr(), wl.dtype, self.mu.data_ptr(), wl.P, wl.seed, TAG_NOISE, k,
                                             self.step_index, float(scale[k]), self._stream()), "grad fill")
        return self.batch_sizes() if batch is None else batch

    def advance(self):
        self.step_index += 1
        if self.wl.drift:
            with self.torch.cuda.device(self.device):
                self._chk(gen_lib().dmxgen_normal_add(self.mu.data_ptr(), self.wl.P, self.wl.seed, TAG_DRIFT, 0,
                                                      self.step_index, DRIFT_STD, self._stream()), "drift")


def read_probe_gbps(tensors, reps=5):
    """Read-only streaming rate (GB/s) over the given equally sized device tensors: the median of
    `reps` timed passes of the generator library's probe kernel after one warm-up pass."""
    import ctypes
    import torch
    L = gen_lib()
    n = len(tensors)
    nbytes = min(t.numel() * t.element_size() for t in tensors) // 16 * 16
    ptrs = (ctypes.c_void_p * n)(*[t.data_ptr() for t in tensors])
    with torch.cuda.device(tensors[0].device):
        sink = torch.zeros(L.dmxgen_probe_sink_words(), dtype=torch.int32, device=tensors[0].device)
    stream = torch.cuda.current_stream(tensors[0].device).cuda_stream
    ts = []
    for i in range(reps + 1):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rc = L.dmxgen_read_probe(ptrs, n, nbytes, sink.data_ptr(), stream)
        e1.record()
        torch.cuda.synchronize()
        if rc != 0:
            raise RuntimeError("dmxgen_read_probe failed: %d" % rc)
        if i:
            ts.append(e0.elapsed_time(e1))
    ts.sort()
    return n * nbytes / ts[len(ts) // 2] / 1e6
