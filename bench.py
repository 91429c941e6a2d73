#!/usr/bin/env python
"""Benchmark of the gradient step: `python bench.py --gpus N --steps K --warmup W`.

A step is one pass of the whole hot path (fused aggregate + statistics + SGD-momentum update,
then finalize) over one batch of synthetic gradients. Metric: achieved GB/s of algorithmic
HBM bytes, P*(K*e + 24) per step, with steps/s beside it. Gradients of every step are
generated on the device between the timed regions; each step is bracketed by CUDA events on
the stream it is launched on, and the total is the sum of those regions (max over ranks).
Inputs (>= 17 GB per step at the timed workloads) are far larger than L2, so no flush is needed.

With N > 1 the path runs as N independent replicas (one process per GPU, no data-path
collective): the job's value is N * bytes / max-over-ranks time.

`--impl reference` times the CPU oracle instead (rank 0 only), on bounded samples.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "dmx_step_GBps"
UNIT = "GB/s"


def kernel_source_digest():
    h = hashlib.sha256()
    for rel in ("paper_2510_08522_b200/csrc/dmx_kernels.cuh", "paper_2510_08522_b200/csrc/dmx.cu"):
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def recorded_traffic(workload_name):
    """DRAM bytes per launch of the fused kernel from the committed ncu capture, if the
    kernel sources are still the ones that were captured; else None."""
    try:
        with open(os.path.join(ROOT, "profiles", "pipe_kernel_dram_traffic.json")) as f:
            rec = json.load(f)
        if rec.get("kernel_source_digest") != kernel_source_digest():
            return None
        return rec.get("traffic_bytes_per_launch", {}).get(workload_name)
    except Exception:
        return None


class ClockSampler:
    """nvidia-smi clock/throttle samples during the timed region (reading only)."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.path = index, None, "/tmp/dmx_clocks_%d_%d.csv" % (os.getpid(), index)

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                p = [x.strip() for x in line.split(",")]
                if len(p) < 7:
                    continue
                try:
                    sm.append(float(p[0])); mx.append(float(p[1]))
                except ValueError:
                    continue
                for n, v in zip(names, p[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            # under-load samples: the upper half of the observed clocks
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def world_is_one():
    return int(os.environ.get("WORLD_SIZE", "1")) == 1


def step_bytes(wl, optimizer):
    """Algorithmic HBM bytes of one step (Adam reads and writes one more fp32 state stream)."""
    return wl.bytes_per_step + (8 * wl.P if optimizer == "adam" else 0)


L2_FLUSH_BELOW = 4 << 30      # workloads streaming less than this per step get an L2 flush between steps
L2_BYTES = 126 << 20          # B200's L2
B2B_MIN_BYTES = 512 << 20     # ... and those streaming at least this much (4 x L2) are also timed back to back


def run_workload(wl, steps, warmup, device, e2e_steps, sample_clocks=True, profile=True, optimizer="sgd", sustained=True,
                 back_to_back=0):
    """Time `steps` steps of workload `wl` on `device`. Returns a dict of local measurements.
    Workloads whose step streams only a few times the L2's size get a 512 MB write between the
    (untimed) input generation and the timed step, so that no step starts on a warm L2."""
    import torch
    import paper_2510_08522_b200 as D
    from paper_2510_08522_b200 import workload as W

    torch.cuda.set_device(device)
    dp = W.DeviceProblem(wl, device)
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    out_state = torch.empty(d.state_len, dtype=torch.float32, device=device)
    d.set_profiling(profile)
    second = torch.zeros(wl.P, dtype=torch.float32, device=device) if optimizer == "adam" else None
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=device) if step_bytes(wl, optimizer) < L2_FLUSH_BELOW else None
    tcount = [0]

    def one_step(b):
        if optimizer == "adam":
            tcount[0] += 1
            d.step_adam(dp.grads, b, dp.params, dp.momentum, second, 1e-3, 0.9, 0.999, 1e-8, tcount[0], dp.prev_agg, out_state)
        else:
            d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg, out_state)

    for _ in range(warmup):
        b = dp.fill()
        one_step(b)
        dp.advance()
    torch.cuda.synchronize()
    sampler = ClockSampler(device.index if device.index is not None else 0)
    if sample_clocks:
        sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    fused, fin = [], []
    wall0 = time.time()
    for s in range(steps):
        b = dp.fill()                     # untimed: next step's gradients
        if flush is not None:
            flush.zero_()                 # untimed: evicts the freshly written gradients and the state from L2
        ev[s][0].record()
        one_step(b)
        ev[s][1].record()
        if profile:
            a, f = d.profile()            # waits for this step
            fused.append(a); fin.append(f)
        dp.advance()
    torch.cuda.synchronize()
    wall = time.time() - wall0
    clocks = sampler.stop() if sample_clocks else None
    times = [e0.elapsed_time(e1) for e0, e1 in ev]
    flags = int(out_state[11].item())
    res = dict(total_ms=sum(times), times=times, fused_ms=fused, finalize_ms=fin, clocks=clocks, flags=flags,
               wall_s=wall, launches=steps * d.launches_per_step, l2_flushed=flush is not None)
    del flush

    # end to end: gradients start in pinned host memory, the state vector ends in host memory
    if e2e_steps > 0 and optimizer == "sgd":
        host = []
        # one pinned buffer per worker at N = 1; with several ranks on one host that would pin N * K * P * e bytes
        # (174 GB at N = 8), so each rank then copies K times from a quarter of the buffers (the bytes per step
        # and the host link's load are the same)
        n_pinned = wl.K if world_is_one() else max(1, wl.K // 4)
        try:
            for g in dp.grads[:n_pinned]:
                hbuf = torch.empty(g.shape, dtype=g.dtype, pin_memory=True)
                hbuf.copy_(g)
                host.append(hbuf)
        except RuntimeError:
            host = host[:1]               # not enough pinnable memory: reuse one pinned buffer K times
        out_host = torch.empty(d.state_len, dtype=torch.float32, pin_memory=True)
        b = dp.batch_sizes()
        stream = torch.cuda.current_stream(device)
        hsrc = [host[k % len(host)] for k in range(wl.K)]
        d.step_host(hsrc, dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg, out_state, out_host)
        t_e2e = []
        for _ in range(e2e_steps):
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            d.step_host(hsrc, dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg, out_state, out_host)
            e1.record(stream)
            torch.cuda.synchronize()
            t_e2e.append(e0.elapsed_time(e1))
        res["e2e_ms"] = sum(t_e2e) / len(t_e2e)
        res["h2d_bytes"] = wl.K * wl.P * wl.elem_bytes
        res["d2h_bytes"] = d.state_len * 4
        res["e2e_launches"] = e2e_steps * d.launches_per_step
        del host
    if sustained and sample_clocks and world_is_one() and optimizer == "sgd":
        # the same step launched back to back for about a second on one set of gradients (inputs far larger
        # than L2): the duty cycle of the timed loop above is low (input generation sits between its steps);
        # at full duty the board reaches its power limit and the SM clock drops, which this path feels
        n_sus = max(60, int(1000.0 / max(res["total_ms"] / steps, 0.05)))
        n_sus = min(n_sus, 400)
        b = dp.batch_sizes()
        sus_sampler = ClockSampler(device.index if device.index is not None else 0)
        sus_sampler.start()
        sus = []
        for _ in range(n_sus):
            one_step(b)
            a, _f = d.profile()
            sus.append(a)
        torch.cuda.synchronize()
        sus_clocks = sus_sampler.stop()
        tail = sorted(sus[-max(20, n_sus // 4):])
        res["sustained"] = {"fused_kernel_ms": tail[len(tail) // 2], "first_fused_kernel_ms": sus[0], "launches": n_sus,
                            "clocks": sus_clocks}
    if back_to_back > 0:
        # whole steps launched straight behind one another inside ONE pair of events (only for workloads
        # whose step streams several times the L2's size, so that no step finds its inputs cached): what a
        # step costs the device once the launch and event latency around an isolated step is out of the picture
        b = dp.batch_sizes()
        for _ in range(3):
            one_step(b)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(back_to_back):
            one_step(b)
        e1.record()
        torch.cuda.synchronize()
        res["back_to_back_ms"] = e0.elapsed_time(e1) / back_to_back
    d.close()
    if sample_clocks and world_is_one():
        # what plain reads of the same gradient buffers stream at in this run (context for the roofline)
        try:
            res["read_probe_gbps"] = W.read_probe_gbps(dp.grads)
        except Exception:
            res["read_probe_gbps"] = None
    res["problem"] = dp
    return res


def oracle_sample(wl, elems, nthreads, reps=1, device=None):
    """Time the CPU oracle, as it stands, on the first `elems` parameters of workload `wl`
    (same structure, same generator). Returns (seconds per sample step, elems, threads)."""
    import numpy as np
    from oracle.dmx_oracle import Oracle
    from paper_2510_08522_b200 import workload as W
    sub = wl.scaled(P=min(elems, wl.P), S=min(wl.S, 64))
    raw = None
    try:
        import torch
        if torch.cuda.is_available():
            dp = W.DeviceProblem(sub, device if device is not None else "cuda:0")
            b = dp.fill()
            torch.cuda.synchronize()
            if sub.dtype == W.F32:
                raw = [g.cpu().numpy() for g in dp.grads]
            else:
                raw = [g.view(torch.int16).cpu().numpy().view(np.uint16) for g in dp.grads]
            params, mom, prev = dp.params.cpu().numpy(), dp.momentum.cpu().numpy(), dp.prev_agg.cpu().numpy()
            seg = dp.seg
            del dp
    except Exception:
        raw = None
    if raw is None:
        hp = W.HostProblem(sub)
        raw, b = hp.grads()
        params, mom, prev, seg = hp.params0.copy(), np.zeros(sub.P, np.float32), np.zeros(sub.P, np.float32), hp.seg
    orc = Oracle(sub.K, sub.P, seg, sub.dtype)
    ts = []
    for _ in range(reps):
        t0 = time.perf_counter()
        orc.step(raw, b, params, mom, sub.lr, sub.beta, prev, nthreads=nthreads)
        ts.append(time.perf_counter() - t0)
    return ts, sub


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=4, help="index into the workload table (default: the largest)")
    ap.add_argument("--also", type=int, default=3, help="second workload reported under 'also' (-1: none)")
    ap.add_argument("--all-workloads", type=int, default=1,
                    help="1: also time the remaining workloads briefly and list them under 'workloads' (N=1 only)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-sample-elems", type=int, default=128 << 20, help="0: skip the CPU-baseline leg")
    ap.add_argument("--sustained", type=int, default=1,
                    help="1: after the timed steps, also launch the step back to back for about a second (N=1 only)")
    ap.add_argument("--optimizer", default="sgd", choices=["sgd", "adam"],
                    help="update applied by the step (the metric's workload uses sgd)")
    ap.add_argument("--P", type=int, default=0, help="run the workload's structure at another size (profiling captures)")
    args = ap.parse_args()

    from paper_2510_08522_b200 import workload as W
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wl = W.WORKLOADS[args.workload]
    if args.P:
        wl = wl.scaled(P=args.P)
    ncores = os.cpu_count() or 1
    dtype_name = "f32"   # arithmetic type of the path: fp32 (gradients stored as fp32 or bf16)
    config = {"workload": wl.name, "K": wl.K, "P": wl.P, "S": wl.S,
              "grad_dtype": "bf16" if wl.dtype == W.BF16 else "f32", "optimizer": args.optimizer,
              "bytes_per_step": step_bytes(wl, args.optimizer),
              "l2": ("flushed between steps (512 MB write)" if step_bytes(wl, args.optimizer) < L2_FLUSH_BELOW
                     else "inputs larger than L2 (gradients regenerated between steps)"), "parallelism": "replicas x%d" % args.gpus}

    if args.impl == "reference":
        if rank != 0:
            return 0
        elems = min(args.cpu_sample_elems // 4, wl.P)
        ts, sub = oracle_sample(wl, elems, ncores, reps=args.warmup + args.steps)
        ts = ts[args.warmup:]
        sec = sum(ts) / len(ts)
        val = sub.bytes_per_step / sec / 1e9
        sample = "first %d of %d parameters of %s per step, all K workers; oracle as it stands, %d threads" % (
            sub.P, wl.P, wl.name, ncores)
        line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
                "steps_per_s_full_size_equivalent": val * 1e9 / wl.bytes_per_step,
                "cpu_baseline": {"value": val, "unit": UNIT, "cores": ncores, "kind": "oracle", "sample": sample},
                "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return 0

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the gradient step has no CPU path")
    from paper_2510_08522_b200 import dist_util as DU
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    DU.init(world, "nccl")
    DU.barrier()
    torch.cuda.synchronize()
    res = run_workload(wl, args.steps, args.warmup, device, args.e2e_steps, optimizer=args.optimizer,
                       sustained=bool(args.sustained))
    torch.cuda.synchronize()
    DU.barrier()
    total_ms = DU.max_over_ranks(res["total_ms"])
    e2e_ms = DU.max_over_ranks(res.get("e2e_ms", 0.0))
    flags_any = int(DU.max_over_ranks(float(res["flags"] & 16)))
    del res["problem"]
    torch.cuda.empty_cache()

    def side_workload(wlx, nsteps):
        """A workload reported beside the main one: whole steps timed without the per-kernel
        events (so the two launches keep their dependent-launch overlap), then the fused kernel's
        own time from a second pass with them."""
        peak_x, _ = measured_peak()
        nbx = step_bytes(wlx, args.optimizer)
        b2b = 100 if B2B_MIN_BYTES <= nbx < L2_FLUSH_BELOW else 0
        r_plain = run_workload(wlx, nsteps, args.warmup, device, 0, sample_clocks=False, profile=False, optimizer=args.optimizer,
                               back_to_back=b2b)
        del r_plain["problem"]
        torch.cuda.empty_cache()
        r_prof = run_workload(wlx, nsteps, args.warmup, device, 0, sample_clocks=False, profile=True, optimizer=args.optimizer)
        del r_prof["problem"]
        torch.cuda.empty_cache()
        msx = r_plain["total_ms"] / len(r_plain["times"])
        fx = sum(r_prof["fused_ms"]) / len(r_prof["fused_ms"])
        out = {"workload": wlx.name, "value": nbx / msx / 1e6, "unit": UNIT, "ms_per_step": msx,
               "ms_per_step_median": statistics.median(r_plain["times"]),
               "steps_per_s": 1e3 / msx, "bytes_per_step": nbx, "fused_kernel_ms": fx,
               "roofline_frac": nbx / fx / 1e6 / peak_x,
               "l2": "flushed between steps" if r_plain["l2_flushed"] else "inputs larger than L2"}
        if nbx < L2_BYTES:
            out["note"] = "a step's bytes are smaller than the L2 (flushed before every step): a latency figure, not an HBM figure"
        if "back_to_back_ms" in r_plain:
            out["back_to_back"] = {"ms_per_step": r_plain["back_to_back_ms"], "value": nbx / r_plain["back_to_back_ms"] / 1e6,
                                   "unit": UNIT, "steps": b2b,
                                   "what": "whole steps launched back to back between one pair of events, no flush: "
                                           "a step streams more than four times the L2's size"}
        return out

    also = None
    if args.also >= 0 and args.also != args.workload and world == 1:
        also = side_workload(W.WORKLOADS[args.also], max(3, args.steps // 2))

    others = []
    if args.all_workloads and world == 1 and not args.P:
        for i, wlo in enumerate(W.WORKLOADS):
            if i not in (args.workload, args.also):
                others.append(side_workload(wlo, max(5, args.steps // 2)))

    if rank != 0:
        DU.finish()
        return 0

    ms_per_step = total_ms / args.steps
    nbytes = step_bytes(wl, args.optimizer)
    value = world * nbytes / ms_per_step / 1e6
    peak, peak_kind = measured_peak()
    fused_ms = sum(res["fused_ms"]) / len(res["fused_ms"])
    achieved = nbytes / fused_ms / 1e6
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": dtype_name, "data": "synthetic", "config": config,
            "ms_per_step_median": statistics.median(res["times"]),
            "steps_per_s": world * 1e3 / ms_per_step,
            "frac_of_8TBps_nominal": value / world / 8000.0,
            "clocks": res["clocks"],
            "gpu_launches": res["launches"],
            "kernel_ms": {"fused": fused_ms, "finalize": sum(res["finalize_ms"]) / len(res["finalize_ms"])},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": UNIT, "frac": achieved / peak,
                         "peak_kind": "of " + peak_kind,
                         "traffic": recorded_traffic(wl.name) if args.optimizer == "sgd" else None,
                         "algorithmic_bytes_per_launch": nbytes},
            "internal_error_flag": bool(flags_any)}
    if res.get("read_probe_gbps"):
        line["roofline"]["read_only_probe"] = {"value": res["read_probe_gbps"], "unit": UNIT,
                                               "what": "plain 128-bit reads of the same K gradient buffers, same run"}
    if res.get("sustained"):
        sm = res["sustained"]
        line["sustained"] = {"value": nbytes / sm["fused_kernel_ms"] / 1e6, "unit": UNIT,
                             "frac_of_peak": nbytes / sm["fused_kernel_ms"] / 1e6 / peak,
                             "fused_kernel_ms": sm["fused_kernel_ms"], "first_fused_kernel_ms": sm["first_fused_kernel_ms"],
                             "launches": sm["launches"], "clocks": sm["clocks"],
                             "what": "the fused kernel launched back to back (no input generation between), median of the "
                                     "last quarter: the board's power limit lowers the SM clock in this regime"}
    if "e2e_ms" in res:
        line["e2e"] = {"value": world * wl.bytes_per_step / e2e_ms / 1e6, "unit": UNIT,
                       "h2d_bytes_per_step": res["h2d_bytes"], "d2h_bytes_per_step": res["d2h_bytes"],
                       "ms_per_step": e2e_ms, "steps": args.e2e_steps,
                       "note": "gradients copied from pinned host memory every step; params, momentum and prev_agg stay resident"}
    if also:
        line["also"] = also
    if others:
        line["workloads"] = others
    if world == 1 and args.cpu_sample_elems > 0:
        ts, sub = oracle_sample(wl, args.cpu_sample_elems, ncores, reps=1, device=device)
        line["cpu_baseline"] = {"value": sub.bytes_per_step / ts[0] / 1e9, "unit": UNIT, "cores": ncores, "kind": "oracle",
                                "sample": "first %d of %d parameters of %s, all K workers, one step (%.2f s)" % (
                                    sub.P, wl.P, wl.name, ts[0])}
    print(json.dumps(line))
    DU.finish()
    return 0


if __name__ == "__main__":
    sys.exit(main())
