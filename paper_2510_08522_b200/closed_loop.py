"""The whole loop of Algorithm 1 on one GPU, on synthetic gradients: k gradient steps at the
current batch sizes, the window statistics of the state vector, the controller's decision, the
new batch sizes; repeat. Every step of it runs in the CUDA library (dmx_step or dmx_step_adam,
dmx_agg_push, dmx_ctl_decide); the host only carries the K new batch sizes back into the next
steps' arguments. The policy weights are random (training the policy is the paper's PPO agent,
outside this library), so the trajectory shows the mechanics, not a learned schedule.

    python -m paper_2510_08522_b200.closed_loop --workload 1 --cycles 5 --k 4
"""
from __future__ import annotations

import argparse

import numpy as np


def run(workload=1, P=0, cycles=4, k=3, hidden=32, adam=False, sample=True, seed=0, device="cuda:0", verbose=False):
    """Returns the list of per-cycle records: dict(batch, action, reward, gns, cos, sigma_norm)."""
    import torch
    from . import binding as B
    from . import workload as W
    wl = W.WORKLOADS[workload]
    if P:
        wl = wl.scaled(P=P)
    dev = torch.device(device)
    torch.cuda.set_device(dev)
    dp = W.DeviceProblem(wl, dev)
    d = B.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    n = d.state_len
    rc, agg = B.dmx_agg_create(n, k)
    if rc != B.OK:
        raise B.DmxError(rc, "dmx_agg_create")
    state = torch.empty(n, dtype=torch.float32, device=dev)
    window = torch.zeros(2 * n, dtype=torch.float32, device=dev)
    second = torch.zeros(wl.P, dtype=torch.float32, device=dev) if adam else None
    M = 3                                             # accuracy, accuracy gain, iteration time: stand-ins
    rng = np.random.default_rng(seed)
    F = B.dmx_ctl_num_features(M)
    weights = torch.from_numpy(rng.normal(scale=1.0 / np.sqrt(max(F, hidden)),
                                          size=B.dmx_ctl_num_weights(M, hidden)).astype(np.float32)).to(dev)
    batch = np.asarray(dp.batch_sizes(), dtype=np.int32).clip(32, 1024)
    stream = torch.cuda.current_stream(dev).cuda_stream
    records, t = [], 0
    for c in range(cycles):
        for _ in range(k):
            dp.fill(batch)
            t += 1
            if adam:
                d.step_adam(dp.grads, batch, dp.params, dp.momentum, second, 1e-3, 0.9, 0.999, 1e-8, t, dp.prev_agg, state)
            else:
                d.step(dp.grads, batch, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg, state)
            rc, emitted = B.dmx_agg_push(agg, state.data_ptr(), window.data_ptr(), stream)
            if rc != B.OK:
                raise B.DmxError(rc, "dmx_agg_push")
            dp.advance()
        assert emitted == 1
        # metrics the training loop itself would supply (here: synthetic): mean batch accuracy,
        # accuracy gain, iteration time growing with the batch size
        aux = np.stack([0.5 + 0.05 * c + 0.01 * rng.standard_normal(wl.K), 0.02 * rng.standard_normal(wl.K),
                        batch / 1024.0], axis=1).astype(np.float32)
        t_aux = torch.from_numpy(aux).to(dev)
        t_b = torch.from_numpy(batch).to(dev)
        u = torch.from_numpy(rng.random(wl.K).astype(np.float32)).to(dev) if sample else None
        out = B.ctl_decide(wl.K, M, hidden, n, window, t_aux, t_b, weights, cols=(0, 1, 2),
                           coef=(1.0, 0.1, 0.05, 0.2 if adam else 0.0), uniforms=u)
        win = window.cpu().numpy()
        rec = dict(batch=batch.copy(), action=out["action"].cpu().numpy(), reward=out["reward"].cpu().numpy(),
                   gns=float(win[B.ST_GNS]), cos=float(win[B.ST_COS_PREV]), sigma_norm=float(win[B.ST_SIGMA_NORM]),
                   flags=int(win[B.ST_FLAGS]))
        records.append(rec)
        if verbose:
            print("cycle %d: B=%d gns=%.1f cos=%.3f sigma_norm=%.3f mean reward %.3f actions %s" % (
                c, int(batch.sum()), rec["gns"], rec["cos"], rec["sigma_norm"], float(rec["reward"].mean()),
                np.bincount(rec["action"], minlength=5).tolist()))
        batch = out["next_batch"].cpu().numpy().astype(np.int32)      # the one read-back of a cycle
    B.dmx_agg_destroy(agg)
    d.close()
    return records


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", type=int, default=1)
    ap.add_argument("--P", type=int, default=0)
    ap.add_argument("--cycles", type=int, default=5)
    ap.add_argument("--k", type=int, default=4)
    ap.add_argument("--hidden", type=int, default=32)
    ap.add_argument("--adam", action="store_true")
    ap.add_argument("--greedy", action="store_true")
    a = ap.parse_args()
    run(a.workload, a.P, a.cycles, a.k, a.hidden, a.adam, not a.greedy, verbose=True)


if __name__ == "__main__":
    main()
