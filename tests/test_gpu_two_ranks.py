"""The worker-per-GPU form of the step (worker k is rank k; the model state is sharded by
parameter range) run end to end by more than one process:

  - two processes on cuda:0 with a gloo group (the exchange goes through host copies): batch
    sizes gathered, gradient ranges exchanged, the fused pass on each rank's shard, the partial
    sums added over the ranks, the state vector derived on both, the parameters rebuilt; every
    rank compares with the oracle of the whole problem. The two processes' kernels never wait on
    one another: all coordination is on the host, between launches.
  - one process with a one-rank nccl group (NVLS off), so that the nccl branches (all_to_all,
    all_gather, all_reduce on device tensors) run.

No timing is taken here: this run has one GPU, and a scaling figure needs several."""
import os
import socket
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import numpy as np, torch
    import paper_2510_08522_b200 as D
    from paper_2510_08522_b200 import binding as B, dist_util as DU
    from oracle.dmx_oracle import Oracle
    from tests import parity as PT
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    backend = os.environ["DMX_TEST_BACKEND"]
    torch.cuda.set_device(0)
    DU.init(world, backend, group_of_one=True)
    P, steps = 300_007, 3
    seg = [0, 1000, 1000, 150_000, 150_001, P]
    rng = np.random.default_rng(21)                                # every rank draws the whole problem
    mu = 0.1 * rng.standard_normal(P)
    batch = [32, 96, 64, 128][:world]
    ranges = DU.shard_ranges(P, world)
    lo, hi = ranges[rank]
    sh = D.ShardedDmx(world, P, seg, B.F32, world, rank)
    p0 = (0.05 * rng.standard_normal(P)).astype(np.float32)
    hp, hm, hv = p0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)
    tp = torch.from_numpy(p0[lo:hi].copy()).cuda()
    tm, tv = torch.zeros(hi - lo, device="cuda"), torch.zeros(hi - lo, device="cuda")
    full = torch.empty(P, device="cuda")
    orc = Oracle(world, P, seg, 0)
    for t in range(steps):
        grads = [(mu + rng.standard_normal(P) / np.sqrt(batch[k])).astype(np.float32) for k in range(world)]
        conds = PT.cond_vectors(grads, batch, hp, hm, 0.1, 0.9)
        ref = orc.step(grads, batch, hp, hm, 0.1, 0.9, hv)
        st = DU.worker_per_gpu_step(sh, rank, ranges, torch.from_numpy(grads[rank]).cuda(), batch[rank], tp, tm, tv, 0.1, 0.9,
                                    params_full=full)
        torch.cuda.synchronize()
        what = "rank %%d of %%d (%%s) step %%d" %% (rank, world, backend, t)
        PT.check_state(st.cpu().numpy(), ref, world, len(seg) - 1, seg, batch, what, seg_scale=PT.seg_scales(conds[0], seg))
        own = (tv.cpu().numpy(), tm.cpu().numpy(), tp.cpu().numpy())
        PT.check_vectors(0, own, (hv[lo:hi], hm[lo:hi], hp[lo:hi]), tuple(c[lo:hi] for c in conds), what)
        assert PT.vec_err(full.cpu().numpy(), hp, conds[2]) <= PT.TOL_V[0], what + " rebuilt parameters"
    sh.close()
    DU.finish()
    print("rank", rank, "ok")
""" % ROOT)


def _launch(world, backend, extra_env=None):
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE=str(world), LOCAL_RANK="0", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), DMX_TEST_BACKEND=backend, **(extra_env or {}))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT))
    for r, p in enumerate(procs):
        out, _ = p.communicate(timeout=600)
        assert p.returncode == 0, out.decode()[-4000:]
        assert ("rank %d ok" % r) in out.decode()


def test_two_processes_one_gpu_gloo():
    _launch(2, "gloo")


def test_four_processes_one_gpu_gloo():
    _launch(4, "gloo")


def test_one_rank_nccl_group_runs_the_device_collectives():
    _launch(1, "nccl", {"NCCL_NVLS_ENABLE": "0"})
