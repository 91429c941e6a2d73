"""Sharding one problem by parameter range: the host logic (ranges, clipped segment tables, the
sum of the shards' partial vectors over two gloo ranks) without a GPU, and on a GPU the shards
of one problem run one after the other against the oracle of the whole problem."""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np
import pytest

import paper_2510_08522_b200 as D
from paper_2510_08522_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("P,n", [(1, 1), (1, 4), (1023, 3), (1024, 2), (1025, 2), (10_000_019, 8), (340_000_000, 8), (5000, 7)])
def test_shard_ranges_tile_the_problem(P, n):
    edges = []
    for r in range(n):
        rc, lo, hi = D.dmx_shard_range(P, n, r)
        assert rc == 0 and 0 <= lo <= hi <= P
        assert lo % 1024 == 0 and (hi % 1024 == 0 or hi == P)
        edges.append((lo, hi))
    assert edges[0][0] == 0 and edges[-1][1] == P
    assert all(edges[i][1] == edges[i + 1][0] for i in range(n - 1))
    sizes = [hi - lo for lo, hi in edges]
    if P >= 1024 * n * 8:
        assert max(sizes) - min(sizes) <= 2048
    assert D.dmx_shard_range(P, n, n)[0] == B.ERR_ARG and D.dmx_shard_range(P, 0, 0)[0] == B.ERR_ARG


def test_shard_segment_tables_partition_every_segment():
    rng = np.random.default_rng(0)
    P, n = 1_000_003, 5
    seg = [0] + sorted(int(v) for v in rng.integers(0, P, 23)) + [P]          # some segments empty or tiny
    total = np.zeros(len(seg) - 1, dtype=np.int64)
    for r in range(n):
        _, lo, hi = D.dmx_shard_range(P, n, r)
        rc, loc = D.dmx_shard_segments(seg, lo, hi)
        assert rc == 0 and loc[0] == 0 and loc[-1] == hi - lo and all(a <= b for a, b in zip(loc, loc[1:]))
        # by hand: the part of segment s inside [lo, hi)
        want = [max(0, min(seg[s + 1], hi) - max(seg[s], lo)) for s in range(len(seg) - 1)]
        assert list(np.diff(loc)) == want
        total += np.diff(loc)
    assert np.array_equal(total, np.diff(seg))
    assert D.dmx_shard_segments(seg, 10, 5)[0] == B.ERR_ARG
    assert D.dmx_shard_segments(seg, 0, P + 1)[0] == B.ERR_SEGMENTS
    assert D.dmx_shard_segments([0, 5, 3, P], 0, P)[0] == B.ERR_SEGMENTS


WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import torch
    from paper_2510_08522_b200 import dist_util as DU
    import paper_2510_08522_b200 as D
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    DU.init(world, "gloo")
    K, S, P = 3, 4, 100_000
    n = K + 5 + 2 * S
    # each rank owns one parameter range; its partial vector here is a stand-in computed from the range
    rc, lo, hi = D.dmx_shard_range(P, world, rank)
    assert rc == 0
    part = torch.arange(n, dtype=torch.float64) * float(hi - lo)
    DU.allreduce_sum(part)
    assert torch.equal(part, torch.arange(n, dtype=torch.float64) * float(P)), part
    # worker k is rank k: every rank ends up with all workers' values of its own parameter range
    Pg = 5000
    ranges = DU.shard_ranges(Pg, world)
    assert ranges[0][0] == 0 and ranges[-1][1] == Pg
    grad = torch.arange(Pg, dtype=torch.float32) + 10000.0 * rank
    rows = DU.exchange_gradient_ranges(grad, ranges, rank)
    lo, hi = ranges[rank]
    assert rows.shape[0] == world and rows.shape[1] %% 8 == 0 and rows.shape[1] >= hi - lo
    for k in range(world):
        assert torch.equal(rows[k, :hi - lo], torch.arange(lo, hi, dtype=torch.float32) + 10000.0 * k)
        assert rows[k].data_ptr() %% 16 == 0
    assert DU.gather_batch_sizes(32 * (rank + 1)) == [32 * (r + 1) for r in range(world)]
    # the updated parameter shards put back together
    full = torch.full((Pg,), -1.0)
    DU.allgather_ranges(torch.arange(lo, hi, dtype=torch.float32) * 2.0, ranges, full)
    assert torch.equal(full, torch.arange(Pg, dtype=torch.float32) * 2.0)
    DU.finish()
    print("rank", rank, "ok")
""" % ROOT)


def test_partials_add_up_over_two_gloo_ranks():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT))
    for r, p in enumerate(procs):
        out, _ = p.communicate(timeout=240)
        assert p.returncode == 0, out.decode()
        assert ("rank %d ok" % r) in out.decode()


# ------------------------------------------------------------------------------------------
# GPU: the shards of one problem, one after the other on one device, against the whole problem's oracle

def _run_sharded(wl, nshards, steps, adam=False, local=False):
    import torch
    from oracle.dmx_oracle import Oracle
    from paper_2510_08522_b200 import workload as W
    from tests import parity as PT
    dp = W.DeviceProblem(wl)
    orc = Oracle(wl.K, wl.P, dp.seg, wl.dtype)
    shards = [D.ShardedDmx(wl.K, wl.P, dp.seg, wl.dtype, nshards, r) for r in range(nshards)]
    hp, hm, hv = dp.params.cpu().numpy().copy(), dp.momentum.cpu().numpy().copy(), dp.prev_agg.cpu().numpy().copy()
    second = torch.zeros(wl.P, dtype=torch.float32, device="cuda") if adam else None
    h2 = np.zeros(wl.P, np.float32)
    for t in range(steps):
        b = dp.fill()
        raw, wide = PT.grads_to_host(torch, dp.grads, wl.dtype)
        if adam:
            ref = orc.step_adam(raw, b, hp, hm, h2, 1e-3, 0.9, 0.999, 1e-8, t + 1, hv)
        else:
            conds = PT.cond_vectors(wide, b, hp, hm, wl.lr, wl.beta)
            ref = orc.step(raw, b, hp, hm, wl.lr, wl.beta, hv)
        total = None
        for sh in shards:
            if local:
                # what a rank holds when worker k is GPU k: every worker's values of its own range (rows
                # padded to 8 elements) and its own shard of the model state
                n = sh.hi - sh.lo
                rows = torch.zeros((wl.K, max(8, (n + 7) // 8 * 8)), dtype=dp.grads[0].dtype, device="cuda")
                for k in range(wl.K):
                    rows[k, :n] = dp.grads[k][sh.lo:sh.hi]
                ps, ms, vs = (x[sh.lo:sh.hi].clone() for x in (dp.params, dp.momentum, dp.prev_agg))
                part = sh.step_partial([rows[k] for k in range(wl.K)], b, ps, ms, wl.lr, wl.beta, vs, local=True)
                dp.params[sh.lo:sh.hi] = ps; dp.momentum[sh.lo:sh.hi] = ms; dp.prev_agg[sh.lo:sh.hi] = vs
            else:
                part = sh.step_partial(dp.grads, b, dp.params, dp.momentum, 1e-3 if adam else wl.lr, 0.9 if adam else wl.beta,
                                       dp.prev_agg, adam=(second, 0.999, 1e-8, t + 1) if adam else None)
            total = part if total is None else total + part
        st = shards[0].finalize(b, total, adam=adam)
        torch.cuda.synchronize()
        what = "%s in %d shards, step %d" % (wl.name, nshards, t)
        assert total[-1].item() == 0.0
        if adam:
            got = st.cpu().numpy()
            assert np.allclose(dp.prev_agg.cpu().numpy(), hv, rtol=4e-3 if wl.dtype else 1e-5, atol=1e-7), what
            assert np.allclose(dp.params.cpu().numpy(), hp, rtol=1e-4, atol=2e-5), what
            assert np.allclose(got[:11], ref[:11], rtol=2e-4, atol=1e-6), what
            assert np.allclose(got[12:15], ref[12:15], rtol=2e-3, atol=1e-4), what
            assert np.allclose(got[16:], ref[16:], rtol=2e-4, atol=1e-7), what
        else:
            PT.check_vectors(wl.dtype, (dp.prev_agg.cpu().numpy(), dp.momentum.cpu().numpy(), dp.params.cpu().numpy()),
                             (hv, hm, hp), conds, what)
            PT.check_state(st.cpu().numpy(), ref, wl.K, wl.S, dp.seg, b, what, seg_scale=PT.seg_scales(conds[0], dp.seg))
        dp.advance()
    for sh in shards:
        sh.close()
    return st


@pytest.mark.gpu
@pytest.mark.parametrize("idx,P,nshards", [(0, 262_147, 2), (1, 333_337, 3), (2, 401_239, 4), (3, 290_011, 8), (4, 523_777, 5),
                                           (1, 1500, 4)])
def test_gpu_shards_match_the_whole_problem_oracle(idx, P, nshards):
    from paper_2510_08522_b200 import workload as W
    _run_sharded(W.WORKLOADS[idx].scaled(P=P, steps=3), nshards, 3)


@pytest.mark.gpu
@pytest.mark.parametrize("idx,P,nshards", [(1, 333_337, 3), (4, 523_777, 4)])
def test_gpu_shards_with_rank_local_buffers(idx, P, nshards):
    from paper_2510_08522_b200 import workload as W
    _run_sharded(W.WORKLOADS[idx].scaled(P=P, steps=2), nshards, 2, local=True)


@pytest.mark.gpu
def test_gpu_worker_per_gpu_step_on_one_rank():
    """The packaged multi-GPU step with a world of one: K = 1 worker, one shard."""
    import torch
    from oracle.dmx_oracle import Oracle
    from paper_2510_08522_b200 import dist_util as DU
    P = 70_001
    rng = np.random.default_rng(9)
    g = rng.normal(size=P).astype(np.float32)
    p0 = rng.normal(scale=0.05, size=P).astype(np.float32)
    seg = [0, 1000, P]
    DU.init(1)
    ranges = DU.shard_ranges(P, 1)
    sh = D.ShardedDmx(1, P, seg, B.F32, 1, 0)
    tp, tm, tv = torch.from_numpy(p0.copy()).cuda(), torch.zeros(P, device="cuda"), torch.zeros(P, device="cuda")
    full = torch.empty(P, device="cuda")
    st = DU.worker_per_gpu_step(sh, 0, ranges, torch.from_numpy(g).cuda(), 64, tp, tm, tv, 0.1, 0.9, params_full=full)
    torch.cuda.synchronize()
    hp, hm, hv = p0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32)
    ref = Oracle(1, P, seg, 0).step([g], [64], hp, hm, 0.1, 0.9, hv)
    assert np.allclose(st.cpu().numpy(), ref, rtol=1e-4, atol=1e-7)
    assert np.allclose(full.cpu().numpy(), hp, rtol=1e-6, atol=1e-8) and np.allclose(tm.cpu().numpy(), hm, rtol=1e-6, atol=1e-8)
    sh.close()


@pytest.mark.gpu
def test_gpu_shards_adam():
    from paper_2510_08522_b200 import workload as W
    _run_sharded(W.WORKLOADS[2].scaled(P=401_239, steps=3), 3, 3, adam=True)


@pytest.mark.gpu
def test_gpu_one_shard_equals_the_plain_step_bitwise():
    import torch
    from paper_2510_08522_b200 import workload as W
    wl = W.WORKLOADS[1].scaled(P=777_777, steps=1)
    dp = W.DeviceProblem(wl)
    b = dp.fill()
    p0, m0, a0 = dp.params.clone(), dp.momentum.clone(), dp.prev_agg.clone()
    d = D.Dmx(wl.K, wl.P, dp.seg, wl.dtype)
    st = d.step(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg).clone()
    p1, m1, a1 = dp.params.clone(), dp.momentum.clone(), dp.prev_agg.clone()
    dp.params.copy_(p0); dp.momentum.copy_(m0); dp.prev_agg.copy_(a0)
    sh = D.ShardedDmx(wl.K, wl.P, dp.seg, wl.dtype, 1, 0)
    st2 = sh.finalize(b, sh.step_partial(dp.grads, b, dp.params, dp.momentum, wl.lr, wl.beta, dp.prev_agg))
    torch.cuda.synchronize()
    assert torch.equal(p1, dp.params) and torch.equal(m1, dp.momentum) and torch.equal(a1, dp.prev_agg)
    assert torch.equal(st, st2)
    d.close(); sh.close()


@pytest.mark.gpu
def test_gpu_partial_argument_errors():
    import torch
    z = torch.zeros(4096, dtype=torch.float32, device="cuda")
    zd = torch.zeros(64, dtype=torch.float64, device="cuda")
    rc, h = D.dmx_create(2, 1024, [0, 1024])
    assert rc == 0 and D.dmx_partials_len(h) == 2 + 5 + 2
    g = [z[:1024].data_ptr(), z[1024:2048].data_ptr()]
    assert D.dmx_step_partial(h, g, [1, 1], z[2048:].data_ptr(), z[3072:].data_ptr(), 0.1, 0.9, z[1024:].data_ptr(), 0) == B.ERR_ARG
    assert D.dmx_step_partial(h, g, [1, 1], z[2048:].data_ptr(), z[3072:].data_ptr(), 0.1, 0.9, z[1024:].data_ptr(),
                              zd.data_ptr()) == B.ERR_ARG                       # prev_agg aliases a gradient
    assert D.dmx_step_partial(h, g, [1, 1], z[2048:].data_ptr(), z[3072:].data_ptr(), 0.1, 0.9, z[1024:].data_ptr(),
                              zd.data_ptr() + 4) == B.ERR_ALIGN
    assert D.dmx_finalize_partials(2, 1, [1, 0], zd.data_ptr(), 0, 1024, z.data_ptr()) == B.ERR_BATCH
    assert D.dmx_finalize_partials(0, 1, [1, 1], zd.data_ptr(), 0, 1024, z.data_ptr()) == B.ERR_ARG
    assert D.dmx_finalize_partials(2, 1, [1, 1], 0, 0, 1024, z.data_ptr()) == B.ERR_ARG
    assert D.dmx_finalize_partials(2, 1, [1, 1], zd.data_ptr(), 0, 1024, z.data_ptr()) == B.OK
    torch.cuda.synchronize()
    D.dmx_destroy(h)
