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

def _run_sharded(wl, nshards, steps, adam=False):
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
