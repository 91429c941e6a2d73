"""The fused pass's work list (host logic, no GPU): every tile in exactly one chunk, the wave
structure, the place of the ragged tile, and how even the shares are."""
import numpy as np
import pytest

import paper_2510_08522_b200 as D
from paper_2510_08522_b200 import binding as B

CASES = [
    # P, K, dtype, tile, resident CTAs
    (1_048_576, 4, B.F32, 896, 148),
    (11_689_512, 8, B.F32, 896, 148),
    (25_557_032, 16, B.BF16, 1792, 148),
    (138_357_544, 32, B.F32, 896, 148),
    (340_000_000, 32, B.BF16, 1792, 148),
    (1, 1, B.F32, 896, 148), (895, 3, B.F32, 896, 148), (896, 3, B.F32, 896, 148), (897, 3, B.BF16, 1792, 148),
    (896 * 148, 2, B.F32, 896, 148), (896 * 149 + 5, 2, B.F32, 896, 148), (1792 * 1000 + 1, 64, B.BF16, 1792, 148),
    (10_000_019, 5, B.F32, 896, 7), (10_000_019, 5, B.F32, 896, 1), (3_000_000, 16, B.BF16, 1792, 296),
]


def tiles_of(first, n, stride, R):
    i = np.arange(n)
    return first + (i // R) * stride + i % R


@pytest.mark.parametrize("P,K,dtype,tile,ctas", CASES)
def test_every_tile_in_exactly_one_chunk(P, K, dtype, tile, ctas):
    n, t0, nt, st, R, grid = D.dmx_plan_chunks(P, K, dtype, tile, ctas)
    assert n > 0 and len(t0) == n and R >= 1 and 1 <= grid <= ctas
    ntiles = -(-P // tile)
    seen = np.zeros(ntiles, dtype=np.int32)
    for c in range(n):
        assert nt[c] >= 1 and st[c] >= R
        t = tiles_of(t0[c], nt[c], st[c], R)
        assert t.min() >= 0 and t.max() < ntiles
        np.add.at(seen, t, 1)
    assert np.all(seen == 1)
    # the chunk with a ragged last tile comes first, and that tile is the chunk's last
    if P % tile:
        t = tiles_of(t0[0], nt[0], st[0], R)
        assert t[-1] == ntiles - 1
    # no chunk is longer than 32 tiles (fp32 partial sums stay short)
    assert max(nt) <= 32


@pytest.mark.parametrize("P,K,dtype,tile,ctas", CASES[:5])
def test_shares_shrink_towards_the_end_and_are_even(P, K, dtype, tile, ctas):
    n, t0, nt, st, R, grid = D.dmx_plan_chunks(P, K, dtype, tile, ctas)
    nt = np.array(nt)
    ntiles = -(-P // tile)
    body = nt[1:] if P % tile else nt          # apart from the chunk moved to the front
    if ntiles >= 64 * grid:
        # chunk sizes never grow along the list, and the last `grid` chunks together hold only a
        # small part of the work: the tail that decides how evenly the CTAs finish
        assert np.all(np.diff(body) <= 0)
        assert body[-min(grid, len(body)):].sum() <= 0.12 * ntiles
    else:
        # a problem of a few tiles per CTA is one even wave
        assert body.max() - body.min() <= R and n <= grid
    # static deal (chunk c to CTA c mod grid, what the plain-load kernel does): shares within 15 %
    share = np.zeros(grid, dtype=np.int64)
    for c in range(n):
        share[c % grid] += nt[c]
    if ntiles >= 8 * grid:
        assert share.max() <= 1.15 * share.mean() + 2 * R


@pytest.mark.parametrize("group,chunk,min_kb", [(1, 4, 48), (2, 8, 0), (4, 64, 384), (8, 16, 0), (16, 128, 0), (3, 5, 1)])
@pytest.mark.parametrize("P,K,dtype,tile,ctas", CASES[1:5] + CASES[7:12])
def test_tuning_knobs_keep_the_list_valid(monkeypatch, group, chunk, min_kb, P, K, dtype, tile, ctas):
    # what the kernel relies on, whatever the knobs: every chunk has at least one tile, every tile
    # is in exactly one chunk, and a ragged last tile is the last tile of the first chunk
    monkeypatch.setenv("DMX_TILE_GROUP", str(group))
    monkeypatch.setenv("DMX_CHUNK_TILES", str(chunk))
    if min_kb:
        monkeypatch.setenv("DMX_MIN_CHUNK_KB", str(min_kb))
    n, t0, nt, st, R, grid = D.dmx_plan_chunks(P, K, dtype, tile, ctas)
    ntiles = -(-P // tile)
    assert n > 0 and R == group and min(nt) >= 1
    seen = np.zeros(ntiles, dtype=np.int32)
    for c in range(n):
        t = tiles_of(t0[c], nt[c], st[c], R)
        np.add.at(seen, t, 1)
        if P % tile and ntiles - 1 in t:
            assert c == 0 and t[-1] == ntiles - 1
    assert np.all(seen == 1)


def test_plan_rejects_bad_arguments():
    assert D.dmx_plan_chunks(0, 4, B.F32, 896, 148)[0] == B.ERR_ARG
    assert D.dmx_plan_chunks(10, 0, B.F32, 896, 148)[0] == B.ERR_ARG
    assert D.dmx_plan_chunks(10, 4, 7, 896, 148)[0] == B.ERR_ARG
    assert D.dmx_plan_chunks(10, 4, B.F32, 0, 148)[0] == B.ERR_ARG
    assert D.dmx_plan_chunks(10, 4, B.F32, 896, 0)[0] == B.ERR_ARG


def test_random_problems_are_always_tiled_exactly():
    hyp = pytest.importorskip("hypothesis")
    st = hyp.strategies

    @hyp.settings(max_examples=150, deadline=None)
    @hyp.given(P=st.integers(1, 60_000_000), K=st.integers(1, 64), dtype=st.sampled_from([B.F32, B.BF16]),
               ctas=st.integers(1, 320))
    def check(P, K, dtype, ctas):
        tile = 896 if dtype == B.F32 else 1792
        n, t0, nt, stv, R, grid = D.dmx_plan_chunks(P, K, dtype, tile, ctas)
        ntiles = -(-P // tile)
        assert n > 0 and 1 <= grid <= ctas and sum(nt) == ntiles and max(nt) <= 32 and min(nt) >= 1
        seen = np.zeros(ntiles, dtype=np.int32)
        for c in range(n):
            np.add.at(seen, tiles_of(t0[c], nt[c], stv[c], R), 1)
        assert np.all(seen == 1)
        if P % tile:
            assert tiles_of(t0[0], nt[0], stv[0], R)[-1] == ntiles - 1

    check()
