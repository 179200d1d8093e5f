"""Host-only checks of the device-side schedules: gemm_plan_schedule walks a plan with the functions the kernels run
(tile decoding with the plan-time divisors, the grouped raster, dealt schedules of structured problems, tail split,
stream-K ranges).  What must hold for any plan: every wanted output tile is computed exactly once, the K stages of a
split tile are covered exactly once, and K stages left out under a triangular operand can only hold zeros."""
import itertools

import numpy as np
import pytest

import paper_2512_16465_b200 as bg

V1, V2, VS, VW = bg.VARIANT_DENSE_1CTA, bg.VARIANT_DENSE_2CTA, bg.VARIANT_SKINNY_STREAMK, bg.VARIANT_DENSE_2CTA_WIDE
CTA, BATCH, ROW, COL, K0, K1, SLICE = range(7)


def plan_and_schedule(M, N, K, flags=0, **kw):
    up = lambda x: -(-x // 8) * 8            # leading dimensions must span multiples of 16 bytes
    batch = kw.get("batch", 1)
    kw.update(lda=up(K), ldb=up(K), ldc=up(N), stride_a=M * up(K), stride_b=N * up(K), stride_c=M * up(N))
    if batch == 1:
        kw.update(stride_a=0, stride_b=0, stride_c=0)
    h = bg.gemm_plan(bg.make_desc(M, N, K, flags=flags, **kw))
    try:
        return bg.gemm_plan_info(h), bg.gemm_plan_schedule(h)
    finally:
        bg.gemm_destroy(h)


def wanted_tiles(info, M, N, batch, d_tri):
    """(batch, tile row, tile column) of every tile that holds at least one wanted element of D."""
    tm, tn = info["tile_m"], info["tile_n"]
    out = set()
    for i in range(-(-M // tm)):
        for j in range(-(-N // tn)):
            r0, r1 = i * tm, min((i + 1) * tm, M) - 1
            c0, c1 = j * tn, min((j + 1) * tn, N) - 1
            if d_tri == 1 and r1 < c0:      # lower triangle wanted (row >= column): the tile lies wholly above the diagonal
                continue
            if d_tri == 2 and r0 > c1:
                continue
            out.update((b, i, j) for b in range(batch))
    return out


def check_dense(info, sched, M, N, K, batch=1, d_tri=0, a_tri=0, b_tri=0):
    clusters = info["grid"] // info["cluster_size"]
    assert sched[:, CTA].min() >= 0 and sched[:, CTA].max() < clusters
    stages = -(-K // info["tile_k"])
    by_tile = {}
    for it in sched:
        by_tile.setdefault((it[BATCH], it[ROW], it[COL]), []).append(it)
    assert set(by_tile) == wanted_tiles(info, M, N, batch, d_tri)          # every wanted tile, and no other
    tm, tn, tk = info["tile_m"], info["tile_n"], info["tile_k"]
    for (b, i, j), items in by_tile.items():
        if len(items) == 1:
            it = items[0]
            assert it[SLICE] == -1
            lo, hi = it[K0], it[K1]
        else:                                                              # K slices: 0 .. n-1, contiguous, disjoint
            items.sort(key=lambda it: it[SLICE])
            assert [it[SLICE] for it in items] == list(range(len(items))) == list(range(info["split"]))
            assert all(x[K1] == y[K0] for x, y in zip(items, items[1:]))
            assert len({it[CTA] for it in items}) == len(items)            # side by side, one CTA (pair) each
            lo, hi = items[0][K0], items[-1][K1]
        assert 0 <= lo < hi <= stages
        # a stage that was left out must lie wholly in the zero part of a triangular operand
        r0, r1 = i * tm, min((i + 1) * tm, M) - 1
        c0, c1 = j * tn, min((j + 1) * tn, N) - 1
        for s in itertools.chain(range(0, lo), range(hi, stages)):
            k0, k1 = s * tk, min((s + 1) * tk, K) - 1
            zero_a = (a_tri == 1 and k0 > r1) or (a_tri == 2 and k1 < r0)   # lower: zero for k > i; upper: zero for k < i
            zero_b = (b_tri == 1 and k1 < c0) or (b_tri == 2 and k0 > c1)   # lower: zero for k < j; upper: zero for k > j
            assert zero_a or zero_b, ((b, i, j), s, (lo, hi))
        if not (a_tri or b_tri):
            assert (lo, hi) == (0, stages)
    # execution order inside a CTA: the static round-robin visits its items in increasing order of the linear work id,
    # which the list reports per CTA; the per-CTA loads differ by at most one item on an unstructured problem
    if not (d_tri or a_tri or b_tri):
        per = np.bincount(sched[:, CTA], minlength=clusters)
        assert per.max() - per.min() <= 1


DENSE_SHAPES = [(512, 512, 512), (1, 1, 1), (129, 257, 65), (1000, 1000, 1000), (2560, 2560, 2560), (4100, 4104, 4104),
                (8192, 8192, 8192), (300, 70000, 64), (16384, 14336, 4096), (130, 258, 66000), (12345, 4328, 2056)]


@pytest.mark.parametrize("shape", DENSE_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("variant,tile_n", [(0, 0), (V1, 64), (V1, 128), (V1, 192), (V1, 256), (V2, 128), (V2, 256), (VW, 0),
                                            (V1, 320), (V2, 384), (V2, 512)])
def test_every_tile_once_dense(shape, variant, tile_n):
    M, N, K = shape
    if variant == VW and M <= 128:
        pytest.skip("a pair needs two tile rows")
    for raster in (0, 1, 3, 7, 100):
        for batch in (1, 3):
            if batch > 1 and M * N > 3e7:
                continue
            try:
                info, sched = plan_and_schedule(M, N, K, bg.make_flags(variant, tile_n, raster=raster), batch=batch, c_dtype=bg.BF16)
            except bg.GemmError as e:
                assert e.status == bg.ERR_UNSUPPORTED
                continue
            check_dense(info, sched, M, N, K, batch)


@pytest.mark.parametrize("shape", [(1024, 1024, 2048), (2560, 2560, 2560), (512, 512, 16384), (1536, 1536, 4096), (130, 258, 66000),
                                   (1000, 1000, 1096), (1280, 4096, 512)], ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("variant,tile_n", [(V1, 128), (V1, 256), (V2, 128), (V2, 256)])
def test_tail_split_covers_k_once(shape, variant, tile_n):
    M, N, K = shape
    info, sched = plan_and_schedule(M, N, K, bg.make_flags(variant, tile_n, tail_split=True), c_dtype=bg.BF16)
    check_dense(info, sched, M, N, K)
    if info["split"] > 1:
        assert (sched[:, SLICE] >= 0).any() and info["workspace_bytes"] > 0
        # the slices of a tile run in the same round of their CTAs: nobody waits for a CTA that is still busy elsewhere
        pos = {}
        for c in np.unique(sched[:, CTA]):
            for k, row in enumerate(np.flatnonzero(sched[:, CTA] == c)):
                pos[row] = k
        for key in {tuple(it[[BATCH, ROW, COL]]) for it in sched if it[SLICE] >= 0}:
            rows = [r for r in range(len(sched)) if tuple(sched[r, [BATCH, ROW, COL]]) == key]
            assert len({pos[r] for r in rows}) == 1


@pytest.mark.parametrize("a_tri,b_tri,d_tri", [(1, 0, 0), (2, 0, 0), (0, 1, 0), (0, 2, 0), (0, 0, 1), (0, 0, 2), (1, 1, 1), (2, 2, 2),
                                               (1, 0, 2), (2, 1, 0)])
@pytest.mark.parametrize("shape", [(512, 264, 512), (1000, 136, 200), (300, 264, 1000), (2048, 2048, 2048), (4100, 4104, 4104),
                                   (600, 2000, 520)], ids=lambda s: "x".join(map(str, s)))
def test_structured_problems(shape, a_tri, b_tri, d_tri):
    M, N, K = shape
    for variant, tile_n, batch in ((0, 0, 1), (V1, 128, 2), (V2, 128, 1), (V2, 256, 3), (V1, 64, 1)):
        fl = bg.make_flags(variant, tile_n, a_lower=a_tri == 1, a_upper=a_tri == 2, d_lower=d_tri == 1, d_upper=d_tri == 2)
        info, sched = plan_and_schedule(M, N, K, fl, structure=b_tri, batch=batch)
        check_dense(info, sched, M, N, K, batch, d_tri, a_tri, b_tri)
        # dealt ahead of time by work: no CTA carries more than the mean plus one tile's worth of K stages
        # (the matrices of a batch are dealt together, so this holds for the batch as a whole)
        work = np.zeros(info["grid"] // info["cluster_size"])
        np.add.at(work, sched[:, CTA], sched[:, K1] - sched[:, K0] + 1)
        assert work.max() <= work.mean() + (sched[:, K1] - sched[:, K0]).max() + 1


@pytest.mark.parametrize("short", [1, 8, 16, 33, 48, 64])
@pytest.mark.parametrize("long_,K", [(128, 64), (256, 4096), (1864, 2136), (4096, 4096), (28672, 8192), (28672, 1024), (50264, 4096),
                                     (4096, 14336), (12288, 4096), (1000, 520), (520, 66000)])
def test_stream_k_units_once(short, long_, K):
    for tall in (False, True):
        M, N = (long_, short) if tall else (short, long_)
        for kslices in (0, 1, 2, 3):
            try:
                info, sched = plan_and_schedule(M, N, K, bg.make_flags(VS, kslices=kslices))
            except bg.GemmError as e:
                assert e.status == bg.ERR_UNSUPPORTED
                continue
            tiles = -(-long_ // 128)
            stages = -(-K // info["tile_k"])
            assert info["num_tiles"] == tiles * stages and info["grid"] <= 148
            tile_ix = sched[:, ROW] if tall else sched[:, COL]
            assert (sched[:, COL if tall else ROW] == 0).all()
            # CTAs in order walk the units in order: concatenating the items gives every (tile, stage) exactly once
            units = np.concatenate([t * stages + np.arange(a, b) for t, a, b in zip(tile_ix, sched[:, K0], sched[:, K1])])
            assert np.array_equal(units, np.arange(tiles * stages))
            assert (np.diff(sched[:, CTA]) >= 0).all() and len(np.unique(sched[:, CTA])) == info["grid"]
            per = np.zeros(info["grid"], int)
            np.add.at(per, sched[:, CTA], sched[:, K1] - sched[:, K0])
            if per.max() - per.min() > 1:
                # grouped ranges (three tiles per four CTAs): two contributors on every tile, the last CTA of a group shorter
                assert info["grid"] == 4 * (tiles // 3) + (tiles % 3 + 1 if tiles % 3 else 0) and info["split"] == 2
                assert all((tile_ix == t).sum() == 2 for t in range(tiles)) and per.max() <= 1.2 * per.mean()
            # contributors of a split tile are numbered 0, 1, 2 ... in CTA order; a whole tile has one item marked -1
            for t in range(tiles):
                sl = sched[tile_ix == t, SLICE]
                assert (len(sl) == 1 and sl[0] == -1) or list(sl) == list(range(len(sl)))
                assert len(sl) <= info["split"]


def test_cluster_mode_of_stream_k():
    """Exactly c <= 8 CTAs per output tile: the plan launches them as clusters and asks for no workspace; otherwise the
    partial tiles go through a workspace."""
    def info(M, N, K, **kw):
        return plan_and_schedule(M, N, K, bg.make_flags(VS), **kw)[0]
    import torch
    for (M, N, K), c in (((8, 4096, 4096), 4), ((64, 4096, 4096), 4), ((16, 2048, 8192), 8), ((33, 4000, 4608), 4),
                         ((4096, 8, 4096), 4), ((4000, 48, 4608), 4), ((64, 6144, 6144), 3), ((48, 4096, 11008), 4)):
        i = info(M, N, K)
        if torch.cuda.is_available():    # how many clusters of a size fit at once is the device's to say
            assert 2 <= i["cluster_size"] <= c
        else:
            assert i["cluster_size"] == c
        assert i["workspace_bytes"] == 0 and i["grid"] == -(-max(M, N) // 128) * i["cluster_size"], (M, N, K, i)
    i = info(8, 4096, 8192, ab_dtype=bg.FP8_E4M3)
    assert i["cluster_size"] >= 2 and i["workspace_bytes"] == 0
    for M, N, K in ((8, 28672, 8192), (8, 10000, 2136), (40, 10240, 8200), (8, 11000, 8200), (33, 10880, 6144)):
        i = info(M, N, K)
        assert i["cluster_size"] == 1 and i["workspace_bytes"] > 0, (M, N, K, i)


@pytest.mark.parametrize("short", [8, 16, 40, 64])
@pytest.mark.parametrize("long_,K", [(10240, 8192), (11008, 4096), (12288, 4096), (9600, 16384), (12800, 4096), (11000, 8200)])
def test_grouped_ranges_of_stream_k(short, long_, K):
    """74 ... 100 tiles: every three tiles are shared by four CTAs (the tiles left over by one more CTA than tiles), each
    tile by two, and the CTA that holds a tile's tail is through with it before the CTA that holds its head has
    finished its own range -- by a margin, so that the head holder can fetch the partial tile ahead of its own end."""
    for tall in (False, True):
        M, N = (long_, short) if tall else (short, long_)
        info, sched = plan_and_schedule(M, N, K, bg.make_flags(VS), options=bg.OPT_STREAMK_WORKSPACE)
        tiles = -(-long_ // 128)
        stages = -(-K // info["tile_k"])
        assert 74 <= tiles <= 100
        assert info["grid"] == 4 * (tiles // 3) + (tiles % 3 + 1 if tiles % 3 else 0), info
        assert info["split"] == 2 and info["cluster_size"] == 1 and info["workspace_bytes"] > 0
        tile_ix = sched[:, ROW] if tall else sched[:, COL]
        per = np.zeros(info["grid"], int)
        np.add.at(per, sched[:, CTA], sched[:, K1] - sched[:, K0])
        first = np.concatenate([[0], np.cumsum(per)])        # first unit of every CTA
        margins = []
        for t in range(tiles):
            rows = sched[tile_ix == t]
            assert len(rows) == 2 and list(rows[:, SLICE]) == [0, 1]
            head, tail = rows[0], rows[1]
            assert head[K0] == 0 and head[K1] == tail[K0] and tail[K1] == stages and head[CTA] + 1 == tail[CTA]
            # the head is the end of its CTA's range, the tail the start of the next CTA's
            assert t * stages + head[K1] == first[head[CTA] + 1]
            margins.append(per[head[CTA]] - (tail[K1] - tail[K0]))
        assert min(margins) >= 2 and per.max() <= 1.2 * per.mean(), (min(margins), per.max(), per.mean())
