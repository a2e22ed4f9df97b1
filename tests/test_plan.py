"""Host logic of the kernel choice and the work decomposition (``dgemm_plan``): no GPU needed.

The decomposition rule is restated here from its description (whole waves of tiles data-parallel,
CTA b taking tiles b, b + G, ...; the k-blocks of the remaining tiles cut into equal spans, one per
CTA, at most two tile segments per span; a forced uniform K split otherwise) and checked for what
must hold for any shape: every (tile, k-block) is computed exactly once, partial-tile slots are
unique, and the grid fits on the device."""
import random

import pytest

import paper_2003_00532_b200 as dg

V_TMA, V_GENERIC, V_WS = dg.DGEMM_VARIANT_TMA, dg.DGEMM_VARIANT_GENERIC, dg.DGEMM_VARIANT_TMA_WS
V_CLUSTER = dg.DGEMM_VARIANT_TMA_CLUSTER
V_GCLUSTER = dg.DGEMM_VARIANT_GENERIC_CLUSTER
V_WSB = dg.DGEMM_VARIANT_TMA_WS_BULK


@pytest.fixture(autouse=True)
def _defaults():
    from paper_2003_00532_b200 import build as _build
    _build.build()
    dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
    dg.dgemm_set_split_k(0)
    dg.dgemm_set_test_flags(0)
    yield
    dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
    dg.dgemm_set_split_k(0)
    dg.dgemm_set_test_flags(0)


@pytest.mark.parametrize("shape,variant,bm,bn,wtm", [
    ((8192, 8192, 8192), V_WS, 128, 128, 64),      # large, aligned: warp-specialised, one CTA per SM
    ((4096, 4096, 4096), V_WS, 128, 128, 64),
    ((16384, 16384, 64), V_WSB, 128, 128, 64),     # many tiles of few k-blocks: the epilogue leaves through the copy engine
    ((16384, 16384, 256), V_WSB, 128, 128, 64),
    ((16384, 16384, 2048), V_WSB, 128, 128, 64),
    ((16384, 16384, 4096), V_WS, 128, 128, 64),    # ... up to 128 k-blocks per tile
    ((2560, 2560, 64), V_WSB, 128, 128, 64),       # ... and from two waves of tiles
    ((2048, 2048, 64), V_WS, 64, 128, 64),         # few tiles, K < 256: the warp-specialised kernel with two CTAs per SM
    ((2088, 2048, 2048), V_WS, 64, 128, 64),       # M just above a multiple of 64 rows: 64-row tiles, two CTAs per SM
    ((1600, 8192, 8192), V_TMA, 64, 128, 64),      # the same on a long problem: inline kernel
    ((256, 256, 256), V_WS, 64, 128, 64),          # one k-block per CTA through the workspace: the general kernels' floor
    ((128, 128, 128), V_WS, 64, 128, 64),
    ((64, 64, 64), V_CLUSTER, 64, 128, 64),        # too few k-blocks for a workspace split: split inside a cluster
    ((320, 320, 320), V_CLUSTER, 64, 128, 64),
    ((512, 512, 256), V_CLUSTER, 64, 128, 64),
    ((384, 384, 384), V_WS, 64, 128, 64),          # 18 tiles x 8 would have to share SMs
    ((128, 128, 4096), V_WS, 64, 128, 64),         # long K runs stay with the general kernels
    ((4097, 31, 4099), V_TMA, 256, 32, 64),        # narrow N
    ((8192, 96, 8192), V_TMA, 256, 32, 64),
    ((64, 64, 262144), V_TMA, 128, 64, 64),        # ... but not with a short M, where other tiles cover less padded area
    ((128, 48, 65536), V_TMA, 128, 64, 64),
    ((64, 96, 100000), V_WS, 64, 128, 64),
    ((200, 64, 30000), V_TMA, 256, 32, 64),
    ((8192, 128, 8192), V_WS, 128, 128, 64),
    ((6514, 146, 4096), V_TMA, 128, 64, 64),       # N just above a multiple of 128
    ((32, 8192, 8192), V_TMA, 32, 128, 32),        # short M
    ((96, 8192, 8192), V_TMA, 32, 128, 32),
    ((128, 8192, 8192), V_WS, 128, 128, 64),
])
def test_kernel_choice(shape, variant, bm, bn, wtm):
    pl = dg.dgemm_plan(*shape)
    assert (pl["variant"], pl["bm"], pl["bn"], pl["wtm"]) == (variant, bm, bn, wtm), pl
    assert pl["ctas_per_sm"] == (1 if (bm, bn) == (128, 128) else 2)


def test_unaddressable_operands_take_the_generic_staging_and_forced_tma_is_refused():
    pl = dg.dgemm_plan(1000, 1000, 1000, tma_addressable=False)
    assert pl["variant"] == V_GENERIC and pl["bm"] == 64
    assert dg.dgemm_plan(8192, 8192, 8192, tma_addressable=False)["bm"] == 128   # many waves: tall generic tiles
    dg.dgemm_set_variant(V_TMA)
    with pytest.raises(dg.DgemmError) as e:
        dg.dgemm_plan(1000, 1000, 1000, tma_addressable=False)
    assert e.value.status == dg.binding.DGEMM_ERR_VARIANT
    with pytest.raises(dg.DgemmError):
        dg.dgemm_plan(0, 5, 5)


def _items(pl, cta):
    """Work items (tile, kb0, kb1, slot) of one CTA, restated from the decomposition rule."""
    G, kb = pl["grid"], pl["kblocks"]
    out = []
    units = pl["dp_tiles"] * pl["split_k"]
    for unit in range(cta, units, G):
        tile, ks = divmod(unit, pl["split_k"])
        k0 = ks * pl["kblocks_per_split"]
        if k0 >= kb:  # a cluster rank beyond the last k-block: no arithmetic, it only shares in the reduction
            assert pl["variant"] in (V_CLUSTER, V_GCLUSTER)
            continue
        out.append((tile, k0, min(k0 + pl["kblocks_per_split"], kb), ks * pl["dp_tiles"] + tile if pl["split_k"] > 1 else -1))
    if pl["tail_tiles"]:
        total = pl["tail_tiles"] * kb
        start, end = cta * pl["tail_ipc"], min((cta + 1) * pl["tail_ipc"], total)
        seg = 0
        while start < end:
            trel = start // kb
            stop = min(end, (trel + 1) * kb)
            whole = (start - trel * kb == 0) and (stop - trel * kb == kb)
            out.append((pl["dp_tiles"] + trel, start - trel * kb, stop - trel * kb, -1 if whole else ("tail", 2 * cta + seg)))
            start = stop
            seg += 1
        assert seg <= 2, "a span may cover at most two tile segments"
    return out


def _check_cover_unaddressable(shape):
    return _check_cover(shape, tma_addressable=False)


def _check_cover(shape, sm_count=148, tma_addressable=True):
    pl = dg.dgemm_plan(*shape, sm_count=sm_count, tma_addressable=tma_addressable)
    tiles = -(-shape[0] // pl["bm"]) * -(-shape[1] // pl["bn"])
    assert pl["dp_tiles"] + pl["tail_tiles"] == tiles
    if pl["variant"] in (V_CLUSTER, V_GCLUSTER):  # one CTA per (tile, rank); clusters beyond the resident ones run in turn
        assert pl["grid"] == tiles * pl["split_k"] and pl["split_k"] in (1, 2, 4, 8) and pl["tail_tiles"] == 0
        assert (pl["bm"], pl["bn"], pl["ctas_per_sm"]) == (64, 128, 2)
    else:
        assert 1 <= pl["grid"] <= sm_count * pl["ctas_per_sm"]
    assert pl["kblocks"] == -(-shape[2] // 16)
    seen = {}
    slots = set()
    for cta in range(pl["grid"]):
        for tile, k0, k1, slot in _items(pl, cta):
            assert 0 <= tile < tiles and 0 <= k0 < k1 <= pl["kblocks"]
            for k in range(k0, k1):
                assert (tile, k) not in seen, (shape, tile, k)
                seen[(tile, k)] = cta
            if slot != -1:
                assert slot not in slots
                slots.add(slot)
            else:
                assert (k0, k1) == (0, pl["kblocks"])  # only a whole tile is added straight into C
    assert len(seen) == tiles * pl["kblocks"], shape
    return pl


@pytest.mark.parametrize("shape", [(128, 128, 128), (256, 256, 256), (512, 512, 512), (1024, 1024, 1024), (2304, 2304, 2304),
                                   (1000, 1537, 777), (2088, 2088, 2088), (4097, 31, 4099), (4096, 4096, 160),
                                   (32, 4096, 4096), (96, 2000, 512), (2000, 64, 2048), (6514, 146, 472), (1, 1, 1), (17, 5, 33)])
def test_every_kblock_of_every_tile_is_computed_once(shape):
    _check_cover(shape)


def test_cover_random_shapes_and_forced_splits():
    rnd = random.Random(0)
    for i in range(150):
        shape = tuple(rnd.choice([rnd.randint(1, 64), rnd.randint(1, 600), rnd.randint(1, 3000)]) for _ in range(3))
        dg.dgemm_set_split_k(rnd.choice([0, 0, 0, 2, 3, 7, 8, 64]))
        dg.dgemm_set_variant(rnd.choice([dg.DGEMM_VARIANT_AUTO, dg.DGEMM_VARIANT_AUTO, V_TMA, V_GENERIC, V_WS, V_CLUSTER]))
        dg.dgemm_set_test_flags(rnd.choice([0, 0, 4, 8, 12, 32]))
        _check_cover(shape, sm_count=rnd.choice([148, 132, 8]))


def test_forced_split_has_no_empty_partition():
    dg.dgemm_set_split_k(7)
    pl = _check_cover((300, 300, 1000))
    assert pl["split_k"] * pl["kblocks_per_split"] >= pl["kblocks"] > (pl["split_k"] - 1) * pl["kblocks_per_split"]
    dg.dgemm_set_split_k(64)
    assert _check_cover((128, 128, 48))["split_k"] == 3   # never more partitions than k-blocks


def test_cluster_plan():
    """AUTO below one wave of tiles: clusters of 2, 4 or 8 CTAs per 64 x 128 tile, every CTA on an SM
    of its own, at most 8 k-blocks per CTA; the test flag restores the workspace split."""
    rnd = random.Random(1)
    picked = 0
    for i in range(400):
        shape = (rnd.randint(1, 1200), rnd.randint(1, 1200), rnd.randint(1, 800))
        pl = dg.dgemm_plan(*shape)
        if pl["variant"] != V_CLUSTER:
            continue
        picked += 1
        tiles = -(-shape[0] // 64) * -(-shape[1] // 128)
        assert pl["split_k"] in (2, 4, 8) and pl["grid"] == tiles * pl["split_k"] <= 148
        assert pl["kblocks_per_split"] == -(-pl["kblocks"] // pl["split_k"]) <= 8
        _check_cover(shape)
        dg.dgemm_set_test_flags(dg.DGEMM_TEST_NO_CLUSTER)
        assert dg.dgemm_plan(*shape)["variant"] != V_CLUSTER
        dg.dgemm_set_test_flags(0)
    assert picked > 20
    assert dg.dgemm_plan(128, 128, 128, sm_count=8)["variant"] != V_CLUSTER  # 16 CTAs do not fit 8 SMs
    # forced: the cluster size follows dgemm_set_split_k when that is a legal size
    dg.dgemm_set_variant(V_CLUSTER)
    for s in (1, 2, 4, 8):
        dg.dgemm_set_split_k(s)
        pl = _check_cover((200, 300, 40))   # 3 k-blocks: with 4 and 8 CTAs some ranks idle
        assert pl["split_k"] == s and pl["kblocks_per_split"] == -(-3 // s)
    dg.dgemm_set_split_k(0)
    assert _check_cover((3000, 3000, 3000))["split_k"] == 1  # 1128 tiles: no room for more than one CTA each
    with pytest.raises(dg.DgemmError):
        dg.dgemm_plan(128, 128, 128, tma_addressable=False)
    # operands TMA cannot address: the same kernel with the generic staging
    dg.dgemm_set_variant(dg.DGEMM_VARIANT_AUTO)
    pl = _check_cover_unaddressable((282, 85, 44))
    assert pl["variant"] == V_GCLUSTER and pl["split_k"] in (2, 4, 8)
    assert dg.dgemm_plan(1000, 1000, 1000, tma_addressable=False)["variant"] == V_GENERIC
    dg.dgemm_set_variant(V_GCLUSTER)
    assert dg.dgemm_plan(200, 300, 40, tma_addressable=False)["variant"] == V_GCLUSTER
