"""Host logic of the tile scheduler, checked against brute force on the CPU: every 128-row
query tile of every (batch, query head) is covered exactly once, GQA stages share a KV head,
and a stage visits exactly the K/V blocks that hold at least one visible key (paper,
Section 2.2: fully masked key blocks are skipped under the causal mask)."""
import math

import pytest

import paper_2603_24517_b200 as lib
from paper_2603_24517_b200 import build as lib_build

TILE = 128


@pytest.fixture(scope="module", autouse=True)
def _built():
    lib_build.build()
    lib.attn_set_option("scheduler", 2)
    lib.attn_set_option("max_ctas", 0)
    lib.attn_set_option("kernel", 0)
    yield
    lib.attn_set_option("kernel", 0)


def packed_group(Hq, Hkv, Sq):
    """Query heads per tile row group when the library packs a GQA group into one tile (short
    query sequences, dual-stage kernel): the whole group must fit two packed tiles."""
    g = Hq // Hkv
    if 2 <= g <= 16 and g & (g - 1) == 0 and Sq <= 2 * (TILE // g):
        return g
    return 1


def visible_blocks_brute(row0, Sq, Sk, causal, tile_rows=TILE):
    rows = range(row0, min(row0 + tile_rows, Sq))
    if not causal:
        return math.ceil(Sk / TILE)
    last_key = max(min(Sk - 1, i + Sk - Sq) for i in rows)
    if last_key < 0:  # Sq > Sk: no row of the tile sees a key; one masked block is still visited
        return 1      # so that the tile's O = 0 and LSE = -inf get written
    return last_key // TILE + 1


CASES = [
    (1, 2, 2, 512, 512, False), (1, 2, 2, 512, 512, True), (2, 3, 3, 384, 640, True),
    (1, 8, 2, 300, 300, True), (1, 8, 2, 300, 700, False), (2, 32, 8, 1024, 1024, True),
    (1, 32, 4, 640, 640, True), (1, 6, 2, 130, 130, True), (1, 5, 5, 1, 1, False),
    (3, 4, 4, 129, 1000, True), (1, 16, 16, 16384, 16384, True),
    (1, 2, 2, 640, 128, True), (2, 4, 2, 700, 77, True), (1, 8, 2, 513, 300, True),  # Sq > Sk
    (2, 8, 2, 1, 700, False), (2, 8, 2, 40, 700, True), (1, 8, 1, 32, 300, True), (3, 4, 2, 128, 128, True),
    (1, 16, 1, 9, 1000, False), (1, 8, 2, 65, 700, True),  # short GQA queries: packed tiles (the last one is too long)
]


@pytest.mark.parametrize("kernel", [0, 1])
@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,causal", CASES)
def test_plan_covers_every_tile_once(kernel, B, Hq, Hkv, Sq, Sk, causal):
    lib.attn_set_option("kernel", kernel)
    plan = lib.attn_plan(B, Hq, Hkv, Sq, Sk, 128, causal, 148)
    g = Hq // Hkv
    pack = packed_group(Hq, Hkv, Sq) if kernel == 0 else 1
    tile_rows = TILE // pack
    if kernel == 1:  # one query tile per work item
        assert plan["pair_heads"] == 0 and plan["n_work"] == B * Hq * math.ceil(Sq / TILE)
    elif pack > 1:   # a tile holds tile_rows query rows of all heads of a KV group
        assert plan["pair_heads"] == 0 and plan["n_work"] == B * Hkv * math.ceil(math.ceil(Sq / tile_rows) / 2)
    else:
        assert plan["pair_heads"] == (1 if g % 2 == 0 else 0)
    assert plan["n_q_tiles"] == math.ceil(Sq / tile_rows) and plan["n_kv_blocks"] == math.ceil(Sk / TILE)
    assert plan["ctas"] == min(148, plan["n_work"])
    seen = {}
    n_work = plan["n_work"]
    step = 1 if n_work <= 4096 else 7  # large cases: a stride-7 sample plus the ends
    ws = sorted(set(list(range(0, n_work, step)) + [n_work - 1]))
    for w in ws:
        it = lib.attn_plan_item(B, Hq, Hkv, Sq, Sk, 128, causal, w)
        assert 0 <= it["b"] < B and 0 <= it["hkv"] < Hkv
        for s in (0, 1):
            hq, row0, n = it[f"hq{s}"], it[f"row0_{s}"], it[f"n_blocks_{s}"]
            assert 0 <= hq < Hq and hq // g == it["hkv"] and row0 % tile_rows == 0
            if pack > 1:
                assert hq == it["hkv"] * g  # the first head of the packed group
            if row0 >= Sq:
                assert n == 0
                continue
            assert n == visible_blocks_brute(row0, Sq, Sk, causal, tile_rows)
            key = (it["b"], hq, row0)
            assert key not in seen
            seen[key] = w
    if step == 1:
        assert len(seen) == B * (Hkv if pack > 1 else Hq) * math.ceil(Sq / tile_rows)


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,causal", CASES)
def test_pair_plan_covers_every_tile_once(B, Hq, Hkv, Sq, Sk, causal):
    """CTA-pair kernel: the four tiles of a work item (two stages x two CTAs) cover every query
    tile exactly once; the two tiles of a stage share a block count, which is what the later of
    them needs (brute force), so the earlier one never misses a visible block."""
    lib.attn_set_option("kernel", 2)
    plan = lib.attn_plan(B, Hq, Hkv, Sq, Sk, 128, causal, 148)
    g = Hq // Hkv
    if packed_group(Hq, Hkv, Sq) > 1:  # packed problems keep the one-CTA kernel's plan
        with pytest.raises(lib.AttnError):
            lib.attn_plan_item_pair(B, Hq, Hkv, Sq, Sk, 128, causal, 0, 0)
        return
    n_qt = math.ceil(Sq / TILE)
    if g % 2 == 0:
        assert plan["pair_heads"] == 1 and plan["n_work"] == B * Hkv * math.ceil(n_qt / 2) * (g // 2)
    else:
        assert plan["pair_heads"] == 0 and plan["n_work"] == B * Hq * math.ceil(n_qt / 4)
    assert plan["ctas"] == 2 * min(74, plan["n_work"])
    seen = set()
    n_work = plan["n_work"]
    step = 1 if n_work <= 2048 else 7
    for w in sorted(set(list(range(0, n_work, step)) + [n_work - 1])):
        views = [lib.attn_plan_item_pair(B, Hq, Hkv, Sq, Sk, 128, causal, w, r) for r in (0, 1)]
        assert views[0] == lib.attn_plan_item(B, Hq, Hkv, Sq, Sk, 128, causal, w)
        for s in (0, 1):
            a, b = views
            hq, n = a[f"hq{s}"], a[f"n_blocks_{s}"]
            assert (b["b"], b["hkv"], b[f"hq{s}"], b[f"n_blocks_{s}"]) == (a["b"], a["hkv"], hq, n)
            assert 0 <= hq < Hq and hq // g == a["hkv"]
            assert b[f"row0_{s}"] == a[f"row0_{s}"] + TILE and a[f"row0_{s}"] % (2 * TILE) == 0
            if a[f"row0_{s}"] >= Sq:
                assert n == 0
                continue
            need = [visible_blocks_brute(v[f"row0_{s}"], Sq, Sk, causal) for v in views if v[f"row0_{s}"] < Sq]
            assert n == max(need)
            for v in views:
                if v[f"row0_{s}"] < Sq:
                    key = (v["b"], hq, v[f"row0_{s}"])
                    assert key not in seen
                    seen.add(key)
    if step == 1:
        assert len(seen) == B * Hq * n_qt


def test_causal_items_run_longest_first_inside_a_head():
    lib.attn_set_option("kernel", 0)
    B, H, S = 2, 3, 2048
    plan = lib.attn_plan(B, H, H, S, S, 128, True, 148)
    per_head = {}
    for w in range(plan["n_work"]):
        it = lib.attn_plan_item(B, H, H, S, S, 128, True, w)
        per_head.setdefault((it["b"], it["hq0"]), []).append(it["n_blocks_0"] + it["n_blocks_1"])
    assert len(per_head) == B * H
    for costs in per_head.values():
        assert len(costs) == plan["items_per_group"] and costs == sorted(costs, reverse=True)


def test_causal_launch_order_interleaves_heads_and_ends_on_short_items():
    """Under the causal mask the longest items of several heads go first and the launch ends on
    the shortest ones (a long item started last would leave the other SMs idle)."""
    lib.attn_set_option("kernel", 0)
    B, H, S = 1, 16, 16384
    plan = lib.attn_plan(B, H, H, S, S, 128, True, 148)
    first = [lib.attn_plan_item(B, H, H, S, S, 128, True, w) for w in range(6)]
    assert len({it["hq0"] for it in first}) == 6                       # six different heads ...
    assert all(it["n_blocks_1"] == plan["n_kv_blocks"] for it in first)  # ... each at its longest item
    last = lib.attn_plan_item(B, H, H, S, S, 128, True, plan["n_work"] - 1)
    assert last["n_blocks_0"] + last["n_blocks_1"] == 3
    # non-causal: strictly head-major
    nc = [lib.attn_plan_item(B, H, H, S, S, 128, False, w) for w in range(3)]
    assert {it["hq0"] for it in nc} == {0}


def test_scheduler_option_changes_grid_only():
    lib.attn_set_option("kernel", 0)
    lib.attn_set_option("scheduler", 0)
    try:
        plan = lib.attn_plan(2, 16, 16, 16384, 16384, 128, False, 148)
        assert plan["ctas"] == plan["n_work"] == 2 * 16 * 64
        lib.attn_set_option("scheduler", 1)
        lib.attn_set_option("max_ctas", 100)
        assert lib.attn_plan(2, 16, 16, 16384, 16384, 128, False, 148)["ctas"] == 100
    finally:
        lib.attn_set_option("scheduler", 2)
        lib.attn_set_option("max_ctas", 0)


def test_plan_rejects_bad_problems():
    with pytest.raises(lib.AttnError):
        lib.attn_plan(1, 3, 2, 128, 128, 128, False, 148)
    with pytest.raises(lib.AttnError):
        lib.attn_plan(1, 2, 2, 256, 128, 64, True, 148)
    with pytest.raises(lib.AttnError):
        lib.attn_plan_item(1, 2, 2, 128, 128, 128, False, 99)
