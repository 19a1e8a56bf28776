"""GPU parity of attn_merge_n (element by element against the oracle's n-way merge) and of
attn_fwd_splitkv (against the oracle's attention over all keys: the split is only a route)."""
import math

import numpy as np
import pytest
import torch

import paper_2603_24517_b200 as lib
from paper_2603_24517_b200 import build as lib_build
from oracle import attn_oracle as orc
from workloads import bf16_bits, bits_to_float64, make_qkv

pytestmark = pytest.mark.gpu

SCALE = float(np.float32(1.0 / math.sqrt(128)))
TOL_O, TOL_LSE = 2e-2, 1e-3


@pytest.fixture(scope="module", autouse=True)
def _library():
    lib_build.build()
    lib.load_library()
    lib.attn_set_option("scheduler", 2)
    lib.attn_set_option("max_ctas", 0)
    lib.attn_set_option("kernel", 0)
    yield


@pytest.mark.parametrize("n", [1, 2, 3, 7])
def test_merge_n_matches_oracle(n):
    B, Sq, Hq = 2, 150, 3
    g = torch.Generator().manual_seed(9500 + n)
    o_parts = (2.0 * torch.randn((n, B, Sq, Hq, 128), generator=g)).to(torch.bfloat16)
    lse_parts = 3.0 * torch.randn((n, B, Hq, Sq), generator=g)
    lse_parts[0, 0, 0, :7] = float("-inf")            # an empty part on some rows
    lse_parts[:, 1, 2, 5] = float("-inf")             # a row whose parts are all empty
    o = torch.full((B, Sq, Hq, 128), float("nan"), device="cuda", dtype=torch.bfloat16)
    lse = torch.full((B, Hq, Sq), float("nan"), device="cuda")
    lib.attn_merge_n(o_parts.cuda(), lse_parts.cuda(), o, lse)
    torch.cuda.synchronize()
    # the oracle's rows are ordered like O: (b, i, h); its LSE parts must follow the same order
    l_rows = lse_parts.permute(0, 1, 3, 2).contiguous()           # [n, B, Sq, Hq]
    o_ref, l_ref = orc.merge_n(bf16_bits(o_parts), l_rows.numpy())
    o64 = bits_to_float64(bf16_bits(o.cpu()))
    l64 = lse.cpu().permute(0, 2, 1).numpy().astype(np.float64)    # -> [B, Sq, Hq]
    assert not np.isnan(o64).any()
    # one rounding of O to BF16: half an ulp, relative 2^-9, plus fp32 accumulation
    assert np.all(np.abs(o64 - o_ref) <= 2.0 ** -8 * np.abs(o_ref) + 1e-5)
    empty = np.isneginf(l_ref)
    assert np.array_equal(np.isneginf(l64), empty) and empty.sum() == 1 + (7 if n == 1 else 0)
    assert np.abs(l64[~empty] - l_ref[~empty]).max() <= 1e-5
    assert np.all(o64[empty] == 0)


CASES = [
    # B, Hq, Hkv, Sq, Sk, causal, n_splits
    (1, 4, 4, 1, 1500, False, 8),       # decoding: one query row, ragged last range
    (2, 8, 2, 16, 2048, False, 4),      # GQA, equal ranges
    (1, 4, 2, 130, 1000, True, 3),      # causal, Sq < Sk: early ranges fully visible, the last one masked
    (1, 2, 2, 300, 300, True, 4),       # causal, Sq = Sk: rows that see nothing of the later ranges
    (1, 2, 2, 64, 100, False, 5),       # fewer keys than ranges: a single range, plain forward
    (1, 2, 1, 200, 700, True, 64),      # more ranges asked for than tiles: one tile per range
]


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,causal,n_splits", CASES)
def test_splitkv_matches_oracle_over_all_keys(B, Hq, Hkv, Sq, Sk, causal, n_splits):
    q, k, v = make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=9600 + Sk)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    o = torch.full_like(qd, float("nan"))
    lse = torch.full((B, Hq, Sq), float("nan"), device="cuda")
    lib.attn_fwd_splitkv(qd, kd, vd, o, lse, causal, SCALE, n_splits)
    torch.cuda.synchronize()
    assert lib.attn_last_device_status()[:2] == (0, 0)
    o_ref, l_ref = orc.attention_full(bf16_bits(q), bf16_bits(k), bf16_bits(v), causal, SCALE)
    o64 = bits_to_float64(bf16_bits(o.cpu()))
    l64 = lse.cpu().numpy().astype(np.float64)
    assert not np.isnan(o64).any() and not np.isnan(l64).any()
    assert np.abs(o64 - o_ref).max() <= TOL_O
    assert np.abs(l64 - l_ref).max() <= TOL_LSE


def test_splitkv_argument_errors_and_workspace():
    q, k, v = (t.cuda() for t in make_qkv(1, 2, 2, 8, 1024, 128, seed=9700))
    o = torch.empty_like(q)
    need = lib.attn_splitkv_workspace_bytes(1, 2, 8, 128, 4)
    assert need == 4 * 1 * 8 * 2 * (2 * 128 + 4)
    small = torch.empty(need - 16, dtype=torch.uint8, device="cuda")
    assert lib.attn_fwd_splitkv_status(q, k, v, o, None, False, SCALE, 4, workspace=small) == 8   # ATTN_ERR_TOO_LARGE
    assert lib.attn_fwd_splitkv_status(q, k, v, o, None, False, SCALE, 0) == 2                     # ATTN_ERR_SHAPE
    assert lib.attn_fwd_splitkv_status(q, k, v, o, None, False, SCALE, 65) == 3                    # ATTN_ERR_UNSUPPORTED
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    assert lib.attn_fwd_splitkv_status(q, k, v, o, None, False, SCALE, 4, workspace=ws) == 0       # lse may be NULL
    torch.cuda.synchronize()


# ---- short GQA query sequences: the heads of a KV group packed into the rows of one tile --------
PACKED = [
    # B, Hq, Hkv, Sq, Sk, causal
    (2, 8, 2, 1, 700, False),      # decoding, group 4: rows 0..3 of a tile are the 4 heads
    (2, 8, 2, 1, 700, True),
    (1, 8, 2, 17, 300, True),      # 17 rows x 4 heads in one tile of 32 x 4
    (2, 8, 2, 40, 700, True),      # two packed tiles: both stages busy, ragged second tile
    (1, 8, 2, 64, 64, True),       # Sq = Sk, diagonal inside the packed tiles
    (1, 8, 1, 32, 515, False),     # group 8: two tiles of 16 rows
    (1, 8, 1, 5, 130, True),
    (3, 4, 2, 128, 128, True),     # group 2: two tiles of 64 rows
    (1, 16, 1, 9, 1000, False),    # group 16: 8 rows per tile
    (1, 8, 2, 20, 9, True),        # Sq > Sk: packed rows without any visible key
]


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,causal", PACKED)
def test_packed_gqa_tiles_match_oracle_and_the_unpacked_path(B, Hq, Hkv, Sq, Sk, causal):
    plan = lib.attn_plan(B, Hq, Hkv, Sq, Sk, 128, causal, 148)
    assert plan["n_work"] == B * Hkv * math.ceil(math.ceil(Sq / (128 // (Hq // Hkv))) / 2)   # the packed plan is in use
    q, k, v = make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=9800 + Sq)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    outs = []
    for pack in (1, 0):
        lib.attn_set_option("gqa_pack", pack)
        try:
            o = torch.full_like(qd, float("nan"))
            lse = torch.full((B, Hq, Sq), float("nan"), device="cuda")
            lib.attn_fwd(qd, kd, vd, o, lse, causal, SCALE)
            torch.cuda.synchronize()
            assert lib.attn_last_device_status()[:2] == (0, 0)
            outs.append((o.cpu(), lse.cpu()))
        finally:
            lib.attn_set_option("gqa_pack", 1)
    # per row the arithmetic is the same in both layouts
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))
    assert torch.equal(outs[0][1], outs[1][1])
    o_ref, l_ref = orc.attention_full(bf16_bits(q), bf16_bits(k), bf16_bits(v), causal, SCALE)
    o64 = bits_to_float64(bf16_bits(outs[0][0]))
    l64 = outs[0][1].numpy().astype(np.float64)
    assert not np.isnan(o64).any() and not np.isnan(l64).any()
    assert np.abs(o64 - o_ref).max() <= TOL_O
    empty = np.isneginf(l_ref)
    assert np.array_equal(np.isneginf(l64), empty)
    assert np.abs(l64[~empty] - l_ref[~empty]).max() <= TOL_LSE
