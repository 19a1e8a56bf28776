"""GPU parity of attn_merge (LSE-weighted merge of partial attention results) against the CPU
oracle, and the split-key use it exists for: two attn_fwd calls on halves of K/V plus one merge
equal attention over all keys."""
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
# The merge is fp32 arithmetic plus ONE rounding of O to BF16: half an ulp is at most 2^-8 |O|.
# LSE is fp32 with expf / logf.
REL_O_MERGE = 2.0 ** -8
TOL_LSE_MERGE = 1e-5


@pytest.fixture(scope="module", autouse=True)
def _library():
    lib_build.build()
    lib.load_library()
    for k, v in (("scheduler", 2), ("max_ctas", 0), ("kernel", 0)):
        lib.attn_set_option(k, v)


@pytest.mark.parametrize("B,Hq,Sq", [(1, 1, 1), (2, 3, 77), (1, 16, 1000), (4, 8, 513)])
def test_merge_matches_oracle_elementwise(B, Hq, Sq):
    g = torch.Generator().manual_seed(8000 + Sq)
    o1 = torch.randn((B, Sq, Hq, 128), generator=g).to(torch.bfloat16)
    o2 = torch.randn((B, Sq, Hq, 128), generator=g).to(torch.bfloat16)
    l1 = (torch.randn((B, Hq, Sq), generator=g) * 3).float()
    l2 = (torch.randn((B, Hq, Sq), generator=g) * 3).float()
    l2[0, 0, 0] = float("-inf")                      # an empty part
    if Sq > 2:
        l1[0, 0, 1] = float("-inf")
        l1[0, 0, 2] = l2[0, 0, 2] = float("-inf")    # both empty
    o = torch.full_like(o1, float("nan")).cuda()
    lse = torch.full((B, Hq, Sq), float("nan")).cuda()
    lib.attn_merge(o1.cuda(), l1.cuda(), o2.cuda(), l2.cuda(), o, lse)
    torch.cuda.synchronize()
    # oracle rows are in O's order [B, Sq, Hq]; LSE tensors are [B, Hq, Sq]
    to_rows = lambda t: t.permute(0, 2, 1).contiguous().numpy()
    o_ref, lse_ref = orc.merge(bf16_bits(o1), to_rows(l1), bf16_bits(o2), to_rows(l2))
    o64 = bits_to_float64(bf16_bits(o.cpu()))
    assert not np.isnan(o64).any()
    assert np.all(np.abs(o64 - o_ref) <= REL_O_MERGE * np.abs(o_ref) + 1e-5)
    got = to_rows(lse.cpu()).astype(np.float64)
    both_empty = np.isneginf(lse_ref)
    assert np.array_equal(np.isneginf(got), both_empty)
    assert np.abs(got[~both_empty] - lse_ref[~both_empty]).max() <= TOL_LSE_MERGE


def test_merge_in_place_and_argument_errors():
    o1 = torch.randn((1, 64, 2, 128)).to(torch.bfloat16).cuda()
    o2 = torch.randn((1, 64, 2, 128)).to(torch.bfloat16).cuda()
    l1 = torch.randn((1, 2, 64)).cuda()
    l2 = torch.randn((1, 2, 64)).cuda()
    o = torch.empty_like(o1)
    lse = torch.empty_like(l1)
    lib.attn_merge(o1, l1, o2, l2, o, lse)
    o1_copy = o1.clone()
    lib.attn_merge(o1_copy, l1, o2, l2, o1_copy, torch.empty_like(l1))  # output over the first input
    torch.cuda.synchronize()
    assert torch.equal(o.view(torch.int16), o1_copy.view(torch.int16))
    assert lib.attn_merge_status(o1, l1, o2, l2, o, l1) == 3             # lse aliases an input
    cdll = lib.load_library()
    assert cdll.attn_merge(None, l1.data_ptr(), o2.data_ptr(), l2.data_ptr(), o.data_ptr(), lse.data_ptr(),
                           1, 2, 64, 128, None) == 1
    assert cdll.attn_merge(o1.data_ptr(), l1.data_ptr(), o2.data_ptr(), l2.data_ptr(), o.data_ptr(),
                           lse.data_ptr(), 1, 2, 64, 64, None) == 3


def test_empty_part_may_hold_anything_also_in_place():
    """A part with LSE = -inf has weight 0 and its O is never used: a buffer nobody wrote (NaN
    here) must not poison the row, whether the result goes to a fresh buffer or over one input.
    The oracle, whose two-part form multiplies by the zero weight, gets zeros in those rows."""
    B, Hq, Sq = 2, 4, 130
    g = torch.Generator().manual_seed(8200)
    o1 = torch.randn((B, Sq, Hq, 128), generator=g).to(torch.bfloat16)
    o2 = torch.randn((B, Sq, Hq, 128), generator=g).to(torch.bfloat16)
    l1 = torch.randn((B, Hq, Sq), generator=g).float()
    l2 = torch.randn((B, Hq, Sq), generator=g).float()
    l1[:, :, ::3] = float("-inf")          # part 1 empty in every third row
    l2[:, 1, 1::3] = float("-inf")         # part 2 empty elsewhere
    o1_dev, o2_dev = o1.clone(), o2.clone()
    o1_dev.permute(0, 2, 1, 3)[torch.isneginf(l1)] = float("nan")
    o2_dev.permute(0, 2, 1, 3)[torch.isneginf(l2)] = float("nan")
    o1_ref, o2_ref = o1.clone(), o2.clone()
    o1_ref.permute(0, 2, 1, 3)[torch.isneginf(l1)] = 0.0
    o2_ref.permute(0, 2, 1, 3)[torch.isneginf(l2)] = 0.0
    to_rows = lambda t: t.permute(0, 2, 1).contiguous().numpy()
    o_ref, lse_ref = orc.merge(bf16_bits(o1_ref), to_rows(l1), bf16_bits(o2_ref), to_rows(l2))
    for in_place in (False, True):
        a, b = o1_dev.cuda(), o2_dev.cuda()
        o = a if in_place else torch.full_like(a, float("nan"))
        lse = torch.full((B, Hq, Sq), float("nan")).cuda()
        lib.attn_merge(a, l1.cuda(), b, l2.cuda(), o, lse)
        torch.cuda.synchronize()
        o64 = bits_to_float64(bf16_bits(o.cpu()))
        assert not np.isnan(o64).any()
        assert np.all(np.abs(o64 - o_ref) <= REL_O_MERGE * np.abs(o_ref) + 1e-5)
        assert np.abs(to_rows(lse.cpu()).astype(np.float64) - lse_ref).max() <= TOL_LSE_MERGE


def test_split_keys_then_merge_equals_attention_over_all_keys():
    B, Hq, Hkv, Sq, Sk = 2, 8, 2, 300, 1000
    q, k, v = make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=8100)
    cut = 384
    qd = q.cuda()
    parts = []
    for ks, vs in ((k[:, :cut], v[:, :cut]), (k[:, cut:], v[:, cut:])):
        o_p = torch.empty_like(qd)
        l_p = torch.empty((B, Hq, Sq), device="cuda", dtype=torch.float32)
        lib.attn_fwd(qd, ks.contiguous().cuda(), vs.contiguous().cuda(), o_p, l_p, False, SCALE)
        parts.append((o_p, l_p))
    o = torch.empty_like(qd)
    lse = torch.empty((B, Hq, Sq), device="cuda", dtype=torch.float32)
    lib.attn_merge(parts[0][0], parts[0][1], parts[1][0], parts[1][1], o, lse)
    torch.cuda.synchronize()
    o_ref, lse_ref = orc.attention_full(bf16_bits(q), bf16_bits(k), bf16_bits(v), False, SCALE)
    assert np.abs(bits_to_float64(bf16_bits(o.cpu())) - o_ref).max() <= 2e-2
    assert np.abs(lse.cpu().numpy().astype(np.float64) - lse_ref).max() <= 1e-3
