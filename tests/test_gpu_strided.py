"""GPU parity of attn_fwd_strided: the same kernel on strided views must give, bit for bit, what
attn_fwd gives on contiguous copies of those views, and that result matches the oracle."""
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


def contiguous_result(q, k, v, causal):
    qc, kc, vc = q.contiguous(), k.contiguous(), v.contiguous()
    o = torch.full_like(qc, float("nan"))
    lse = torch.full((q.shape[0], q.shape[2], q.shape[1]), float("nan"), device="cuda", dtype=torch.float32)
    lib.attn_fwd(qc, kc, vc, o, lse, causal, SCALE)
    torch.cuda.synchronize()
    return o, lse


def check_oracle(q, k, v, causal, o, lse):
    o_ref, lse_ref = orc.attention_full(bf16_bits(q.contiguous().cpu()), bf16_bits(k.contiguous().cpu()),
                                        bf16_bits(v.contiguous().cpu()), causal, SCALE)
    assert np.abs(bits_to_float64(bf16_bits(o.contiguous().cpu())) - o_ref).max() <= TOL_O
    assert np.abs(lse.cpu().numpy().astype(np.float64) - lse_ref).max() <= TOL_LSE


@pytest.mark.parametrize("causal", [False, True])
def test_head_major_buffers_viewed_as_sequence_major(causal):
    B, Hq, Hkv, Sq, Sk = 2, 4, 2, 300, 427
    q, k, v = (t.cuda() for t in make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=9100))
    # [B, H, S, D] storage, handed over as [B, S, H, D] views; O is written into such a view too
    qv = q.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    kv = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vv = v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert not qv.is_contiguous() and qv.stride(2) == Sq * 128
    o_store = torch.full((B, Hq, Sq, 128), float("nan"), device="cuda", dtype=torch.bfloat16)
    ov = o_store.permute(0, 2, 1, 3)
    lse = torch.full((B, Hq, Sq), float("nan"), device="cuda", dtype=torch.float32)
    lib.attn_fwd_strided(qv, kv, vv, ov, lse, causal, SCALE)
    torch.cuda.synchronize()
    assert lib.attn_last_device_status()[:2] == (0, 0)
    o_ref, lse_ref = contiguous_result(q, k, v, causal)
    assert torch.equal(ov.contiguous().view(torch.int16), o_ref.view(torch.int16))
    assert torch.equal(lse, lse_ref)
    check_oracle(q, k, v, causal, ov, lse)


def test_slices_of_a_packed_projection():
    B, S, H = 1, 260, 3
    g = torch.Generator().manual_seed(9200)
    packed = torch.randn((B, S, 3, H, 128), generator=g).to(torch.bfloat16).cuda()
    q, k, v = packed[:, :, 0], packed[:, :, 1], packed[:, :, 2]
    assert q.stride(1) == 3 * H * 128 and not q.is_contiguous()
    o = torch.full((B, S, H, 128), float("nan"), device="cuda", dtype=torch.bfloat16)
    lse = torch.full((B, H, S), float("nan"), device="cuda", dtype=torch.float32)
    lib.attn_fwd_strided(q, k, v, o, lse, True, SCALE)
    torch.cuda.synchronize()
    o_ref, lse_ref = contiguous_result(q, k, v, True)
    assert torch.equal(o.view(torch.int16), o_ref.view(torch.int16)) and torch.equal(lse, lse_ref)
    check_oracle(q, k, v, True, o, lse)


def test_key_ranges_plus_merge_equal_the_whole_sequence():
    """Split-KV by views: two launches on disjoint key ranges of the same K/V buffers, merged with
    attn_merge, against the oracle over all keys."""
    B, Hq, Hkv, Sq, Sk, cut = 1, 4, 4, 130, 700, 384
    q, k, v = (t.cuda() for t in make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=9300))
    parts = []
    for lo, hi in ((0, cut), (cut, Sk)):
        o = torch.full_like(q, float("nan"))
        lse = torch.full((B, Hq, Sq), float("nan"), device="cuda", dtype=torch.float32)
        lib.attn_fwd_strided(q, k[:, lo:hi], v[:, lo:hi], o, lse, False, SCALE)
        parts.append((o, lse))
    o = torch.empty_like(q)
    lse = torch.empty((B, Hq, Sq), device="cuda", dtype=torch.float32)
    lib.attn_merge(parts[0][0], parts[0][1], parts[1][0], parts[1][1], o, lse)
    torch.cuda.synchronize()
    o_ref, lse_ref = orc.attention_full(bf16_bits(q.cpu()), bf16_bits(k.cpu()), bf16_bits(v.cpu()), False, SCALE)
    # three BF16 roundings of O on this path (two partial results, one merged)
    assert np.abs(bits_to_float64(bf16_bits(o.cpu())) - o_ref).max() <= TOL_O
    assert np.abs(lse.cpu().numpy().astype(np.float64) - lse_ref).max() <= TOL_LSE


def test_bad_strides_are_refused_before_launch():
    q, k, v = (t.cuda() for t in make_qkv(1, 2, 2, 128, 128, 128, seed=9400))
    o = torch.empty_like(q)
    odd = torch.empty((1, 128, 2, 136), device="cuda", dtype=torch.bfloat16)[..., :128]   # row stride 136: fine
    assert lib.attn_fwd_strided_status(q, k, v, odd, None, False, SCALE) == 0
    bad = torch.empty((1, 128, 2, 132), device="cuda", dtype=torch.bfloat16)[..., :128]   # 132 % 8 != 0
    assert lib.attn_fwd_strided_status(q, k, v, bad, None, False, SCALE) == 4            # ATTN_ERR_ALIGN
    torch.cuda.synchronize()
    assert o is not None
