"""The CTA-pair kernel ("kernel" = 2) behind every entry point that launches the forward kernel:
its per-row arithmetic is the default kernel's, so attn_fwd, attn_fwd_strided, attn_fwd_host,
attn_fwd_noalloc and attn_fwd_splitkv must give, bit for bit, what they give with "kernel" = 0
(whose results the other GPU tests compare with the oracle), and one case is checked against
the oracle directly."""
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
    for name, value in (("scheduler", 2), ("max_ctas", 0), ("kernel", 0)):
        lib.attn_set_option(name, value)
    yield
    lib.attn_set_option("kernel", 0)


def both_kernels(run):
    """run() -> (o, lse) under the option in force; returns the results of kernels 0 and 2."""
    out = {}
    try:
        for kern in (0, 2):
            lib.attn_set_option("kernel", kern)
            o, lse = run()
            torch.cuda.synchronize()
            assert lib.attn_last_device_status()[:2] == (0, 0)
            out[kern] = (o.clone(), lse.clone())
    finally:
        lib.attn_set_option("kernel", 0)
    return out[0], out[2]


def assert_same_bits(a, b):
    assert torch.equal(a[0].contiguous().view(torch.int16), b[0].contiguous().view(torch.int16))
    assert torch.equal(a[1], b[1])


def fresh_outputs(q, device="cuda"):
    B, Sq, Hq, _ = q.shape
    o = torch.full((B, Sq, Hq, 128), float("nan"), device=device, dtype=torch.bfloat16)
    lse = torch.full((B, Hq, Sq), float("nan"), device=device, dtype=torch.float32)
    return o, lse


CASES = [(2, 4, 4, 1100, 1100, True), (1, 6, 2, 700, 900, False), (1, 3, 3, 513, 640, True)]


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,causal", CASES)
def test_contiguous_and_noalloc_entry_points(B, Hq, Hkv, Sq, Sk, causal):
    q, k, v = (t.cuda() for t in make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=9400 + Sq))

    def plain():
        o, lse = fresh_outputs(q)
        lib.attn_fwd(q, k, v, o, lse, causal, SCALE)
        return o, lse

    def noalloc():
        o, lse = fresh_outputs(q)
        lib.attn_fwd_noalloc(q, k, v, o, lse, causal, SCALE)
        return o, lse

    a0, a2 = both_kernels(plain)
    assert_same_bits(a0, a2)
    b0, b2 = both_kernels(noalloc)
    assert_same_bits(a0, b2)
    assert_same_bits(b0, b2)


def test_against_the_oracle():
    B, Hq, Hkv, Sq, Sk, causal = 1, 4, 2, 900, 1030, True
    qc, kc, vc = make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=9500)
    q, k, v = qc.cuda(), kc.cuda(), vc.cuda()
    lib.attn_set_option("kernel", 2)
    try:
        o, lse = fresh_outputs(q)
        lib.attn_fwd(q, k, v, o, lse, causal, SCALE)
        torch.cuda.synchronize()
        assert lib.attn_last_device_status()[:2] == (0, 0)
    finally:
        lib.attn_set_option("kernel", 0)
    o_ref, lse_ref = orc.attention_full(bf16_bits(qc), bf16_bits(kc), bf16_bits(vc), causal, SCALE)
    assert np.abs(bits_to_float64(bf16_bits(o.cpu())) - o_ref).max() <= TOL_O
    assert np.abs(lse.cpu().numpy().astype(np.float64) - lse_ref).max() <= TOL_LSE


def test_strided_views():
    B, Hq, Hkv, Sq, Sk = 2, 4, 2, 600, 777
    q, k, v = (t.cuda() for t in make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=9600))
    # [B, H, S, D] storage handed over as [B, S, H, D] views
    qv, kv, vv = (t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for t in (q, k, v))

    def strided():
        o_store = torch.full((B, Hq, Sq, 128), float("nan"), device="cuda", dtype=torch.bfloat16)
        lse = torch.full((B, Hq, Sq), float("nan"), device="cuda", dtype=torch.float32)
        lib.attn_fwd_strided(qv, kv, vv, o_store.permute(0, 2, 1, 3), lse, True, SCALE)
        return o_store, lse

    assert_same_bits(*both_kernels(strided))


def test_host_buffers_and_split_kv():
    B, Hq, Hkv, Sq, Sk, causal = 1, 4, 4, 1536, 1536, True
    qc, kc, vc = make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=9700)

    def host():
        o, lse = fresh_outputs(qc, device="cpu")
        lib.attn_fwd_host(qc, kc, vc, o, lse, causal, SCALE)
        return o, lse

    assert_same_bits(*both_kernels(host))
    q, k, v = qc.cuda(), kc.cuda(), vc.cuda()

    def split():
        o, lse = fresh_outputs(q)
        lib.attn_fwd_splitkv(q, k, v, o, lse, causal, SCALE, 3)
        return o, lse

    assert_same_bits(*both_kernels(split))
    lib.attn_release_host_staging()
