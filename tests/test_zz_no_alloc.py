"""The no-allocation entry point, through the C ABI.

Some callers of this library are not allowed to allocate device memory: a server that gave
all of HBM to its own pools at start-up, a latency-critical thread that must stay off the
driver's allocation lock, a runtime that bans library-side allocations.  For them
``attn_fwd_noalloc`` runs the same kernel with its scratch (tile-scheduler counter, status
words) in a fixed 256-byte array inside the library image instead of cudaMalloc'ed memory.
Every call shares that array and it keeps the previous call's contents, so these tests call
the entry point several times in a row, on problems whose grids differ, and compare every
result bit for bit with ``attn_fwd``'s on the same inputs (same kernel, same arithmetic) and,
independently of the CUDA path, with the CPU oracle.

Collected last on purpose (file name), so that a run that stops at the first failure has
already run every other test.  Passes alone in a fresh process and after the other tests.
"""
import math

import numpy as np
import pytest
import torch

import paper_2603_24517_b200 as lib
from paper_2603_24517_b200 import build as lib_build
from oracle import attn_oracle as orc
from workloads import bf16_bits, bits_to_float64, make_qkv, sample_rows

pytestmark = pytest.mark.gpu

TOL_O = 2e-2     # the tolerances of the oracle parity tests
TOL_LSE = 1e-3
SCALE = float(np.float32(1.0 / math.sqrt(128)))


@pytest.fixture(scope="module", autouse=True)
def _library():
    lib_build.build()
    lib.load_library()
    lib.attn_set_option("scheduler", 2)
    lib.attn_set_option("max_ctas", 0)


def _run(fn, q, k, v, causal):
    o = torch.full_like(q, float("nan"))
    lse = torch.full((q.shape[0], q.shape[2], q.shape[1]), float("nan"), device=q.device, dtype=torch.float32)
    fn(q, k, v, o, lse, causal, SCALE)
    torch.cuda.synchronize()
    return o.cpu(), lse.cpu()


def _same_bits(o, lse, o_ref, lse_ref):
    return (torch.equal(o.view(torch.int16), o_ref.view(torch.int16)) and
            torch.equal(lse.view(torch.int32), lse_ref.view(torch.int32)))


def _check_against_oracle(q, k, v, causal, o, lse, rows=None):
    qb, kb, vb = (bf16_bits(t.cpu()) for t in (q, k, v))
    o64 = bits_to_float64(bf16_bits(o))
    l64 = lse.numpy().astype(np.float64)
    if rows is None:
        o_ref, lse_ref = orc.attention_full(qb, kb, vb, causal, SCALE)
    else:
        o_ref, lse_ref = orc.attention_rows(qb, kb, vb, causal, SCALE, rows)
        o64 = o64[rows[:, 0], rows[:, 2], rows[:, 1]]
        l64 = l64[rows[:, 0], rows[:, 1], rows[:, 2]]
    assert not np.isnan(o64).any() and not np.isnan(l64).any()
    assert np.abs(o64 - o_ref).max() <= TOL_O
    assert np.abs(l64 - lse_ref).max() <= TOL_LSE


def test_two_calls_in_a_row_match_the_allocating_entry_point_and_the_oracle():
    cases = [((2, 8, 2, 700, 900), True, 9001), ((1, 4, 4, 1536, 1536), False, 9002)]
    for (B, Hq, Hkv, Sq, Sk), causal, seed in cases:   # two different problems, back to back
        q, k, v = (t.cuda() for t in make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=seed))
        o_ref, lse_ref = _run(lib.attn_fwd, q, k, v, causal)
        for _ in range(2):                               # and each of them twice in a row
            o, lse = _run(lib.attn_fwd_noalloc, q, k, v, causal)
            assert _same_bits(o, lse, o_ref, lse_ref)
        _check_against_oracle(q, k, v, causal, o, lse)


def test_the_shared_work_counter_is_cleared_between_calls():
    """A problem with several work items per CTA leaves the scheduler's counter (word 0 of the
    static array) far above zero; the next call, on a problem with another grid size, would hand
    out no work at all (its outputs would keep their poison) if the entry point did not clear
    the counter on the stream first.  Large, small, large again: each result must carry the
    bits ``attn_fwd`` produces."""
    big = make_qkv(2, 16, 16, 2560, 2560, 128, seed=9003)      # 320 work items for at most 148 CTAs
    small = make_qkv(1, 2, 2, 300, 300, 128, seed=9004)        # 4 work items
    mid = make_qkv(1, 16, 4, 2048, 2048, 128, seed=9005)       # 256 work items, stages pair query heads
    for qkv, causal in ((big, True), (small, False), (big, False), (mid, True), (small, True)):
        q, k, v = (t.cuda() for t in qkv)
        o_ref, lse_ref = _run(lib.attn_fwd, q, k, v, causal)
        o, lse = _run(lib.attn_fwd_noalloc, q, k, v, causal)
        assert not torch.isnan(o).any() and not torch.isnan(lse).any()
        assert _same_bits(o, lse, o_ref, lse_ref)
    # the last large result also against the oracle, on sampled rows
    q, k, v = (t.cuda() for t in big)
    o, lse = _run(lib.attn_fwd_noalloc, q, k, v, True)
    _check_against_oracle(q, k, v, True, o, lse, rows=sample_rows(2, 16, 2560, 512, seed=9003))


def test_sizes_beyond_the_maximum_are_refused():
    # 2^20 + 1 query tiles: refused before anything touches the device; pointers are never read
    q = torch.empty((1, 128, 1, 128), dtype=torch.bfloat16, device="cuda")
    cdll = lib.load_library()
    rc = cdll.attn_fwd_noalloc(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr() + 16, None,
                               (1 << 20) + 1, 1, 1, 128, 128, 128, 0, SCALE, None)
    assert rc == 8 and lib.attn_status_str(rc) == "ATTN_ERR_TOO_LARGE"
    rc = cdll.attn_fwd_noalloc(None, q.data_ptr(), q.data_ptr(), q.data_ptr(), None,
                               1, 1, 1, 128, 128, 128, 0, SCALE, None)
    assert rc == 1
