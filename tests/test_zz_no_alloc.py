"""The no-allocation entry point, through the C ABI.

Some callers of this library are not allowed to allocate device memory: a server that gave
all of HBM to its own pools at start-up, a latency-critical thread that must stay off the
driver's allocation lock, a runtime that bans library-side allocations.  For them
``attn_fwd_noalloc`` runs the same kernel with its scratch (tile-scheduler counter, status
words) in a fixed 256-byte array inside the library image instead of cudaMalloc'ed memory.
Every call shares that array and it keeps the previous call's contents, so this test calls the
entry point twice in a row and compares each result with ``attn_fwd``'s on the same inputs.

Collected last on purpose (file name), so that a run that stops at the first failure has
already run every other test.  Passes alone in a fresh process and after the other tests.
"""
import math

import numpy as np
import pytest
import torch

import paper_2603_24517_b200 as lib
from paper_2603_24517_b200 import build as lib_build
from workloads import bf16_bits, bits_to_float64, make_qkv

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


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    cases = [((2, 8, 2, 700, 900), True, 9001), ((1, 4, 4, 1536, 1536), False, 9002)]
    for (B, Hq, Hkv, Sq, Sk), causal, seed in cases:   # two different problems, back to back
        q, k, v = (t.cuda() for t in make_qkv(B, Hq, Hkv, Sq, Sk, 128, seed=seed))
        o_ref, lse_ref = _run(lib.attn_fwd, q, k, v, causal)
        for _ in range(2):                               # and each of them twice in a row
            o, lse = _run(lib.attn_fwd_noalloc, q, k, v, causal)
            d_o = np.abs(bits_to_float64(bf16_bits(o)) - bits_to_float64(bf16_bits(o_ref))).max()
            d_l = np.abs(lse.numpy().astype(np.float64) - lse_ref.numpy().astype(np.float64)).max()
            assert not np.isnan(d_o) and not np.isnan(d_l)
            assert d_o <= TOL_O and d_l <= TOL_LSE, (d_o, d_l)
    st, code, detail = lib.attn_last_device_status()
    assert (st, code) == (0, 0)


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
