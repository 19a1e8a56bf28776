"""Host logic of bench.py's scoring: the correctness gate (a result outside the tolerances or with
unwritten elements has no throughput) and the clock-normalised figure.  CPU only: the "GPU output"
here is the oracle's own result rounded to BF16, with mistakes planted in copies of it."""
import numpy as np
import torch

import bench
from oracle import attn_oracle as orc
from workloads import Workload, bf16_bits, make_workload_inputs


def _case():
    w = Workload("gate_case", 1, 2, 2, 256, 256, 128, True, 4242)
    q, k, v = make_workload_inputs(w)
    rate, dt, rows, o_ref, lse_ref, cores = bench.oracle_sample(w, q, k, v, 64, seed=3)
    assert rate > 0 and dt > 0 and cores >= 1 and rows.shape == (64, 3)
    o_full, lse_full = orc.attention_full(bf16_bits(q), bf16_bits(k), bf16_bits(v), w.causal, w.scale)
    o_host = torch.from_numpy(o_full).to(torch.bfloat16)            # [B, Sq, Hq, D], one BF16 rounding
    lse_host = torch.from_numpy(lse_full).to(torch.float32)         # [B, Hq, Sq]
    return w, rows, o_ref, lse_ref, o_host, lse_host


def test_gate_passes_a_correct_result_and_fails_planted_mistakes():
    w, rows, o_ref, lse_ref, o_host, lse_host = _case()
    good = bench.parity_of_rows(o_host, lse_host, rows, o_ref, lse_ref)
    assert good["ok"] and good["rows"] == 64 and good["max_dO"] <= 2e-2 and good["max_dLSE"] <= 1e-3
    b, h, i = (int(x) for x in rows[5])
    wrong = o_host.clone()
    wrong[b, i, h, 17] += 0.25                       # one element of one sampled row
    assert not bench.parity_of_rows(wrong, lse_host, rows, o_ref, lse_ref)["ok"]
    wrong_lse = lse_host.clone()
    wrong_lse[b, h, i] += 0.01                       # an LSE off by ten times the bound
    assert not bench.parity_of_rows(o_host, wrong_lse, rows, o_ref, lse_ref)["ok"]
    poisoned = o_host.clone()
    poisoned[b, i, h, 0] = float("nan")              # an element the launch never wrote
    res = bench.parity_of_rows(poisoned, lse_host, rows, o_ref, lse_ref)
    assert not res["ok"] and res["max_dO"] == float("inf")


def test_block_pairs_follow_the_flop_convention():
    w = Workload("x", 2, 16, 16, 16384, 16384, 128, False, 1)
    # 2 * 16 heads * 128 row tiles * 128 key blocks = 524288 blocks, 2 per pair, over 148 SMs
    assert abs(bench.block_pairs_per_sm(w, 148) - 524288 / 2 / 148) < 1e-9
    wc = Workload("xc", 2, 16, 16, 16384, 16384, 128, True, 1)
    assert abs(bench.block_pairs_per_sm(wc, 148) - 524288 / 4 / 148) < 1e-9
