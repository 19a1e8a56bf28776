"""A/B measurements of the kernel's design switches, in the shape of the paper's Table 1
(Section 5: geometric-mean throughput change, non-causal and causal, over the benchmark
sequence lengths).

    python -m paper_2603_24517_b200.ablation [--seqlens 4096 8192 16384 32768] [--launches 20]

Every switch is an ``attn_set_option`` value; each variant is timed interleaved with the default
(default, variant, default, variant, ...) so that clock drift under the power cap cancels.
Prints one JSON line per switch.  The register split between the warp roles is a build-time
constant (``ATTN_REGS_SOFTMAX`` / ``ATTN_REGS_EPILOGUE`` / ``ATTN_REGS_OTHER``) and is not
covered here.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import paper_2603_24517_b200 as lib  # noqa: E402
from workloads import all_workloads  # noqa: E402

DEFAULTS = {"scheduler": 2, "kernel": 0, "rescale_threshold": 8, "split_p": 1, "overlap_epilogue": 1}
SWITCHES = [
    ("rescale whenever the row maximum moves (threshold 0 instead of 8)", {"rescale_threshold": 0}),
    ("P released in one piece instead of two halves", {"split_p": 0}),
    ("epilogue waits for both stages (no correction/MMA overlap)", {"overlap_epilogue": 0}),
    ("static round-robin tile scheduler instead of the work counter", {"scheduler": 1}),
    ("one CTA per work item (hardware block scheduler)", {"scheduler": 0}),
    ("triple score buffer kernel instead of dual query stage", {"kernel": 1}),
    ("CTA-pair kernel (cta_group::2, P through shared memory) instead of dual query stage", {"kernel": 2}),
    ("two softmax threads per row (sixteen softmax warps, no epilogue warps)", {"kernel": 3}),
]


def set_options(opts):
    for k, v in {**DEFAULTS, **opts}.items():
        lib.attn_set_option(k, v)


def time_ms(tensors, w, launches):
    q, k, v, o, lse = tensors
    for _ in range(3):
        lib.attn_fwd(q, k, v, o, lse, w.causal, w.scale)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(launches):
        lib.attn_fwd(q, k, v, o, lse, w.causal, w.scale)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / launches


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--seqlens", type=int, nargs="+", default=[4096, 8192, 16384, 32768])
    ap.add_argument("--launches", type=int, default=20)
    ap.add_argument("--rounds", type=int, default=3)
    args = ap.parse_args()
    lib.load_library()
    W = all_workloads()
    for label, opts in SWITCHES:
        out = {"switch": label, "options": opts}
        for mask in ("noncausal", "causal"):
            ratios = []
            for S in args.seqlens:
                w = W[f"mha_{mask}_s{S}"]
                g = torch.Generator(device="cuda")
                g.manual_seed(w.seed)
                q = torch.randn((w.B, w.Sq, w.Hq, w.D), device="cuda", generator=g).to(torch.bfloat16)
                k = torch.randn((w.B, w.Sk, w.Hkv, w.D), device="cuda", generator=g).to(torch.bfloat16)
                v = torch.randn((w.B, w.Sk, w.Hkv, w.D), device="cuda", generator=g).to(torch.bfloat16)
                o = torch.empty_like(q)
                lse = torch.empty((w.B, w.Hq, w.Sq), device="cuda", dtype=torch.float32)
                t_def, t_var = [], []
                for _ in range(args.rounds):
                    set_options({})
                    t_def.append(time_ms((q, k, v, o, lse), w, args.launches))
                    set_options(opts)
                    t_var.append(time_ms((q, k, v, o, lse), w, args.launches))
                ratios.append(min(t_def) / min(t_var))  # > 1: the variant is faster
            geo = math.exp(sum(math.log(r) for r in ratios) / len(ratios))
            out[mask] = {"geomean_speedup_of_variant": round(geo, 4),
                         "per_seqlen": {str(S): round(r, 4) for S, r in zip(args.seqlens, ratios)}}
        set_options({})
        st, code, detail = lib.attn_last_device_status()
        out["device_status"] = st
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
