"""A/B measurements of the kernel's design switches, in the shape of the paper's Table 1
(Section 5: geometric-mean throughput change, non-causal and causal, over the benchmark
sequence lengths).

    python -m paper_2603_24517_b200.ablation [--seqlens 4096 8192 16384 32768] [--launches 20]

Every switch is an ``attn_set_option`` value; each variant is timed interleaved with the default
(default, variant, default, variant, ...) so that clock drift under the power cap cancels.
Prints one JSON line per switch.

    python -m paper_2603_24517_b200.ablation --register-splits 192/80/48 184/88/56 184/72/72 176/80/80

The register split between the warp roles (Section 5.3 of the paper; softmax / correction / other
warps there, softmax / epilogue / MMA-and-loader warps here) is a build-time constant, so each
split is compiled into a library of its own in a scratch directory (``build.build_variant``), loaded
beside the in-tree one, timed interleaved with it in the same way, compared with it bit for bit
(the arithmetic does not depend on the split) and run through the small-case oracle parity tests
(a pytest child process with ``ATTN_B200_LIB`` pointing at the variant).  One JSON line per split,
with the spill bytes ptxas reports.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import math
import os
import subprocess
import sys
import tempfile

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


def load_variant(path):
    """A second build of the library, loaded beside the in-tree one: only attn_fwd is bound."""
    cdll = ctypes.CDLL(path)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    cdll.attn_fwd.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, cf, vp]
    cdll.attn_fwd.restype = ci
    return cdll


def variant_fwd(cdll, tensors, w):
    q, k, v, o, lse = tensors
    st = cdll.attn_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(), w.B, w.Hq, w.Hkv,
                       w.Sq, w.Sk, w.D, int(w.causal), w.scale, torch.cuda.current_stream().cuda_stream)
    if st != 0:
        raise RuntimeError(f"variant attn_fwd returned {st}")


def time_variant_ms(cdll, tensors, w, launches):
    for _ in range(3):
        variant_fwd(cdll, tensors, w)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(launches):
        variant_fwd(cdll, tensors, w)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / launches


def make_tensors(w):
    g = torch.Generator(device="cuda")
    g.manual_seed(w.seed)
    q = torch.randn((w.B, w.Sq, w.Hq, w.D), device="cuda", generator=g).to(torch.bfloat16)
    k = torch.randn((w.B, w.Sk, w.Hkv, w.D), device="cuda", generator=g).to(torch.bfloat16)
    v = torch.randn((w.B, w.Sk, w.Hkv, w.D), device="cuda", generator=g).to(torch.bfloat16)
    o = torch.empty_like(q)
    lse = torch.empty((w.B, w.Hq, w.Sq), device="cuda", dtype=torch.float32)
    return q, k, v, o, lse


def register_splits(args):
    """One JSON line per register split: geomean speed-up over the in-tree build (192/64/64),
    causal and non-causal, spill bytes, bitwise agreement with it and the oracle parity run."""
    from paper_2603_24517_b200 import build as lib_build
    lib.load_library()
    set_options({})
    W = all_workloads()
    scratch = tempfile.mkdtemp(prefix="attn_regsplit_")
    for split in args.register_splits:
        a, b, c = (int(x) for x in split.split("/"))
        if 8 * a + 4 * b + 4 * c > 2048 or min(a, b, c) < 24 or any(x % 8 for x in (a, b, c)):
            raise SystemExit(f"{split}: 8 a + 4 b + 4 c must not exceed 2048, multiples of 8, at least 24 each")
        path = os.path.join(scratch, f"libattn_b200_{a}_{b}_{c}.so")
        info = lib_build.build_variant(path, [f"-DATTN_REGS_SOFTMAX={a}", f"-DATTN_REGS_EPILOGUE={b}",
                                              f"-DATTN_REGS_OTHER={c}"])
        cdll = load_variant(path)
        out = {"register_split": split, "baseline_split": "192/64/64",
               "spill_store_bytes": info["spill_store_bytes"], "spill_load_bytes": info["spill_load_bytes"]}
        same_bits = True
        for mask in ("noncausal", "causal"):
            ratios = []
            for S in args.seqlens:
                w = W[f"mha_{mask}_s{S}"]
                t = make_tensors(w)
                t_def, t_var = [], []
                for _ in range(args.rounds):
                    t_def.append(time_ms(t, w, args.launches))
                    t_var.append(time_variant_ms(cdll, t, w, args.launches))
                ratios.append(min(t_def) / min(t_var))  # > 1: the variant is faster
                # same arithmetic per row whatever the split: the outputs must agree bit for bit
                o_var, l_var = t[3].clone(), t[4].clone()
                lib.attn_fwd(*t, w.causal, w.scale)
                torch.cuda.synchronize()
                same_bits &= bool(torch.equal(o_var.view(torch.int16), t[3].view(torch.int16)) and
                                  torch.equal(l_var.view(torch.int32), t[4].view(torch.int32)))
            geo = math.exp(sum(math.log(r) for r in ratios) / len(ratios))
            out[mask] = {"geomean_speedup_of_variant": round(geo, 4),
                         "per_seqlen": {str(S): round(r, 4) for S, r in zip(args.seqlens, ratios)}}
        out["bitwise_equal_to_baseline"] = same_bits
        if not args.no_parity_tests:
            res = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"),
                                  "-q", "-x", "-k", "small_cases_match_oracle_everywhere and dual_stage"],
                                 env=dict(os.environ, ATTN_B200_LIB=path), capture_output=True, text=True, cwd=ROOT)
            tail = (res.stdout.strip().splitlines() or [""])[-1]
            out["oracle_parity_small_cases"] = {"returncode": res.returncode, "summary": tail}
        print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--seqlens", type=int, nargs="+", default=[4096, 8192, 16384, 32768])
    ap.add_argument("--launches", type=int, default=20)
    ap.add_argument("--rounds", type=int, default=3)
    ap.add_argument("--register-splits", nargs="+", default=None, metavar="A/B/C",
                    help="registers per thread of the softmax / epilogue / other warps; builds and times each split")
    ap.add_argument("--no-parity-tests", action="store_true")
    args = ap.parse_args()
    if args.register_splits:
        register_splits(args)
        return
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
