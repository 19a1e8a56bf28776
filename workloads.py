"""Seeded synthetic attention workloads (inputs only -- none of the method's arithmetic).

The paper times its kernels on random BF16 tensors with head dimension 128, a fixed
total of 32768 tokens and sequence lengths 4096..32768, 16 heads for multi-head
attention and 32 query / 8 or 4 key-value heads for grouped-query attention
(Section 4.1, "Benchmark Configurations").  The workloads below have those shapes;
values are iid N(0,1) drawn in fp32 from a seeded generator and rounded to BF16.
They stand in for the paper's benchmark tensors.

Both the CPU oracle's tests and the CUDA library's tests and benchmark draw their
inputs from here, so the two sides always see the same BF16 bits.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch

HEAD_DIM = 128


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    Hq: int
    Hkv: int
    Sq: int
    Sk: int
    D: int = HEAD_DIM
    causal: bool = False
    seed: int = 0
    q_gain: float = 1.0  # Q is multiplied by this power of two before rounding (exact in BF16)

    @property
    def scale(self) -> float:
        """1/sqrt(D) as the fp32 value every caller passes."""
        return float(np.float32(1.0 / math.sqrt(self.D)))

    @property
    def flops(self) -> float:
        """4*B*Hq*Sq*Sk*D, halved when causal (the convention of the paper's TFLOPS figures)."""
        f = 4.0 * self.B * self.Hq * self.Sq * self.Sk * self.D
        return f / 2 if self.causal else f

    @property
    def algorithmic_bytes(self) -> int:
        """Read Q, K, V once; write O (BF16) and LSE (fp32) once."""
        q = self.B * self.Sq * self.Hq * self.D * 2
        kv = 2 * self.B * self.Sk * self.Hkv * self.D * 2
        return q + kv + q + self.B * self.Hq * self.Sq * 4


def _sweep(prefix, Hq, Hkv, causal, seqs, seed0):
    out = []
    for S in seqs:
        out.append(Workload(f"{prefix}_s{S}", 32768 // S, Hq, Hkv, S, S, HEAD_DIM, causal,
                            seed0 + int(math.log2(S))))
    return out


def all_workloads() -> dict[str, Workload]:
    w = [Workload("tiny_mha", 1, 2, 2, 512, 512, HEAD_DIM, False, 1001)]
    w += _sweep("mha_noncausal", 16, 16, False, (1024, 4096, 8192, 16384, 32768), 2000)
    w += _sweep("mha_causal", 16, 16, True, (1024, 4096, 8192, 16384, 32768), 3000)
    w += _sweep("gqa4_noncausal", 32, 8, False, (4096, 8192, 16384, 32768), 4000)
    w += _sweep("gqa4_causal", 32, 8, True, (4096, 8192, 16384, 32768), 4100)
    w += _sweep("gqa8_noncausal", 32, 4, False, (4096, 8192, 16384, 32768), 4200)
    w += _sweep("gqa8_causal", 32, 4, True, (4096, 8192, 16384, 32768), 4300)
    w.append(Workload("long_causal_peaked", 1, 16, 16, 65536, 65536, HEAD_DIM, True, 5001, q_gain=4.0))
    return {x.name: x for x in w}


def make_qkv(B, Hq, Hkv, Sq, Sk, D, seed, q_gain=1.0):
    """Q [B,Sq,Hq,D], K, V [B,Sk,Hkv,D] as CPU torch.bfloat16 tensors, iid N(0,1)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    q = torch.randn((B, Sq, Hq, D), generator=g, dtype=torch.float32)
    if q_gain != 1.0:
        q *= q_gain
    q = q.to(torch.bfloat16)
    k = torch.randn((B, Sk, Hkv, D), generator=g, dtype=torch.float32).to(torch.bfloat16)
    v = torch.randn((B, Sk, Hkv, D), generator=g, dtype=torch.float32).to(torch.bfloat16)
    return q, k, v


def make_workload_inputs(w: Workload):
    return make_qkv(w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.D, w.seed, w.q_gain)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The BF16 bit patterns of a CPU bfloat16 tensor as a numpy uint16 array (no copy)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_float64(bits: np.ndarray) -> np.ndarray:
    """Widen BF16 bit patterns (uint16) to float64 exactly."""
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def sample_rows(B, Hq, Sq, n_rows, seed, tile=128):
    """A seeded set of (b, hq, i) query rows for spot checks against the oracle:
    tile-edge rows of every (b, hq), one row in every `tile`-row block of one head,
    the rest uniform.  int32 [n, 3], unique, sorted."""
    rng = np.random.default_rng(seed)
    rows = set()
    edge = [0, 1, tile - 1, tile, tile + 1, 2 * tile - 1, 2 * tile, Sq - tile - 1, Sq - tile, Sq - 1]
    edge = sorted({i for i in edge if 0 <= i < Sq})
    for b in range(B):
        for h in range(Hq):
            for i in edge:
                rows.add((b, h, i))
    for t in range((Sq + tile - 1) // tile):
        lo, hi = t * tile, min(Sq, (t + 1) * tile)
        rows.add((B - 1, Hq - 1, int(rng.integers(lo, hi))))
    target = min(max(n_rows, len(rows)), B * Hq * Sq)
    while len(rows) < target:
        rows.add((int(rng.integers(B)), int(rng.integers(Hq)), int(rng.integers(Sq))))
    return np.array(sorted(rows), dtype=np.int32)
