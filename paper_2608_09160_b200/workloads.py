"""Seeded synthetic inputs for layerwise QK-RMSNorm.

This module only draws numbers and slices tensors.  It holds none of the
method's arithmetic (no squares, no means, no scaling by a statistic), so the
CPU oracle and the CUDA path can both be fed from it without sharing any code
that computes the result.

The five named workloads stand in for the projected Q/K activations of the
OLMo-family models the paper serves (Section IV-A); the cost of QK-Norm depends
only on (tokens, dq, dk, shards), which these shapes supply.

Recipe (identical for every workload):
  * one ``torch.Generator`` on the CPU, seeded with ``Workload.seed``;
  * fixed draw order: q, k, gamma_q, gamma_k, then the outlier permutations
    (q first, then k);
  * q, k ~ N(0, sigma) drawn in fp32; gamma ~ U(0.5, 1.5) drawn in fp32;
  * outlier channels (a fixed set per tensor, the same for all tokens) are
    multiplied by ``outlier_scale`` in fp32;
  * every tensor is rounded to bf16 exactly once.
Sharded inputs are column slices of the same full tensors copied into separate
contiguous buffers, so sharded and unsharded runs see identical values.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Tuple

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    tokens: int
    dq: int
    dk: int
    shards: Tuple[int, ...]       # shard counts this workload is run with (1 = unsharded)
    sigma: float = 1.0
    outlier_frac: float = 0.0     # fraction of channels scaled by outlier_scale
    outlier_scale: float = 20.0
    eps: float = 1e-6
    seed: int = 0
    in_place: bool = False
    note: str = ""

    @property
    def algorithmic_bytes(self) -> int:
        """Each element read once and written once, each gamma read once."""
        return 2 * self.tokens * (self.dq + self.dk) * 2 + (self.dq + self.dk) * 2


WORKLOADS: Dict[str, Workload] = {
    w.name: w
    for w in (
        Workload("C1", tokens=8, dq=4096, dk=4096, shards=(1,), seed=0,
                 note="decode tiny, unsharded"),
        Workload("C2", tokens=64, dq=4096, dk=4096, shards=(4, 1), seed=1,
                 note="decode batch, 4 logical shards (also run unsharded)"),
        Workload("C3", tokens=8192, dq=5120, dk=5120, shards=(1, 4), seed=2,
                 outlier_frac=0.01, note="prefill MHA, 1% outlier channels x20"),
        Workload("C4", tokens=16384, dq=5120, dk=1024, shards=(8,), seed=3,
                 note="prefill GQA, 8 logical shards"),
        Workload("C5", tokens=65536, dq=8192, dk=1024, shards=(8,), sigma=2.0, seed=4,
                 in_place=True, note="large prefill GQA, 8 logical shards, in place"),
    )
}


def scaled(w: Workload, tokens: int) -> Workload:
    """Same workload with a different token count (a bounded sample of it)."""
    return replace(w, tokens=int(tokens))


def _outlier_channels(d: int, frac: float, gen: torch.Generator) -> torch.Tensor:
    n = int(d * frac)
    perm = torch.randperm(d, generator=gen)
    return perm[:n]


def make_inputs(w: Workload) -> Dict[str, torch.Tensor]:
    """Returns CPU bf16 tensors q[T,dq], k[T,dk], gamma_q[dq], gamma_k[dk]."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(int(w.seed))
    q = torch.empty((w.tokens, w.dq), dtype=torch.float32).normal_(0.0, w.sigma, generator=gen)
    k = torch.empty((w.tokens, w.dk), dtype=torch.float32).normal_(0.0, w.sigma, generator=gen)
    gq = torch.empty((w.dq,), dtype=torch.float32).uniform_(0.5, 1.5, generator=gen)
    gk = torch.empty((w.dk,), dtype=torch.float32).uniform_(0.5, 1.5, generator=gen)
    if w.outlier_frac > 0.0:
        cq = _outlier_channels(w.dq, w.outlier_frac, gen)
        ck = _outlier_channels(w.dk, w.outlier_frac, gen)
        q[:, cq] *= w.outlier_scale
        k[:, ck] *= w.outlier_scale
    return {
        "q": q.to(torch.bfloat16),
        "k": k.to(torch.bfloat16),
        "gamma_q": gq.to(torch.bfloat16),
        "gamma_k": gk.to(torch.bfloat16),
    }


E4M3_MAX = 448.0


def make_inputs_e4m3(w: Workload) -> Dict[str, torch.Tensor]:
    """The same draws as make_inputs with the activations rounded ONCE from fp32 to FP8-E4M3
    (torch.float8_e4m3fn; fp32 values are clamped to the finite range first).  gamma stays bf16."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(int(w.seed))
    q = torch.empty((w.tokens, w.dq), dtype=torch.float32).normal_(0.0, w.sigma, generator=gen)
    k = torch.empty((w.tokens, w.dk), dtype=torch.float32).normal_(0.0, w.sigma, generator=gen)
    gq = torch.empty((w.dq,), dtype=torch.float32).uniform_(0.5, 1.5, generator=gen)
    gk = torch.empty((w.dk,), dtype=torch.float32).uniform_(0.5, 1.5, generator=gen)
    if w.outlier_frac > 0.0:
        cq = _outlier_channels(w.dq, w.outlier_frac, gen)
        ck = _outlier_channels(w.dk, w.outlier_frac, gen)
        q[:, cq] *= w.outlier_scale
        k[:, ck] *= w.outlier_scale
    return {
        "q": q.clamp_(-E4M3_MAX, E4M3_MAX).to(torch.float8_e4m3fn),
        "k": k.clamp_(-E4M3_MAX, E4M3_MAX).to(torch.float8_e4m3fn),
        "gamma_q": gq.to(torch.bfloat16),
        "gamma_k": gk.to(torch.bfloat16),
    }


def e4m3_bits(x: torch.Tensor):
    """Raw bit patterns of a CPU float8_e4m3fn tensor as a numpy uint8 array (a view)."""
    assert x.dtype == torch.float8_e4m3fn and x.device.type == "cpu"
    return x.contiguous().view(torch.uint8).numpy()


def shard_columns(x: torch.Tensor, num_shards: int) -> List[torch.Tensor]:
    """Equal contiguous column slices, slice s = columns [s*w, (s+1)*w), each in
    its own contiguous buffer (the layout a column-parallel projection leaves on
    each tensor-parallel rank)."""
    d = x.shape[-1]
    if num_shards < 1 or d % num_shards != 0:
        raise ValueError(f"width {d} is not divisible into {num_shards} equal shards")
    wdt = d // num_shards
    return [x[..., s * wdt:(s + 1) * wdt].clone(memory_format=torch.contiguous_format)
            for s in range(num_shards)]


def unshard_columns(parts: List[torch.Tensor]) -> torch.Tensor:
    """Inverse of shard_columns."""
    return torch.cat(parts, dim=-1).contiguous()


def bf16_bits(x: torch.Tensor):
    """Raw bf16 bit patterns of a CPU bf16 tensor as a numpy uint16 array (a view)."""
    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return x.contiguous().view(torch.int16).numpy().view("uint16")


def from_bf16_bits(bits) -> torch.Tensor:
    """numpy uint16 bit patterns -> CPU bf16 tensor (a view of the same memory)."""
    import numpy as np
    a = np.ascontiguousarray(bits, dtype=np.uint16)
    return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)


def small_parity_shapes() -> List[Workload]:
    """Shapes the oracle finishes in well under a second that still cross several
    tiles, ragged tails and every dispatch path (odd widths, single tokens,
    token counts that do not divide the grid, K absent or narrower than Q)."""
    shapes = [
        # name, T, dq, dk, shards
        ("s_t1", 1, 4096, 4096, (1,)),
        ("s_t3_odd", 3, 1000, 136, (1, 2)),
        ("s_tiny", 2, 8, 8, (1,)),
        ("s_24", 5, 24, 8, (1,)),
        ("s_unaligned", 7, 1001, 77, (1, 7)),
        ("s_149", 149, 5120, 1024, (1, 8)),
        ("s_2305", 2305, 640, 128, (1, 4)),
        ("s_8200", 33, 8200, 8200, (1, 5)),
        ("s_wide", 9, 16384, 2048, (1, 16)),
        ("s_max", 2, 65536, 8, (1,)),
        ("s_gqa8", 300, 8192, 1024, (8, 2)),
        ("s_mha4", 257, 5120, 5120, (4,)),
        ("s_konly", 17, 0, 1024, (1, 4)),
        ("s_qonly", 17, 2048, 0, (1, 4)),
        ("s_prefill_gqa", 2500, 5120, 1024, (8, 1)),     # warp-per-token kernel, several rows per warp
        ("s_prefill_odd", 2177, 1000, 136, (1,)),         # warp-per-token kernel, lanes with ragged chunk counts
        ("s_prefill_s3", 2150, 1536, 768, (3,)),          # shard count that leaves lanes idle
        ("s_prefill_konly", 2200, 0, 1024, (2,)),
        ("s_prefill_s16", 2140, 4096, 1024, (16,)),       # two lanes per shard, every lane issues a bulk copy
        ("s_prefill_s5", 2110, 2240, 560, (5, 7)),        # shard counts that are not powers of two
        ("s_prefill_wide", 2100, 16384, 4096, (1, 4)),    # rows too wide for one warp: the CTA-per-token TMA ring
        ("s_tile_gqa", 3001, 1024, 128, (1,)),           # short unsharded rows: several tokens per warp, ragged last tile
        ("s_tile_tiny", 2600, 64, 8, (1,)),              # 128-byte and 16-byte rows
        ("s_tile_konly", 2277, 0, 256, (1,)),
        ("s_tile_qonly", 2101, 1280, 0, (1,)),
        ("s_mid_gqa", 1500, 5120, 1024, (1, 8)),         # a thousand-odd tokens: still the register-resident rows kernel
        ("s_mid_mha", 1900, 2048, 2048, (2,)),
    ]
    out = []
    for i, (name, t, dq, dk, sh) in enumerate(shapes):
        out.append(Workload(name, tokens=t, dq=dq, dk=dk, shards=sh, seed=100 + i,
                            outlier_frac=0.01 if i % 3 == 0 else 0.0,
                            sigma=(0.25, 1.0, 3.0)[i % 3]))
    return out
