"""Seeded synthetic workloads shaped like the paper's experiments.

This module only describes the five benchmark configurations and draws
their random inputs (Q/K/V tensors and key-padding masks).  It contains
none of the method's arithmetic: no attention graph, no softmax, no
random-block selection.  Both the CUDA library's tests and the CPU oracle's
tests take their inputs from here so that they see identical numbers.

Shapes follow the paper's hyper-parameter tables (App. E, Tab. "MLM
hyperparameters": 12 heads x 64 for base, 16 heads x 64 for large,
sequence length 4096, block size 64, 2 global / 3 window / 3 random blocks).
The tensors stand in for the projected queries, keys and values of an
encoder layer on MLM / QA batches: i.i.d. Gaussians with scale 1/sqrt(D)
give scores distributed like N(0, 1), a non-degenerate softmax.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str          # "fp32" | "bf16"
    B: int
    H: int
    N: int              # total tokens per sequence (ETC: includes the prepended global tokens)
    D: int
    b: int              # block size in tokens
    w: int              # window width in blocks (odd)
    g: int              # number of global blocks
    r: int              # random blocks per (head, query block)
    mode: int           # 0 = ITC (existing first/last blocks are global), 1 = ETC (first g blocks)
    seed: int
    sigma: float = 1.0  # std-dev of the Gaussian Q/K/V entries
    lengths: str = "full"   # "full" | "fixed:<L>" | "ragged:<lo>:<hi>"

    @property
    def nb(self) -> int:
        return self.N // self.b

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(self.D))


# The five configurations the library is measured and checked on.
WORKLOADS = {
    "c1_tiny_itc_fp32": Workload("c1_tiny_itc_fp32", "fp32", 1, 2, 512, 64, 64, 3, 2, 3, 0, seed=0),
    "c2_base_itc_bf16": Workload("c2_base_itc_bf16", "bf16", 8, 12, 4096, 64, 64, 3, 2, 3, 0, seed=1),
    "c3_etc_bf16": Workload("c3_etc_bf16", "bf16", 8, 12, 4096 + 128, 64, 64, 3, 2, 0, 1, seed=2),
    "c4_long_itc_bf16": Workload("c4_long_itc_bf16", "bf16", 1, 12, 16384, 64, 64, 3, 2, 3, 0, seed=3,
                                 sigma=0.5, lengths="fixed:13000"),
    "c5_large_ragged_bf16": Workload("c5_large_ragged_bf16", "bf16", 16, 16, 4096, 64, 64, 3, 2, 3, 0,
                                     seed=4, lengths="ragged:1024:4096"),
}
ORDER = list(WORKLOADS)


def torch_dtype(name: str) -> torch.dtype:
    return {"fp32": torch.float32, "bf16": torch.bfloat16}[name]


def valid_lengths(wl: Workload) -> Optional[np.ndarray]:
    """Per-sequence valid lengths (int64[B]) or None when nothing is padded."""
    if wl.lengths == "full":
        return None
    kind, *args = wl.lengths.split(":")
    if kind == "fixed":
        return np.full(wl.B, int(args[0]), dtype=np.int64)
    if kind == "ragged":
        lo, hi = int(args[0]), int(args[1])
        gen = torch.Generator(device="cpu").manual_seed(wl.seed + 1)
        raw = torch.randint(lo, hi + 1, (wl.B,), generator=gen).numpy().astype(np.int64)
        return ((raw + wl.b - 1) // wl.b) * wl.b      # rounded up to whole blocks
    raise ValueError(wl.lengths)


def key_padding_mask(wl: Workload) -> Optional[torch.Tensor]:
    """uint8[B, N], 1 = valid token, 0 = padding (tail of each sequence); None if unpadded."""
    lens = valid_lengths(wl)
    if lens is None:
        return None
    pos = np.arange(wl.N, dtype=np.int64)[None, :]
    return torch.from_numpy((pos < lens[:, None]).astype(np.uint8))


def make_qkv(wl: Workload, batch_limit: Optional[int] = None):
    """Draw Q, K, V of shape [B, H, N, D] on the CPU, in the workload's dtype.

    One CPU generator seeded with the workload's seed, drawn in the order
    q, k, v in fp32 and then cast, so the values are the same on every
    machine.  `batch_limit` draws only the first few batch elements (the
    draws for different batch elements are independent streams keyed by
    (seed, tensor, batch) so a prefix equals the full draw's prefix).
    """
    B = wl.B if batch_limit is None else min(wl.B, batch_limit)
    out = []
    for t in range(3):
        parts = []
        for bi in range(B):
            gen = torch.Generator(device="cpu").manual_seed((wl.seed * 3 + t) * 100003 + bi)
            x = torch.randn((wl.H, wl.N, wl.D), generator=gen, dtype=torch.float32)
            if wl.sigma != 1.0:
                x = x * wl.sigma
            parts.append(x.to(torch_dtype(wl.dtype)))
        out.append(torch.stack(parts, 0).contiguous())
    return tuple(out)
