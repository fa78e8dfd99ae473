"""Seeded synthetic workloads for the DiT spatiotemporal self-attention path.

This module only *describes* and *generates* inputs: shapes, value
distributions, key-padding masks and the sampled query rows that parity tests
look at.  It contains none of the method's arithmetic (no RoPE, no softmax, no
matmul) so that both the CPU oracle's callers and the CUDA path's callers can
use it without sharing any computation.

The five named configurations stand in for the paper's low-resolution and
high-resolution denoising stages (Section 3.1, cross-resolution two-stage
scheduler) and for the batched / packed variants a server sees.  The paper
measures on prompts and trained weights that are not available; the tensors
here are i.i.d. draws with the same shapes and layout: a flat
``(total_tokens, heads, head_dim)`` activation layout (Section 3.2, "Optimized
attention collectives") with every sequence packed prefix-first (Section 3.4,
"Safety rails and the exact prefix KV sink").
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class SeqSpec:
    """One packed sequence: ``text_len`` prefix tokens, then a T*H*W video grid."""

    text_len: int
    T: int
    H: int
    W: int

    @property
    def n_video(self) -> int:
        return self.T * self.H * self.W

    @property
    def n_tokens(self) -> int:
        return self.text_len + self.n_video


@dataclass(frozen=True)
class Workload:
    name: str
    seqs: Tuple[SeqSpec, ...]
    heads: int
    head_dim: int
    rope_dims: Tuple[int, int, int]
    theta: float = 10000.0
    seed: int = 0
    # value recipe
    k_scale: float = 1.0            # K <- k_scale * K (power of two: exact in bf16)
    v_dist: str = "normal"          # "normal" or "uniform" (-1, 1)
    # per-sequence number of *valid* prefix tokens (None = all valid); the
    # remaining prefix keys are masked out by the key-padding mask
    valid_text: Optional[Tuple[int, ...]] = None
    rows_per_head: int = 0          # 0 = compare every row; else sampled rows per (seq, head)
    note: str = ""

    @property
    def n_seqs(self) -> int:
        return len(self.seqs)

    @property
    def total_tokens(self) -> int:
        return sum(s.n_tokens for s in self.seqs)

    @property
    def cu_seqlens(self) -> List[int]:
        out = [0]
        for s in self.seqs:
            out.append(out[-1] + s.n_tokens)
        return out

    @property
    def has_mask(self) -> bool:
        return self.valid_text is not None

    def flops(self, valid_keys_only: bool = True) -> float:
        """4 * N_q * N_k * D * heads summed over sequences (QK^T and PV)."""
        total = 0.0
        for i, s in enumerate(self.seqs):
            nk = s.n_tokens
            if valid_keys_only and self.valid_text is not None:
                nk = s.n_tokens - (s.text_len - self.valid_text[i])
            total += 4.0 * s.n_tokens * nk * self.head_dim * self.heads
        return total

    def algorithmic_bytes(self) -> int:
        """Read Q, K, V once and write O once, bf16."""
        return 4 * self.total_tokens * self.heads * self.head_dim * 2


def _grid(text_len, T, H, W):
    return SeqSpec(text_len, T, H, W)


# The five configurations of the benchmark contract.
CONFIGS = {
    "tiny": Workload(
        name="tiny", seqs=(_grid(0, 4, 8, 8),), heads=4, head_dim=64,
        rope_dims=(16, 24, 24), seed=1001, note="correctness case, all rows compared"),
    "lowres": Workload(
        name="lowres", seqs=(_grid(256, 16, 30, 52),), heads=40, head_dim=128,
        rope_dims=(32, 48, 48), seed=1002, k_scale=0.5, rows_per_head=4096,
        note="low-resolution stage; K scaled by 0.5 to mimic post-QK-norm logits"),
    "highres": Workload(
        name="highres", seqs=(_grid(256, 31, 45, 80),), heads=40, head_dim=128,
        rope_dims=(32, 48, 48), seed=1003, rows_per_head=4096,
        note="high-resolution stage"),
    "cfg_batch": Workload(
        name="cfg_batch", seqs=(_grid(512, 31, 45, 80), _grid(512, 31, 45, 80)),
        heads=40, head_dim=128, rope_dims=(32, 48, 48), seed=1004,
        valid_text=(512, 77), rows_per_head=4096,
        note="classifier-free-guidance pair, prefix 512 / 77 padded to 512"),
    "varlen": Workload(
        name="varlen",
        seqs=(_grid(256, 8, 30, 52), _grid(256, 16, 30, 52),
              _grid(256, 16, 45, 80), _grid(256, 31, 45, 80)),
        heads=48, head_dim=128, rope_dims=(32, 48, 48), seed=1005,
        v_dist="uniform", rows_per_head=1024,
        note="four packed videos, block-diagonal attention; 1024 rows per (seq, head)"),
}
CONFIG_ORDER = ["tiny", "lowres", "highres", "cfg_batch", "varlen"]


def shrunk(name: str) -> Workload:
    """Scaled-down siblings of the big configurations.

    Same structure (prefix, ragged tails, mask, packing, value recipe) at sizes
    the fp64 oracle finishes in seconds with *all* rows compared, while still
    spanning several 128-row tiles and a ragged tail.
    """
    if name == "tiny":
        return CONFIGS["tiny"]
    if name == "lowres":       # 256 + 4*7*13 = 620 tokens: 4 full tiles + 108 tail
        return replace(CONFIGS["lowres"], name="lowres_small", seqs=(_grid(256, 4, 7, 13),),
                       heads=3, rows_per_head=0)
    if name == "highres":      # 256 + 5*9*20 = 1156 tokens: 9 tiles + 4 tail
        return replace(CONFIGS["highres"], name="highres_small", seqs=(_grid(256, 5, 9, 20),),
                       heads=3, rows_per_head=0)
    if name == "cfg_batch":    # 2 x (512 + 3*9*16 = 944): 7 tiles + 48 tail, mask 77..511 on seq 1
        return replace(CONFIGS["cfg_batch"], name="cfg_batch_small",
                       seqs=(_grid(512, 3, 9, 16), _grid(512, 3, 9, 16)), heads=2, rows_per_head=0)
    if name == "varlen":
        return replace(CONFIGS["varlen"], name="varlen_small",
                       seqs=(_grid(256, 1, 6, 10), _grid(256, 2, 6, 10),
                             _grid(256, 2, 9, 16), _grid(256, 4, 9, 16)),
                       heads=3, rows_per_head=0)
    raise KeyError(name)


@dataclass
class Inputs:
    q: torch.Tensor                 # [total, heads, D] bf16
    k: torch.Tensor
    v: torch.Tensor
    key_mask: Optional[torch.Tensor]  # [total] uint8, nonzero = attend; None = all valid


def make_key_mask(w: Workload, device="cpu") -> Optional[torch.Tensor]:
    """uint8 [total_tokens]; prefix keys at or beyond a sequence's valid text length are 0."""
    if w.valid_text is None:
        return None
    m = torch.ones(w.total_tokens, dtype=torch.uint8)
    cu = w.cu_seqlens
    for i, s in enumerate(w.seqs):
        m[cu[i] + w.valid_text[i]: cu[i] + s.text_len] = 0
    return m.to(device)


def make_inputs(w: Workload, device="cpu") -> Inputs:
    """Draw Q, K, V for a workload from its seed on ``device`` and round to bf16.

    Values at masked key positions are ordinary finite random numbers: the
    result must not depend on them.
    """
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed)
    shape = (w.total_tokens, w.heads, w.head_dim)

    def normal():
        # generated in fp32 in slabs to bound peak memory, rounded to bf16 (RNE)
        out = torch.empty(shape, dtype=torch.bfloat16, device=dev)
        step = max(1, (1 << 26) // (w.heads * w.head_dim))
        for a in range(0, shape[0], step):
            b = min(shape[0], a + step)
            out[a:b] = torch.randn((b - a,) + shape[1:], generator=g, device=dev,
                                   dtype=torch.float32).to(torch.bfloat16)
        return out

    def uniform():
        out = torch.empty(shape, dtype=torch.bfloat16, device=dev)
        step = max(1, (1 << 26) // (w.heads * w.head_dim))
        for a in range(0, shape[0], step):
            b = min(shape[0], a + step)
            u = torch.rand((b - a,) + shape[1:], generator=g, device=dev, dtype=torch.float32)
            out[a:b] = (2.0 * u - 1.0).to(torch.bfloat16)
        return out

    q = normal()
    k = normal()
    if w.k_scale != 1.0:
        k.mul_(w.k_scale)
    v = uniform() if w.v_dist == "uniform" else normal()
    return Inputs(q=q, k=k, v=v, key_mask=make_key_mask(w, dev))


def sample_rows(w: Workload, seq: int, head: int, count: Optional[int] = None) -> np.ndarray:
    """Sorted distinct local query rows of one (sequence, head) to compare.

    Counter-based: depends only on (workload seed, seq, head).  Always contains
    the rows where indexing mistakes show first: 0, the last prefix row, the
    first video row, the last row, and the first and last row of the ragged
    tail tile (128-row tiles).
    """
    s = w.seqs[seq]
    n = s.n_tokens
    count = w.rows_per_head if count is None else count
    if count <= 0 or count >= n:
        return np.arange(n, dtype=np.int64)
    forced = {0, n - 1, (n - 1) // 128 * 128, max(0, (n - 1) // 128 * 128 - 1)}
    if s.text_len > 0:
        forced |= {s.text_len - 1, min(n - 1, s.text_len)}
    rng = np.random.default_rng([w.seed, seq, head, 0x5EED])
    extra = rng.choice(n, size=min(n, count), replace=False)
    rows = list(forced)
    seen = set(forced)
    for r in extra:
        if len(rows) >= count:
            break
        r = int(r)
        if r not in seen:
            seen.add(r)
            rows.append(r)
    return np.sort(np.asarray(rows, dtype=np.int64))
