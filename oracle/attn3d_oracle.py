"""fp64 CPU oracle for 3D-RoPE joint self-attention.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition the CUDA path is checked against.  It
is never on the product path: only tests, the smoke check and the benchmark's
CPU-baseline leg may import it.  It shares no code, tables or constants with
the CUDA sources and imports nothing from the package.

What it computes (the attention that Section 3.2 of the paper calls "SDPA"
and times at 341 ms per denoising step, together with the rotary embedding of
fusion group (2) in Section 3.5, on the prefix-first packed sequence of
Section 3.4):

  O0  widen the inputs to fp64 exactly;
  O1  a packed tensor holds one or more sequences back to back; attention is
      block-diagonal over sequences;
  O2  local token i of a sequence with prefix length L and grid (T, H, W) has
      no position if i < L, else p = i - L, t = p // (H*W), h = (p // W) % H,
      w = p % W   (t slowest, w fastest);
  O3  rotary embedding, per axis a in (T, H, W) with width d_a starting at
      head-dim offset o_a = (0, d_T, d_T + d_H): for j < d_a/2,
      omega = theta ** (-2j/d_a), phi = pos_a * omega and the ADJACENT pair
      (x[o_a+2j], x[o_a+2j+1]) is rotated by phi.  Head dims beyond
      d_T+d_H+d_W pass through.  Prefix tokens and V are never rotated;
  O3' optional QK normalisation before O3 (fusion group (2) of Section 3.5): RMS norm over head_dim
      per (token, head) with a learned gain vector, see qk_rms_norm;
  O4  s_ij = <q~_i, k~_j> / sqrt(head_dim) for keys j of the same sequence
      whose key-padding mask is nonzero;
  O5  two-pass softmax in fp64: m_i = max_j s_ij, e_ij = exp(s_ij - m_i),
      o_i = sum_j e_ij v_j / sum_j e_ij.  A row with no valid key returns 0;
  O6  fp64 rows are returned; nothing is rounded to bf16 anywhere.

The convention choices (adjacent pairs, per-axis frequencies, 0-based integer
positions, axis order T/H/W from head-dim 0 up, scale by full head_dim) are
definitions the paper does not print; they are fixed by the benchmark
contract's configuration text and listed with their reasons in the design
notes.  Matrix products use the library matmul as a step; there is no tiling,
online rescaling or fusion.

Parity pins for every function here are in tests/test_oracle_pins.py
(closed forms, invariants, brute force, library special case).  Nothing in
this file is "parity unpinned".
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import torch

F64 = torch.float64


def widen(x: torch.Tensor) -> torch.Tensor:
    """O0: exact widening of bf16/fp16/fp32 values to fp64 on the CPU."""
    return x.detach().to("cpu").to(F64)


def token_positions(text_len: int, T: int, H: int, W: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """O2: integer (t, h, w) of every local token and whether it has one.

    Returns (pos [N, 3] int64, has_pos [N] bool); prefix rows get pos 0 and
    has_pos False.
    """
    n = text_len + T * H * W
    pos = torch.zeros(n, 3, dtype=torch.int64)
    has = torch.zeros(n, dtype=torch.bool)
    p = torch.arange(T * H * W, dtype=torch.int64)
    pos[text_len:, 0] = p // (H * W)
    pos[text_len:, 1] = (p // W) % H
    pos[text_len:, 2] = p % W
    has[text_len:] = True
    return pos, has


def rope_angles(pos_a: torch.Tensor, d_a: int, theta: float) -> torch.Tensor:
    """O3: phi[n, j] = pos_a[n] * theta ** (-2j / d_a) for j < d_a / 2, in fp64."""
    j = torch.arange(d_a // 2, dtype=F64)
    omega = torch.exp(-(2.0 * j / d_a) * math.log(theta))
    return pos_a.to(F64)[:, None] * omega[None, :]


def rope_rotate(x: torch.Tensor, pos: torch.Tensor, has_pos: torch.Tensor,
                rope_dims: Sequence[int], theta: float,
                origin: Sequence[int] = (0, 0, 0), pairing: str = "adjacent") -> torch.Tensor:
    """O3: rotate x [N, ..., D] (fp64) token by token; returns a new tensor.

    ``origin`` is added to every position that exists (used only by the
    shift-invariance pin).  ``pairing`` is "adjacent" (the definition used
    here) or "half" (pairs (j, j + d_a/2), kept so the other common convention
    can be compared in one line).
    """
    assert x.dtype == F64
    out = x.clone()
    D = x.shape[-1]
    assert sum(rope_dims) <= D and all(d % 2 == 0 and d >= 0 for d in rope_dims)
    bshape = (x.shape[0],) + (1,) * (x.dim() - 2)
    off = 0
    for a, d_a in enumerate(rope_dims):
        if d_a > 0:
            phi = rope_angles(pos[:, a] + int(origin[a]), d_a, theta)      # [N, d_a/2]
            phi = torch.where(has_pos[:, None], phi, torch.zeros_like(phi))  # no position: identity
            c = torch.cos(phi).reshape(bshape + (d_a // 2,))
            s = torch.sin(phi).reshape(bshape + (d_a // 2,))
            if pairing == "adjacent":
                xe = x[..., off: off + d_a: 2]
                xo = x[..., off + 1: off + d_a: 2]
                out[..., off: off + d_a: 2] = xe * c - xo * s
                out[..., off + 1: off + d_a: 2] = xe * s + xo * c
            elif pairing == "half":
                xe = x[..., off: off + d_a // 2]
                xo = x[..., off + d_a // 2: off + d_a]
                out[..., off: off + d_a // 2] = xe * c - xo * s
                out[..., off + d_a // 2: off + d_a] = xe * s + xo * c
            else:
                raise ValueError(pairing)
        off += d_a
    return out


def qk_rms_norm(x: torch.Tensor, gain: torch.Tensor, eps: float) -> torch.Tensor:
    """QK normalisation, the first half of fusion group (2) in Section 3.5 ("QK normalization with partial
    RoPE"): RMS norm over head_dim of every (token, head) row, times a learned gain of length head_dim.

        y = x / sqrt(mean_d(x_d^2) + eps) * gain            (fp64, nothing rounded)

    The paper prints no formula; per-head normalisation over head_dim with a gain shared by all heads is
    the reading taken here (it is the common "QK-norm" of video DiTs).  x: [..., D] fp64, gain: [D].
    """
    assert x.dtype == F64
    ms = (x * x).mean(dim=-1, keepdim=True)
    return x / torch.sqrt(ms + eps) * gain.to(F64)


def attention_rows(q_rot: torch.Tensor, k_rot: torch.Tensor, v: torch.Tensor,
                   valid: Optional[torch.Tensor], head_dim: int,
                   row_chunk: Optional[int] = None) -> torch.Tensor:
    """O4-O5 for one (sequence, head): q_rot [R, D], k_rot [N, D], v [N, Dv] -> [R, Dv].

    ``valid`` is a bool [N] key mask or None.  Query rows are independent, so
    they are processed in chunks only to bound memory.
    """
    R, N = q_rot.shape[0], k_rot.shape[0]
    out = torch.zeros(R, v.shape[1], dtype=F64)
    if N == 0 or (valid is not None and not bool(valid.any())):
        return out                                           # no valid key: zeros
    if row_chunk is None:
        row_chunk = max(1, min(R, (1 << 27) // max(N, 1)))
    scale = 1.0 / math.sqrt(head_dim)
    kt = k_rot.t().contiguous()
    s = torch.empty(min(row_chunk, R), N, dtype=F64)
    for a in range(0, R, row_chunk):
        b = min(R, a + row_chunk)
        sc = s[: b - a]
        torch.matmul(q_rot[a:b], kt, out=sc)                 # O4 scores
        sc.mul_(scale)
        if valid is not None:
            sc.masked_fill_(~valid[None, :], float("-inf"))
        m = sc.max(dim=1, keepdim=True).values               # O5 first pass
        sc.sub_(m).exp_()                                    # e_ij (masked keys: exp(-inf) = 0)
        l = sc.sum(dim=1, keepdim=True)
        out[a:b] = torch.matmul(sc, v) / l
    return out


def attn3d_oracle_pos(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                      cu_seqlens: Sequence[int],
                      pos: torch.Tensor, has_pos: torch.Tensor,
                      rope_dims: Sequence[int], theta: float,
                      key_mask: Optional[torch.Tensor] = None,
                      select: Optional[List[Tuple[int, int, torch.Tensor]]] = None,
                      origin: Sequence[int] = (0, 0, 0), pairing: str = "adjacent",
                      q_gain: Optional[torch.Tensor] = None, k_gain: Optional[torch.Tensor] = None,
                      norm_eps: float = 1e-6):
    """Internal entry with explicit per-token positions.

    q, k, v: [total, heads, D]; pos [total, 3] int64; has_pos [total] bool;
    key_mask [total] (nonzero = attend) or None.

    ``select`` is a list of (seq, head, local_rows LongTensor); the result is a
    list of fp64 [len(rows), D] tensors in the same order.  With select=None
    every row is computed and a dense fp64 [total, heads, D] tensor returned.
    """
    total, heads, D = q.shape
    assert k.shape == q.shape and v.shape[:2] == q.shape[:2]
    dense = select is None
    if dense:
        select = [(s, h, None) for s in range(len(cu_seqlens) - 1) for h in range(heads)]
        out_dense = torch.zeros(total, heads, v.shape[2], dtype=F64)
    results = []
    for (s, h, rows) in select:
        a, b = int(cu_seqlens[s]), int(cu_seqlens[s + 1])
        kh = widen(k[a:b, h, :])
        vh = widen(v[a:b, h, :])
        if k_gain is not None:
            kh = qk_rms_norm(kh, widen(k_gain), norm_eps)          # normalise, then rotate (Section 3.5 (2))
        k_rot = rope_rotate(kh, pos[a:b], has_pos[a:b], rope_dims, theta, origin, pairing)
        if rows is None:
            rows_t = torch.arange(b - a, dtype=torch.int64)
        else:
            rows_t = torch.as_tensor(rows, dtype=torch.int64)
        qh = widen(q[a:b, h, :][rows_t])
        if q_gain is not None:
            qh = qk_rms_norm(qh, widen(q_gain), norm_eps)
        q_rot = rope_rotate(qh, pos[a:b][rows_t], has_pos[a:b][rows_t], rope_dims, theta, origin, pairing)
        valid = None if key_mask is None else (key_mask[a:b].to("cpu") != 0)
        o = attention_rows(q_rot, k_rot, vh, valid, D)
        if dense:
            out_dense[a:b, h, :] = o
        else:
            results.append(o)
    return out_dense if dense else results


def layout_positions(seqs: Sequence[Tuple[int, int, int, int]]):
    """O1-O2 for a packed batch: seqs = [(text_len, T, H, W), ...] ->
    (cu_seqlens list, pos [total, 3], has_pos [total])."""
    cu = [0]
    ps, hs = [], []
    for (L, T, H, W) in seqs:
        p, hp = token_positions(L, T, H, W)
        ps.append(p)
        hs.append(hp)
        cu.append(cu[-1] + p.shape[0])
    return cu, torch.cat(ps, 0), torch.cat(hs, 0)


def attn3d_oracle(q, k, v, seqs: Sequence[Tuple[int, int, int, int]],
                  rope_dims: Sequence[int], theta: float = 10000.0,
                  key_mask: Optional[torch.Tensor] = None,
                  select: Optional[List[Tuple[int, int, torch.Tensor]]] = None,
                  q_gain: Optional[torch.Tensor] = None, k_gain: Optional[torch.Tensor] = None,
                  norm_eps: float = 1e-6):
    """Public entry: q, k, v [total, heads, D] packed prefix-first per sequence.

    A batch of B equal sequences is the packed case with B identical entries
    in ``seqs`` (batch b starts at token b*N).  With q_gain / k_gain given, Q and K are RMS-normalised
    over head_dim (qk_rms_norm) before the rotary embedding.
    """
    cu, pos, has = layout_positions(seqs)
    assert cu[-1] == q.shape[0], "token count does not match the sequence list"
    return attn3d_oracle_pos(q, k, v, cu, pos, has, rope_dims, theta, key_mask, select,
                             q_gain=q_gain, k_gain=k_gain, norm_eps=norm_eps)


def rope_oracle(x, seqs: Sequence[Tuple[int, int, int, int]], rope_dims: Sequence[int],
                theta: float = 10000.0, gain: Optional[torch.Tensor] = None, norm_eps: float = 1e-6) -> torch.Tensor:
    """O0-O3 only: the (optionally RMS-normalised, then) rotated tensor in fp64, [total, heads, D]."""
    _, pos, has = layout_positions(seqs)
    xw = widen(x)
    if gain is not None:
        xw = qk_rms_norm(xw, widen(gain), norm_eps)
    return rope_rotate(xw, pos, has, rope_dims, theta)


# ---------------------------------------------------------------------------------------------
# Block-sparse variant: the per-step dynamic sparsity of Section 3.4 ("Sparse Attention").
# This is an approximation of dense attention, so the oracle follows the algorithm step by step.
# Steps and notation (the paper gives the rule, not the block statistic nor the block sizes; readings are
# marked).  Nothing is rounded anywhere: the statistic is taken in fp64 on the un-rounded rotated operands.
#   B1  query blocks of qblk tokens, KV blocks of kblk tokens, per sequence and head; both sizes are arguments
#       of every function below                                                                    [reading]
#   B2  block-level score  b_ij = < mean of q~ over block i , mean of k~ over block j > / sqrt(D)    [reading:
#       mean-pooled pre-softmax logits; by bilinearity this is the mean of the block's logits]
#   B3  per query block: mu_i, sigma_i = mean and (population) standard deviation of b_ij over all KV
#       blocks j; KV block j is selected iff b_ij > mu_i + tau * sigma_i                      [Section 3.4]
#   B4  safety rails [Section 3.4]: KV blocks holding any prefix token are always selected (exact prefix
#       sink); query blocks holding any prefix token attend densely.  The block with the largest score
#       is always kept, so no query block is left without keys.                                [last: reading]
#   B5  attention as O4-O5 restricted to the keys of the selected blocks (and to valid keys).
# ---------------------------------------------------------------------------------------------
def block_scores(q_rot: torch.Tensor, k_rot: torch.Tensor, head_dim: int, qblk: int, kblk: int) -> torch.Tensor:
    """B2 for one (sequence, head): q_rot, k_rot [N, D] fp64 -> [ceil(N/qblk), ceil(N/kblk)]."""
    n = q_rot.shape[0]
    nq, nk = (n + qblk - 1) // qblk, (n + kblk - 1) // kblk
    qbar = torch.stack([q_rot[i * qblk: min(n, (i + 1) * qblk)].mean(0) for i in range(nq)])
    kbar = torch.stack([k_rot[j * kblk: min(n, (j + 1) * kblk)].mean(0) for j in range(nk)])
    return (qbar @ kbar.t()) / math.sqrt(head_dim)


def block_select(scores: torch.Tensor, tau: float, text_len: int, qblk: int, kblk: int) -> torch.Tensor:
    """B3-B4: bool [n_qblocks, n_kblocks], True = KV block attended."""
    mu = scores.mean(dim=1, keepdim=True)
    sigma = torch.sqrt(((scores - mu) ** 2).mean(dim=1, keepdim=True))
    sel = scores > mu + tau * sigma
    sel[torch.arange(scores.shape[0]), scores.argmax(dim=1)] = True
    if text_len > 0:
        sel[:, : (text_len + kblk - 1) // kblk] = True           # exact prefix KV sink
        sel[: (text_len + qblk - 1) // qblk, :] = True           # prefix queries stay dense
    return sel


def sparse_rows(q_rot: torch.Tensor, k_rot: torch.Tensor, v: torch.Tensor, sel: torch.Tensor,
                valid: Optional[torch.Tensor], rows: torch.Tensor, head_dim: int, qblk: int, kblk: int) -> torch.Tensor:
    """B5 for one (sequence, head) and the given local query rows: q_rot, k_rot [N, D], v [N, Dv] fp64,
    sel bool [n_qblocks, n_kblocks] -> fp64 [len(rows), Dv].  Rows of one query block share their key set."""
    n = k_rot.shape[0]
    rows = torch.as_tensor(rows, dtype=torch.int64)
    out = torch.zeros(rows.shape[0], v.shape[1], dtype=F64)
    blk = rows // qblk
    for i in torch.unique(blk).tolist():
        keys = sel[i].repeat_interleave(kblk)[:n]
        if valid is not None:
            keys = keys & valid
        here = blk == i
        out[here] = attention_rows(q_rot[rows[here]], k_rot, v, keys, head_dim)
    return out


def attn3d_sparse_oracle(q, k, v, seqs: Sequence[Tuple[int, int, int, int]], rope_dims: Sequence[int],
                         theta: float, tau: float, qblk: int, kblk: int, key_mask: Optional[torch.Tensor] = None,
                         selection=None, select: Optional[List[Tuple[int, int, torch.Tensor]]] = None):
    """Block-sparse attention.  Returns (out, selection, scores).

    With ``select`` = None every row is computed: out is fp64 [total, heads, D], selection[s][h] the bool block
    mask used and scores[s][h] the block scores (None where a selection was supplied).  With ``select`` = a list
    of (seq, head, local rows) only those rows are computed: out, selection and scores are lists in that order
    (this is how full-size cases are sampled).  ``selection`` overrides B2-B4 (to check the attention
    arithmetic on a given choice of blocks): indexed [s][h] in the first form, a list parallel to ``select`` in
    the second.
    """
    cu, pos, has = layout_positions(seqs)
    total, heads, D = q.shape
    dense = select is None
    if dense:
        select = [(s, h, None) for s in range(len(seqs)) for h in range(heads)]
        out_dense = torch.zeros(total, heads, v.shape[2], dtype=F64)
        used = [[None] * heads for _ in seqs]
        scs = [[None] * heads for _ in seqs]
    outs, used_l, scs_l = [], [], []
    for idx, (s, h, rows) in enumerate(select):
        a, b = cu[s], cu[s + 1]
        n = b - a
        L = seqs[s][0]
        valid = None if key_mask is None else (key_mask[a:b].to("cpu") != 0)
        q_rot = rope_rotate(widen(q[a:b, h]), pos[a:b], has[a:b], rope_dims, theta)
        k_rot = rope_rotate(widen(k[a:b, h]), pos[a:b], has[a:b], rope_dims, theta)
        if selection is None:
            sc = block_scores(q_rot, k_rot, D, qblk, kblk)
            sel = block_select(sc, tau, L, qblk, kblk)
        else:
            sc, sel = None, (selection[s][h] if dense else selection[idx])
        rows_t = torch.arange(n, dtype=torch.int64) if rows is None else torch.as_tensor(rows, dtype=torch.int64)
        o = sparse_rows(q_rot, k_rot, widen(v[a:b, h]), sel, valid, rows_t, D, qblk, kblk)
        if dense:
            out_dense[a:b, h] = o
            used[s][h], scs[s][h] = sel, sc
        else:
            outs.append(o)
            used_l.append(sel)
            scs_l.append(sc)
    return (out_dense, used, scs) if dense else (outs, used_l, scs_l)


def compare(gpu_rows: torch.Tensor, ref_rows: torch.Tensor) -> Tuple[float, float]:
    """O6: (max-abs error, relative L2 error) of widened GPU rows against fp64 rows."""
    g = widen(gpu_rows)
    d = g - ref_rows
    max_abs = float(d.abs().max()) if d.numel() else 0.0
    den = float(torch.linalg.vector_norm(ref_rows))
    rel = float(torch.linalg.vector_norm(d)) / den if den > 0 else float(torch.linalg.vector_norm(d))
    return max_abs, rel
