"""CPU oracle for the sequence-parallel exchange around the attention and its FP8 output.  TEST INFRASTRUCTURE ONLY.

Never on the product path: only tests, the smoke check and the benchmark's CPU-baseline leg may import it.  It
shares no code, tables or constants with the CUDA sources and imports nothing from the package.

What it states (Section 3.2 of the paper, "Optimized attention collectives" and "Quantized communication", and
Section 3.3, "Joint optimization with quantized communication"):

  X1  sequence-sharded layout: rank g of G holds a contiguous range of the flat token axis, all heads,
      tensors [n_g, heads, D] (the flat (total, heads, head_dim) layout; no batch dimension);
  X2  head-sharded layout: rank g holds every token and heads [g*heads/G, (g+1)*heads/G);
  X3  the packed QKV exchange: ONE all-to-all.  What rank s sends to rank g is the reference permutation
      stack((q, k, v), 1) -> [n_s, 3, G, heads/G, D] -> permute(2, 0, 1, 3, 4)[g] = [n_s, 3, heads/G, D];
      rank g concatenates what it receives in source order and so holds [total, 3, heads/G, D];
  X4  the output return: ONE all-to-all of the rows [n_g, heads/G, D] each rank owes to token owner g, then
      the inverse head merge [G, n, heads/G, D] -> permute(1, 0, 2, 3) -> [n, heads, D] (rank-major heads);
  X5  layout steps move bytes and change none: exact for any element type;
  X6  attention between X3 and X4 over the head shard is the plain attention of attn3d_oracle restricted
      to those heads (heads are independent), so the whole exchange returns to every rank exactly its token
      rows of the single-device attention: that definition is the oracle of the end-to-end result;
  X7  the FP8 output format: each output element becomes one raw E4M3 byte (OCP 8-bit float, 4 exponent bits
      with bias 7, 3 mantissa bits, no infinities, 0x7f / 0xff = NaN, largest finite 448), unit scale, no
      metadata, no padding.  Conversion: round to nearest, ties to even, magnitudes beyond 448 (infinities
      included) saturate to +-448, NaN -> 0x7f.  (The paper fixes the format, not the rounding rule; this
      is the rule of the hardware conversion instruction and of the OCP text's "saturating" mode.)

  X8-X11  the block-INT8 wire formats: see the comment block above ue5m3_decode.

Pins: tests/test_oracle_pins_exchange.py (code table values, round trip of all codes, ties, nearest-code brute
force, the library cast as a special case; permutation brute force, exchange-then-merge identity, the
end-to-end identity X6 on a tiny problem; for the block-INT8 formats: scale-table constants, smallest-scale rule
by brute force and at exact boundaries, error bound, power-of-two scaling and sign symmetries, byte positions of a
hand-made record).
"""
from __future__ import annotations

import math
from typing import Callable, List, Sequence, Tuple

import torch

# --------------------------------------------------------------------------------------------- E4M3 (X7)


def e4m3_decode(codes: torch.Tensor) -> torch.Tensor:
    """uint8 codes -> fp64 values (NaN for 0x7f / 0xff)."""
    c = codes.to(torch.int64)
    sign = torch.where((c & 0x80) != 0, -1.0, 1.0).to(torch.float64)
    e = (c >> 3) & 0xF
    m = (c & 0x7).to(torch.float64)
    normal = torch.ldexp(1.0 + m / 8.0, (e - 7).to(torch.int32))
    subnormal = m / 8.0 * 2.0 ** -6
    mag = torch.where(e == 0, subnormal, normal)
    mag = torch.where((c & 0x7F) == 0x7F, torch.full_like(mag, float("nan")), mag)
    return sign * mag


def _round_half_even(x: torch.Tensor) -> torch.Tensor:
    fl = torch.floor(x)
    diff = x - fl
    up = (diff > 0.5) | ((diff == 0.5) & (torch.remainder(fl, 2.0) == 1.0))
    return fl + up.to(x.dtype)


def e4m3_encode(x: torch.Tensor) -> torch.Tensor:
    """fp64 (or anything widened exactly to fp64) -> uint8 E4M3 codes: RNE, saturating, NaN -> 0x7f."""
    x = x.to(torch.float64)
    neg = torch.signbit(x)
    a = torch.clamp(torch.abs(x), max=448.0)                 # saturate (inf too); NaN stays NaN
    nan = torch.isnan(x)
    a = torch.where(nan, torch.zeros_like(a), a)
    # subnormal range: multiples of 2^-9 up to 2^-6 (the first normal), continuous in the code
    sub = a < 2.0 ** -6
    code_sub = _round_half_even(a * 2.0 ** 9)                # 0 .. 8
    # normal range: a = m * 2^e with m in [1, 2)
    mant, ex = torch.frexp(torch.where(sub, torch.ones_like(a), a))   # a = mant * 2^ex, mant in [0.5, 1)
    e = ex.to(torch.int64) - 1
    q = _round_half_even((mant * 2.0 - 1.0) * 8.0)           # 0 .. 8
    carry = q == 8.0
    e = e + carry.to(torch.int64)
    q = torch.where(carry, torch.zeros_like(q), q)
    code_norm = ((e + 7) << 3) + q.to(torch.int64)
    code = torch.where(sub, code_sub.to(torch.int64), code_norm)
    code = torch.clamp(code, max=0x7E)
    code = torch.where(nan, torch.full_like(code, 0x7F), code)
    code = code + torch.where(neg & ~nan, 0x80, 0)
    return code.to(torch.uint8)


# --------------------------------------------------------------------------------------------- layouts (X1-X5)


def shard_ranges(total: int, G: int) -> List[Tuple[int, int]]:
    """X1: contiguous token ranges, ceil(total/G) each, the last ones shorter (possibly empty)."""
    per = -(-total // G)
    return [(min(g * per, total), min((g + 1) * per, total)) for g in range(G)]


def pack_qkv_reference(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, G: int) -> torch.Tensor:
    """X3, the sender's side: [n, heads, D] x 3 -> [G, n, 3, heads/G, D] (slice g goes to rank g)."""
    n, heads, D = q.shape
    hl = heads // G
    x = torch.stack((q, k, v), dim=1)                        # [n, 3, heads, D]
    return x.reshape(n, 3, G, hl, D).permute(2, 0, 1, 3, 4).contiguous()


def all_to_all_reference(send: Sequence[Sequence[torch.Tensor]]) -> List[torch.Tensor]:
    """send[s][g] = what rank s sends to rank g (first axis = rows).  Returns recv[g] = concatenation over s."""
    G = len(send)
    return [torch.cat([send[s][g] for s in range(G)], dim=0) for g in range(G)]


def merge_heads_reference(recv: torch.Tensor) -> torch.Tensor:
    """X4, the receiver's side: [G, n, heads/G, D] -> [n, heads, D], head = g * heads/G + local head."""
    G, n, hl, D = recv.shape
    return recv.permute(1, 0, 2, 3).reshape(n, G * hl, D).contiguous()


def ulysses_reference(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, G: int,
                      attend: Callable[[torch.Tensor, torch.Tensor, torch.Tensor, int], torch.Tensor]) -> List[torch.Tensor]:
    """The whole exchange on one host, step by step (X1 -> X3 -> attention -> X4).

    q, k, v: [total, heads, D] (any dtype).  attend(q_g, k_g, v_g, g) -> [total, heads/G, D] is the attention of
    head shard g over all tokens.  Returns, per rank, its [n_g, heads, D] output rows.
    """
    total, heads, D = q.shape
    ranges = shard_ranges(total, G)
    send = []
    for (a, b) in ranges:
        packed = pack_qkv_reference(q[a:b], k[a:b], v[a:b], G)
        send.append([packed[g] for g in range(G)])
    recv = all_to_all_reference(send)                        # recv[g]: [total, 3, heads/G, D]
    outs = [attend(r[:, 0], r[:, 1], r[:, 2], g) for g, r in enumerate(recv)]
    back = [[outs[s][a:b] for (a, b) in ranges] for s in range(G)]   # rank s owes rows [a, b) to their owner
    merged = []
    for g, (a, b) in enumerate(ranges):
        stacked = torch.stack([back[s][g] for s in range(G)], dim=0)  # [G, n_g, heads/G, D]
        merged.append(merge_heads_reference(stacked))
    return merged


# --------------------------------------------------------------------------------------------- block-INT8 wire formats
#
# Section 3.2, "Quantized communication".  What the paper fixes: the QKV record of one (token, head) is 384 int8
# values, twelve scale codes (one per group of 32 values, "finite-positive UE5M3"), four zero bytes = 400 bytes; the
# output record is 128 values, four scale codes, padded from 132 to 144 bytes; all padding bytes are written.
# What it leaves open, and the reading taken here (X8-X11):
#   X8   UE5M3 = unsigned 8-bit float, 5 exponent bits (bias 15), 3 mantissa bits: code c, e = c >> 3, m = c & 7,
#        value (8 + m) * 2^(e - 18) for 1 <= e <= 30 and m * 2^-17 for e = 0; e = 31 is reserved.  "Finite-positive":
#        only codes 0x01 .. 0xf7 are ever produced;
#   X9   the scale of a group is the SMALLEST such value s with 127 * s >= max|x| (nothing clips; 127 * s is exact in
#        fp32 and fp64, so the choice does not depend on the precision it is made in); an all-zero group gets 0x01;
#   X10  q = clamp(round_half_even(x * (1 / s)), -127, 127) with the reciprocal and the product each rounded to
#        fp32: a float decides an integer here, so the decision is taken in the kernel's precision (IEEE fp32,
#        round to nearest) and is reproducible bit for bit; dequantised value = q * s (exact in fp32);
#   X11  record layout, head_dim D (D = 128 in the paper): [q values D | k values D | v values D | D/32 q codes |
#        D/32 k codes | D/32 v codes | zeros up to a multiple of 16 bytes] (396 -> 400); output record [values D |
#        D/32 codes | zeros up to a multiple of 16 bytes] (132 -> 144, "to align each record to 16 bytes").

GROUP = 32


def ue5m3_decode(codes: torch.Tensor) -> torch.Tensor:
    c = codes.to(torch.int64)
    e = c >> 3
    m = (c & 7).to(torch.float64)
    normal = torch.ldexp(8.0 + m, (e - 18).to(torch.int32))
    sub = m * 2.0 ** -17
    val = torch.where(e == 0, sub, normal)
    return torch.where(e == 31, torch.full_like(val, float("nan")), val)


def ue5m3_encode_up(bound127: torch.Tensor) -> torch.Tensor:
    """Smallest code in 0x01..0xf7 whose value s satisfies 127 * s >= bound127 (X9)."""
    table = ue5m3_decode(torch.arange(1, 0xF8, dtype=torch.uint8)) * 127.0      # ascending, exact
    idx = torch.searchsorted(table, bound127.to(torch.float64).contiguous(), right=False)
    return (torch.clamp(idx, max=table.numel() - 1) + 1).to(torch.uint8)


def block_int8_quantize(x: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    """x [..., D] (D a multiple of 32) -> (int8 values [..., D], uint8 scale codes [..., D/32])  (X9, X10)."""
    D = x.shape[-1]
    xg = x.to(torch.float64).reshape(*x.shape[:-1], D // GROUP, GROUP)
    amax = xg.abs().amax(dim=-1)
    codes = ue5m3_encode_up(amax)
    s32 = ue5m3_decode(codes).to(torch.float32)
    inv = torch.reciprocal(s32)                                                  # fp32, round to nearest
    q = torch.round(xg.to(torch.float32) * inv[..., None])                      # fp32 product, half-even
    q = torch.clamp(q, -127.0, 127.0).to(torch.int8)
    return q.reshape(x.shape), codes


def block_int8_dequantize(q: torch.Tensor, codes: torch.Tensor) -> torch.Tensor:
    D = q.shape[-1]
    s = ue5m3_decode(codes)
    return (q.to(torch.float64).reshape(*q.shape[:-1], D // GROUP, GROUP) * s[..., None]).reshape(q.shape)


def _padded(n: int) -> int:
    return (n + 15) // 16 * 16


def qkv_record_bytes(D: int) -> int:
    return _padded(3 * D + 3 * D // GROUP)


def out_record_bytes(D: int) -> int:
    return _padded(D + D // GROUP)


def qkv_records(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor) -> torch.Tensor:
    """[n, heads, D] x 3 -> uint8 [n, heads, qkv_record_bytes(D)]  (X11)."""
    n, heads, D = q.shape
    rec = torch.zeros((n, heads, qkv_record_bytes(D)), dtype=torch.uint8)
    ng = D // GROUP
    for w, x in enumerate((q, k, v)):
        vals, codes = block_int8_quantize(x)
        rec[:, :, w * D:(w + 1) * D] = vals.view(torch.uint8)
        rec[:, :, 3 * D + w * ng:3 * D + (w + 1) * ng] = codes
    return rec


def qkv_from_records(rec: torch.Tensor, D: int) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """uint8 records -> dequantised q, k, v in fp64 (each value is exactly representable in fp32)."""
    ng = D // GROUP
    out = []
    for w in range(3):
        vals = rec[..., w * D:(w + 1) * D].contiguous().view(torch.int8)
        codes = rec[..., 3 * D + w * ng:3 * D + (w + 1) * ng]
        out.append(block_int8_dequantize(vals, codes))
    return tuple(out)


def out_records(o: torch.Tensor) -> torch.Tensor:
    """[n, heads, D] -> uint8 [n, heads, out_record_bytes(D)]  (X11)."""
    n, heads, D = o.shape
    rec = torch.zeros((n, heads, out_record_bytes(D)), dtype=torch.uint8)
    vals, codes = block_int8_quantize(o)
    rec[:, :, :D] = vals.view(torch.uint8)
    rec[:, :, D:D + D // GROUP] = codes
    return rec


def out_from_records(rec: torch.Tensor, D: int) -> torch.Tensor:
    vals = rec[..., :D].contiguous().view(torch.int8)
    return block_int8_dequantize(vals, rec[..., D:D + D // GROUP])
