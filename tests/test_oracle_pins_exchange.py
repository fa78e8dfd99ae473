"""Pins for the exchange / FP8-output oracle (Section 3.3: attention collectives and quantized communication).
CPU only.  None of them re-types the oracle's formula: code values are the format's published constants,
nearest-code is a brute-force search, the cast is re-checked against the library's own, the permutations are
pure-Python index loops, and the end-to-end identity is checked against the single-device attention."""
import itertools
import math

import pytest
import torch

from oracle import attn3d_oracle as orc
from oracle import exchange_oracle as xo

F64 = torch.float64


# ------------------------------------------------------------------------------------------------ E4M3
def test_e4m3_code_values_from_the_format_definition():
    # OCP 8-bit floating point, E4M3: bias 7, largest finite 448 = 0x7e, smallest subnormal 2^-9 = 0x01,
    # smallest normal 2^-6 = 0x08, 1.0 = 0x38, 0x7f and 0xff are NaN, there are no infinities.
    dec = xo.e4m3_decode(torch.arange(256, dtype=torch.uint8))
    assert dec[0x38].item() == 1.0
    assert dec[0x7E].item() == 448.0
    assert dec[0x01].item() == 2.0 ** -9
    assert dec[0x08].item() == 2.0 ** -6
    assert dec[0x07].item() == 7 * 2.0 ** -9
    assert dec[0x40].item() == 2.0 and dec[0x44].item() == 3.0
    assert dec[0xB8].item() == -1.0
    assert math.isnan(dec[0x7F].item()) and math.isnan(dec[0xFF].item())
    assert dec[0x00].item() == 0.0 and dec[0x80].item() == 0.0 and math.copysign(1.0, dec[0x80].item()) == -1.0
    finite = dec[~torch.isnan(dec)]
    assert torch.isfinite(finite).all() and finite.abs().max().item() == 448.0
    # positive codes are strictly increasing in value
    pos = dec[:0x7F]
    assert (pos[1:] > pos[:-1]).all()


def test_e4m3_round_trip_of_every_code():
    codes = torch.arange(256, dtype=torch.uint8)
    dec = xo.e4m3_decode(codes)
    enc = xo.e4m3_encode(dec)
    keep = ~torch.isnan(dec)
    assert torch.equal(enc[keep], codes[keep])
    assert enc[0x7F].item() == 0x7F and enc[0xFF].item() == 0x7F


def test_e4m3_ties_go_to_the_even_code_and_saturation():
    dec = xo.e4m3_decode(torch.arange(0x7F, dtype=torch.uint8))
    mid = (dec[:-1] + dec[1:]) / 2                      # exact in fp64
    enc = xo.e4m3_encode(mid).to(torch.int64)
    lo = torch.arange(0x7E)
    even = torch.where(lo % 2 == 0, lo, lo + 1)
    assert torch.equal(enc, even)
    # a hair off the midpoint goes to the nearer neighbour
    eps = (dec[1:] - dec[:-1]) * 1e-6
    assert torch.equal(xo.e4m3_encode(mid - eps).to(torch.int64), lo)
    assert torch.equal(xo.e4m3_encode(mid + eps).to(torch.int64), lo + 1)
    # the same, mirrored
    assert torch.equal(xo.e4m3_encode(-mid).to(torch.int64), even + 0x80)
    big = torch.tensor([449.0, 464.0, 480.0, 1e6, float("inf"), -1e6, float("-inf"), float("nan")], dtype=F64)
    assert xo.e4m3_encode(big).tolist() == [0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0xFE, 0xFE, 0x7F]


def test_e4m3_encode_is_the_nearest_code_brute_force():
    g = torch.Generator().manual_seed(7)
    x = torch.cat([torch.randn(4000, generator=g, dtype=F64) * s for s in (1e-3, 0.02, 1.0, 30.0, 200.0)])
    x = x[x.abs() <= 448.0]
    table = xo.e4m3_decode(torch.arange(256, dtype=torch.uint8))
    table = torch.where(torch.isnan(table), torch.full_like(table, float("inf")), table)
    dist = (x[:, None] - table[None, :]).abs()
    best = dist.min(dim=1).values
    got = xo.e4m3_decode(xo.e4m3_encode(x))
    assert torch.equal((got - x).abs(), best)
    # sign of zero results follows the input
    assert xo.e4m3_encode(torch.tensor([-1e-9], dtype=F64)).item() == 0x80


def test_e4m3_encode_equals_the_library_cast_in_range():
    g = torch.Generator().manual_seed(11)
    x32 = torch.cat([torch.randn(20000, generator=g) * s for s in (0.01, 1.0, 100.0)])
    x32 = x32[x32.abs() <= 448.0]
    lib = x32.to(torch.float8_e4m3fn).view(torch.uint8)
    assert torch.equal(xo.e4m3_encode(x32.to(F64)), lib)


# ------------------------------------------------------------------------------------------------ layouts
def test_shard_ranges_cover_the_token_axis():
    for total, G in itertools.product((0, 1, 7, 8, 9, 1000, 111856), (1, 2, 3, 4, 8)):
        r = xo.shard_ranges(total, G)
        assert len(r) == G and r[0][0] == 0 and r[-1][1] == total
        assert all(a <= b for a, b in r) and all(r[i][1] == r[i + 1][0] for i in range(G - 1))
        sizes = [b - a for a, b in r]
        assert max(sizes) == -(-total // G) if total else max(sizes) == 0
        assert sizes == sorted(sizes, reverse=True)


def test_pack_and_merge_are_the_index_maps_brute_force():
    n, heads, D, G = 5, 6, 4, 3
    hl = heads // G
    q = torch.arange(n * heads * D, dtype=torch.int32).reshape(n, heads, D)
    k = q + 1000
    v = q + 2000
    packed = xo.pack_qkv_reference(q, k, v, G)
    assert packed.shape == (G, n, 3, hl, D) and packed.is_contiguous()
    src = (q, k, v)
    for g, t, w, h, d in itertools.product(range(G), range(n), range(3), range(hl), range(D)):
        assert packed[g, t, w, h, d].item() == src[w][t, g * hl + h, d].item()
    recv = torch.arange(G * n * hl * D, dtype=torch.int32).reshape(G, n, hl, D)
    merged = xo.merge_heads_reference(recv)
    assert merged.shape == (n, heads, D)
    for g, t, h, d in itertools.product(range(G), range(n), range(hl), range(D)):
        assert merged[t, g * hl + h, d].item() == recv[g, t, h, d].item()


@pytest.mark.parametrize("total,G", [(13, 2), (16, 4), (9, 3), (5, 6)])
def test_exchange_with_identity_attention_returns_each_ranks_rows(total, G):
    # attend = "return v" (resp. q, k): the round trip must hand every rank exactly its token rows of the
    # full tensor, all heads, whatever the (ragged, possibly empty) shard sizes.
    heads, D = 12, 4
    q = torch.arange(total * heads * D, dtype=torch.int64).reshape(total, heads, D)
    k, v = q + 10 ** 6, q + 2 * 10 ** 6
    hl = heads // G
    for which, full in enumerate((q, k, v)):
        seen = []

        def attend(qg, kg, vg, g, which=which):
            seen.append(g)
            # head shard g of the full tensors, every token, in order
            assert torch.equal(qg, q[:, g * hl:(g + 1) * hl]) and torch.equal(kg, k[:, g * hl:(g + 1) * hl])
            assert torch.equal(vg, v[:, g * hl:(g + 1) * hl])
            return (qg, kg, vg)[which]

        outs = xo.ulysses_reference(q, k, v, G, attend)
        assert seen == list(range(G))
        for (a, b), o in zip(xo.shard_ranges(total, G), outs):
            assert torch.equal(o, full[a:b])


def test_exchange_around_the_attention_equals_single_device_attention():
    # X6: heads are independent, so head-sharded attention between the two exchanges is the plain attention.
    seqs = [(3, 2, 2, 3), (0, 1, 3, 2)]
    total = sum(L + T * H * W for (L, T, H, W) in seqs)
    heads, D, rope = 4, 16, (4, 6, 6)
    g = torch.Generator().manual_seed(3)
    q, k, v = (torch.randn(total, heads, D, generator=g).to(torch.bfloat16) for _ in range(3))
    mask = torch.ones(total, dtype=torch.uint8)
    mask[1] = 0
    full = orc.attn3d_oracle(q, k, v, seqs, rope, 10000.0, key_mask=mask)
    for G in (2, 4):
        outs = xo.ulysses_reference(q, k, v, G,
                                    lambda qg, kg, vg, r: orc.attn3d_oracle(qg.contiguous(), kg.contiguous(), vg.contiguous(),
                                                                            seqs, rope, 10000.0, key_mask=mask))
        got = torch.cat(outs, dim=0)
        assert got.shape == full.shape
        assert (got - full).abs().max().item() < 1e-13
