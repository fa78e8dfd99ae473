"""Pins for the exchange / FP8-output oracle (Section 3.2: attention collectives and quantized communication).
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


# ------------------------------------------------------------------------------------------------ block-INT8
def test_ue5m3_table_constants_and_order():
    dec = xo.ue5m3_decode(torch.arange(256, dtype=torch.uint8))
    assert dec[0x78].item() == 1.0                     # e = 15, m = 0
    assert dec[0x7C].item() == 1.5 and dec[0x80].item() == 2.0
    assert dec[0x01].item() == 2.0 ** -17 and dec[0x07].item() == 7 * 2.0 ** -17
    assert dec[0x08].item() == 2.0 ** -14              # first normal continues the subnormal ladder
    assert dec[0xF7].item() == 15 * 2.0 ** 12 == 61440.0
    assert dec[0x00].item() == 0.0 and torch.isnan(dec[0xF8:]).all()
    pos = dec[1:0xF8]
    assert (pos[1:] > pos[:-1]).all()
    # neighbouring values are never more than 9/8 apart once normal: the scale wastes at most 12.5 % of the range
    assert ((pos[8:] / pos[7:-1]).max().item() <= 9.0 / 8.0 + 1e-15)


def test_ue5m3_encode_up_brute_force_and_boundaries():
    table = [xo.ue5m3_decode(torch.tensor([c], dtype=torch.uint8)).item() for c in range(1, 0xF8)]
    g = torch.Generator().manual_seed(2)
    amax = torch.cat([torch.rand(300, generator=g, dtype=F64) * s for s in (1e-6, 1e-3, 1.0, 50.0, 5e4)])
    amax = torch.cat([amax, torch.tensor([0.0, 127.0, 127.0 * 1.125, 127.0 * 2.0 ** -17, 1e9], dtype=F64)])
    got = xo.ue5m3_encode_up(amax).tolist()
    for a, c in zip(amax.tolist(), got):
        want = next((i + 1 for i, v in enumerate(table) if 127.0 * v >= a), 0xF7)
        assert c == want, (a, c, want)
    # exactly on a grid point -> that point; one ulp above -> the next one
    for c in (0x01, 0x08, 0x40, 0x78, 0x7F, 0xF6):
        on = 127.0 * table[c - 1]
        assert xo.ue5m3_encode_up(torch.tensor([on], dtype=F64)).item() == c
        assert xo.ue5m3_encode_up(torch.tensor([math.nextafter(on, math.inf)], dtype=F64)).item() == c + 1


def test_block_int8_error_bound_range_use_and_symmetries():
    g = torch.Generator().manual_seed(4)
    x = (torch.randn(64, 3, 128, generator=g) * torch.tensor([0.01, 1.0, 40.0])[None, :, None]).to(torch.bfloat16)
    x[0, 0, :32] = 0                                                  # an all-zero group
    q, codes = xo.block_int8_quantize(x)
    assert q.dtype == torch.int8 and codes.dtype == torch.uint8 and codes.shape == (64, 3, 4)
    assert int(q.to(torch.int32).abs().max()) <= 127 and int(codes.min()) >= 1 and int(codes.max()) <= 0xF7
    assert codes[0, 0, 0].item() == 1 and not q[0, 0, :32].any()
    s = xo.ue5m3_decode(codes)
    xg = x.to(F64).reshape(64, 3, 4, 32)
    amax = xg.abs().amax(-1)
    # smallest scale that does not clip: 127 s >= amax, and the next smaller scale would clip
    assert bool((127.0 * s >= amax).all())
    prev = xo.ue5m3_decode((codes.to(torch.int64) - 1).clamp(min=0).to(torch.uint8))
    assert bool(((127.0 * prev < amax) | (codes == 1)).all())
    # rounding error at most half a step (+ fp32 rounding of the product), the largest element uses >= 8/9 of the range
    deq = xo.block_int8_dequantize(q, codes)
    err = (deq - x.to(F64)).reshape(64, 3, 4, 32).abs()
    assert bool((err <= s[..., None] * (0.5 + 1e-5)).all())
    qmax = q.to(torch.int32).reshape(64, 3, 4, 32).abs().amax(-1)
    assert bool(((qmax >= 112) | (amax == 0) | (codes <= 8)).all())
    # x -> 2^k x: same integers, codes move by 8 k (every step is exact for powers of two)
    q2, c2 = xo.block_int8_quantize((x.to(F64) * 8.0).to(torch.bfloat16))
    keep = (codes > 8) & (amax > 0)                                       # away from the subnormal codes
    assert torch.equal(q2.reshape(64, 3, 4, 32)[keep], q.reshape(64, 3, 4, 32)[keep])
    assert torch.equal(c2[keep].to(torch.int64), codes[keep].to(torch.int64) + 24)
    # x -> -x: integers negate, codes stay
    q3, c3 = xo.block_int8_quantize(-x)
    assert torch.equal(q3, -q) and torch.equal(c3, codes)


def test_block_int8_hand_made_group():
    # amax = 127 -> s = 1 exactly (code 0x78) and q = x for integers; amax = 128 -> next scale 1.125 (0x79)
    x = torch.zeros(1, 32, dtype=F64)
    x[0, :5] = torch.tensor([127.0, -3.0, 2.5, 3.5, -0.5])
    q, c = xo.block_int8_quantize(x)
    assert c.item() == 0x78 and q[0, :5].tolist() == [127, -3, 2, 4, 0]            # ties to even: 2.5 -> 2, 3.5 -> 4, -0.5 -> 0
    x[0, 0] = 128.0
    q, c = xo.block_int8_quantize(x)
    assert c.item() == 0x79 and q[0, 0].item() == 114                              # 128 / 1.125 = 113.78


def test_record_layouts_byte_for_byte():
    assert xo.qkv_record_bytes(128) == 400 and xo.out_record_bytes(128) == 144     # the paper's sizes
    assert xo.qkv_record_bytes(64) == 208 and xo.out_record_bytes(64) == 80
    D = 128
    q = torch.zeros(2, 3, D, dtype=F64); k = torch.zeros_like(q); v = torch.zeros_like(q)
    q[1, 2, 0] = 127.0            # group 0 of q: scale 1, value 127
    q[1, 2, 33] = -254.0          # group 1 of q: scale 2 (0x80), value -127
    k[1, 2, 127] = 63.5           # group 3 of k: scale 0.5 (0x70), value 127
    v[1, 2, 64] = 1.0             # group 2 of v: smallest s with 127 s >= 1: 2^-7 * 1.125 = 0.0087890625 (0x41): q = 114
    rec = xo.qkv_records(q, k, v)
    assert rec.shape == (2, 3, 400) and rec.dtype == torch.uint8
    r = rec[1, 2].tolist()
    assert r[0] == 127 and r[33] == 0x81 and r[128 + 127] == 127 and r[256 + 64] == 114
    assert r[384:388] == [0x78, 0x80, 0x01, 0x01]
    assert r[388:392] == [0x01, 0x01, 0x01, 0x70]
    assert r[392:396] == [0x01, 0x01, 0x41, 0x01]
    assert r[396:400] == [0, 0, 0, 0]
    assert not rec[0].view(-1)[:384].any()                                         # other records: zero values, code 1
    dq, dk, dv = xo.qkv_from_records(rec, D)
    assert dq[1, 2, 0].item() == 127.0 and dq[1, 2, 33].item() == -254.0 and dk[1, 2, 127].item() == 63.5
    assert abs(dv[1, 2, 64].item() - 1.0) <= 0.0087890625 / 2
    orec = xo.out_records(q)
    assert orec.shape == (2, 3, 144)
    ro = orec[1, 2].tolist()
    assert ro[0] == 127 and ro[33] == 0x81 and ro[128:132] == [0x78, 0x80, 0x01, 0x01] and ro[132:144] == [0] * 12
    assert torch.equal(xo.out_from_records(orec, D), xo.block_int8_dequantize(*xo.block_int8_quantize(q)))
