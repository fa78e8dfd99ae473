"""Pins for the fp64 oracle: closed forms, invariants, brute force and a library
special case.  None of these re-type the oracle's formulae with the same
primitives; each is chosen so that a plausible slip (wrong sign, swapped pair
members, wrong axis offset, wrong frequency, transposed operand, dropped
scale, mask polarity) fails at least one of them.  CPU only."""
import cmath
import math
import os

import numpy as np
import pytest
import torch

from oracle import attn3d_oracle as orc

F64 = torch.float64
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "closed_forms.txt")


def rnd(*shape, seed=0, dtype=torch.bfloat16):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(*shape, generator=g).to(dtype)


# ---------------------------------------------------------------- brute force
def brute_force(q, k, v, seqs, rope_dims, theta, key_mask=None):
    """Pure-Python loops; RoPE as a complex multiplication; full score rows."""
    total, heads, D = q.shape
    q = q.to(F64).tolist(); k = k.to(F64).tolist(); v = v.to(F64).tolist()
    out = [[[0.0] * D for _ in range(heads)] for _ in range(total)]
    start = 0
    for (L, T, H, W) in seqs:
        n = L + T * H * W

        def rot(vec, i):
            if i < L:
                return list(vec)
            p = i - L
            coords = (p // (H * W), (p // W) % H, p % W)
            res = list(vec)
            off = 0
            for a in range(3):
                d = rope_dims[a]
                for j in range(d // 2):
                    z = complex(vec[off + 2 * j], vec[off + 2 * j + 1])
                    z = z * cmath.exp(1j * coords[a] * theta ** (-2.0 * j / d))
                    res[off + 2 * j], res[off + 2 * j + 1] = z.real, z.imag
                off += d
            return res

        for h in range(heads):
            kr = [rot(k[start + j][h], j) for j in range(n)]
            for i in range(n):
                qi = rot(q[start + i][h], i)
                sc = []
                for j in range(n):
                    if key_mask is not None and int(key_mask[start + j]) == 0:
                        sc.append(None)
                    else:
                        sc.append(sum(a * b for a, b in zip(qi, kr[j])) / math.sqrt(D))
                live = [x for x in sc if x is not None]
                if not live:
                    continue
                m = max(live)
                l = 0.0
                acc = [0.0] * D
                for j in range(n):
                    if sc[j] is None:
                        continue
                    e = math.exp(sc[j] - m)
                    l += e
                    for d_ in range(D):
                        acc[d_] += e * v[start + j][h][d_]
                out[start + i][h] = [x / l for x in acc]
        start += n
    return torch.tensor(out, dtype=F64)


@pytest.mark.parametrize("case", range(5))
def test_p7_brute_force_tiny_grids(case):
    cases = [
        ([(0, 2, 2, 3)], (2, 2, 4), 8, 2, None),
        ([(3, 1, 3, 2)], (4, 2, 2), 8, 1, None),
        ([(2, 2, 1, 2), (0, 1, 2, 2), (5, 1, 1, 3)], (2, 4, 2), 10, 2, None),   # ragged, partial rope
        ([(4, 2, 2, 2)], (2, 2, 2), 6, 2, "mask"),
        ([(3, 1, 2, 2), (3, 2, 1, 2)], (0, 4, 2), 6, 1, "mask"),
    ]
    seqs, rd, D, heads, mk = cases[case]
    total = sum(L + T * H * W for (L, T, H, W) in seqs)
    q, k, v = (rnd(total, heads, D, seed=10 * case + i) for i in range(3))
    mask = None
    if mk:
        mask = torch.ones(total, dtype=torch.uint8)
        mask[1] = 0
        mask[2] = 0
        mask[total - 1] = 0
    ref = brute_force(q, k, v, seqs, rd, 100.0, mask)
    got = orc.attn3d_oracle(q, k, v, seqs, rd, 100.0, mask)
    assert torch.allclose(got, ref, rtol=0, atol=1e-12)


def test_p7_brute_force_on_slice_of_tiny_config():
    # the tiny contract case (grid 4x8x8, D=64, split 16/24/24) on 24 rows of one head
    seqs = [(0, 4, 8, 8)]
    q, k, v = (rnd(256, 1, 64, seed=i + 40) for i in range(3))
    ref = brute_force(q, k, v, seqs, (16, 24, 24), 10000.0)
    got = orc.attn3d_oracle(q, k, v, seqs, (16, 24, 24), 10000.0)
    assert torch.allclose(got, ref, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- closed forms
def _golden():
    vals = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, w0, w1 = line.split()
        vals[name] = (float(w0), float(w1))
    return vals


def test_p6_two_token_closed_forms():
    g = _golden()
    v = torch.tensor([[[3.0, -1.0]], [[-2.0, 5.0]]], dtype=F64)
    # case A: D=2, d_T=2 -> omega_0 = 1 whatever theta is
    q = torch.tensor([[[1.0, 0.0]], [[1.0, 0.0]]], dtype=F64)
    out = orc.attn3d_oracle(q, q.clone(), v, [(0, 2, 1, 1)], (2, 0, 0), theta=123.0)
    w0, w1 = g["A"]
    assert torch.allclose(out[0, 0], w0 * v[0, 0] + w1 * v[1, 0], atol=1e-15)
    # case B/C: D=4, d_T=4, theta=1e4; tokens at t=0, t=7 and t=50 (others are dummies we mask)
    T = 51
    q4 = torch.zeros(T, 1, 4, dtype=F64)
    q4[:, 0, 2] = 1.0
    v4 = torch.zeros(T, 1, 4, dtype=F64)
    v4[0, 0] = torch.tensor([1.0, 2.0, 3.0, 4.0])
    v4[50, 0] = torch.tensor([-4.0, 0.5, 0.25, 8.0])
    mask = torch.zeros(T, dtype=torch.uint8)
    mask[0] = 1
    mask[50] = 1
    out = orc.attn3d_oracle(q4, q4.clone(), v4, [(0, T, 1, 1)], (4, 0, 0), 10000.0, mask)
    w0, w1 = g["B"]
    assert torch.allclose(out[0, 0], w0 * v4[0, 0] + w1 * v4[50, 0], atol=1e-15)
    w0, w1 = g["C"]
    assert torch.allclose(out[7, 0], w0 * v4[0, 0] + w1 * v4[50, 0], atol=1e-15)


def test_axis_offsets_and_order_closed_form():
    """Each axis owns its own slice of the head dims, in T, H, W order, and the
    grid is walked t-slowest / w-fastest.  One pair per axis, theta irrelevant
    (omega_0 = 1), so the relative angle seen through axis a is just the
    coordinate difference along a."""
    T, H, W = 2, 3, 4
    n = T * H * W
    for axis in range(3):
        q = torch.zeros(n, 1, 8, dtype=F64)
        q[:, 0, 2 * axis] = 2.0             # only the pair of this axis carries signal
        v = torch.eye(n, dtype=F64)[:, None, :8].clone() if n <= 8 else torch.randn(n, 1, 8, dtype=F64)
        out = orc.attn3d_oracle(q, q.clone(), v, [(0, T, H, W)], (2, 2, 2), 77.0)
        # expected weights for query token 0: scores 4*cos(delta_axis)/sqrt(8)
        coords = [(p // (H * W), (p // W) % H, p % W) for p in range(n)]
        sc = torch.tensor([4.0 * math.cos(c[axis]) / math.sqrt(8.0) for c in coords], dtype=F64)
        wts = torch.softmax(sc, 0)
        assert torch.allclose(out[0, 0], (wts[:, None] * v[:, 0]).sum(0), atol=1e-14)
    # dims past the rotary width pass through: signal in dims 6,7 gives uniform-angle-free scores
    q = torch.zeros(n, 1, 8, dtype=F64)
    q[:, 0, 6] = 1.5
    v = torch.randn(n, 1, 8, dtype=F64)
    out = orc.attn3d_oracle(q, q.clone(), v, [(0, T, H, W)], (2, 2, 2), 77.0)
    assert torch.allclose(out[5, 0], v[:, 0].mean(0), atol=1e-14)


def test_frequency_ladder():
    """omega_j = theta^(-2j/d_a): rotate unit vectors and read the angle back."""
    d, theta, pos = 8, 10000.0, 3
    x = torch.zeros(1, d, dtype=F64)
    x[0, 0::2] = 1.0
    y = orc.rope_rotate(x, torch.tensor([[pos, 0, 0]]), torch.tensor([True]), (d, 0, 0), theta)
    for j in range(d // 2):
        ang = math.atan2(float(y[0, 2 * j + 1]), float(y[0, 2 * j]))
        assert abs(ang - pos * 10000.0 ** (-2.0 * j / d)) < 1e-14
    # positive position rotates counter-clockwise: (1,0) -> (cos, +sin)
    assert float(y[0, 1]) > 0


# ---------------------------------------------------------------- invariants
def test_p1_uniform_scores_give_mean_of_valid_v():
    seqs = [(3, 2, 2, 2), (1, 1, 2, 3)]
    total = 11 + 7
    q = torch.zeros(total, 2, 8, dtype=torch.bfloat16)
    k, v = rnd(total, 2, 8, seed=1), rnd(total, 2, 8, seed=2)
    mask = torch.ones(total, dtype=torch.uint8)
    mask[[0, 5, 12]] = 0
    out = orc.attn3d_oracle(q, k, v, seqs, (2, 2, 4), 10000.0, mask)
    vv = v.to(F64)
    m0 = [i for i in range(11) if i not in (0, 5)]
    m1 = [i for i in range(11, 18) if i != 12]
    assert torch.allclose(out[:11], vv[m0].mean(0)[None].expand(11, -1, -1), atol=1e-14)
    assert torch.allclose(out[11:], vv[m1].mean(0)[None].expand(7, -1, -1), atol=1e-14)


def test_p2_one_hot_keys_reproduce_v_rows():
    # 2x4x4 grid = 32 tokens, D = 64; token n lives in pair plane n: q_n = k_n = c e_{2n}
    n, D = 32, 64
    c = math.sqrt(800.0 * math.sqrt(D)) + 1.0
    q = torch.zeros(n, 1, D, dtype=F64)
    for i in range(n):
        q[i, 0, 2 * i] = c
    v = rnd(n, 1, D, seed=5).to(F64)
    out = orc.attn3d_oracle(q, q.clone(), v, [(0, 2, 4, 4)], (16, 24, 24), 10000.0)
    assert torch.equal(out, v)


def test_p3_permutation_of_keys_and_queries():
    L, T, H, W = 2, 2, 3, 2
    seqs = [(L, T, H, W)]
    n = L + T * H * W
    q, k, v = (rnd(n, 2, 8, seed=i + 7) for i in range(3))
    cu, pos, has = orc.layout_positions(seqs)
    base = orc.attn3d_oracle_pos(q, k, v, cu, pos, has, (2, 4, 2), 50.0)
    perm = torch.randperm(n, generator=torch.Generator().manual_seed(3))
    # keys/values travel with their positions; queries stay: output unchanged
    out = orc.attn3d_oracle_pos(q, k[perm], v[perm], cu, pos, has, (2, 4, 2), 50.0)
    assert not torch.allclose(out, base, atol=1e-6)          # positions matter ...
    kq_pos = pos.clone()
    # ... so give K its permuted positions by running keys and queries through separate calls
    k_rot = orc.rope_rotate(orc.widen(k[perm]), pos[perm], has[perm], (2, 4, 2), 50.0)
    q_rot = orc.rope_rotate(orc.widen(q), pos, has, (2, 4, 2), 50.0)
    for h in range(2):
        o = orc.attention_rows(q_rot[:, h], k_rot[:, h], orc.widen(v[perm])[:, h], None, 8)
        assert torch.allclose(o, base[:, h], atol=1e-12)
    # permuting queries (with their positions) permutes rows
    out = orc.attn3d_oracle_pos(q[perm], k, v, cu, pos, has, (2, 4, 2), 50.0)
    q_rot_p = orc.rope_rotate(orc.widen(q[perm]), pos[perm], has[perm], (2, 4, 2), 50.0)
    k_rot0 = orc.rope_rotate(orc.widen(k), pos, has, (2, 4, 2), 50.0)
    for h in range(2):
        o = orc.attention_rows(q_rot_p[:, h], k_rot0[:, h], orc.widen(v)[:, h], None, 8)
        assert torch.allclose(o, base[perm][:, h], atol=1e-12)


def test_p4_rope_norms_inverse_identity():
    seqs = [(3, 3, 4, 5)]
    n = 3 + 60
    x = rnd(n, 2, 16, seed=9).to(F64)
    _, pos, has = orc.layout_positions(seqs)
    y = orc.rope_rotate(x, pos, has, (4, 6, 4), 10000.0)
    # per pair and per row norms
    assert torch.allclose(y[..., 0:14:2] ** 2 + y[..., 1:14:2] ** 2,
                          x[..., 0:14:2] ** 2 + x[..., 1:14:2] ** 2, atol=1e-13)
    assert torch.allclose(y.norm(dim=-1), x.norm(dim=-1), atol=1e-13)
    # pass-through dims and prefix rows untouched; position 0 is the identity
    assert torch.equal(y[..., 14:], x[..., 14:])
    assert torch.equal(y[:3], x[:3])
    assert torch.equal(y[3], x[3])
    # video rows off the origin do change
    assert not torch.allclose(y[10], x[10], atol=1e-3)
    # R(p) R(-p) = I
    z = orc.rope_rotate(y, -pos, has, (4, 6, 4), 10000.0)
    assert torch.allclose(z, x, atol=1e-13)


def test_p5_shift_invariance_video_only():
    seqs = [(0, 3, 2, 4)]
    q, k, v = (rnd(24, 2, 12, seed=i + 20) for i in range(3))
    cu, pos, has = orc.layout_positions(seqs)
    a = orc.attn3d_oracle_pos(q, k, v, cu, pos, has, (4, 4, 4), 10000.0)
    b = orc.attn3d_oracle_pos(q, k, v, cu, pos, has, (4, 4, 4), 10000.0, origin=(5, -3, 11))
    assert torch.allclose(a, b, atol=1e-10)
    # with a prefix the origin matters (prefix has no position): guards against a vacuous pin
    seqs = [(2, 3, 2, 4)]
    q, k, v = (rnd(26, 2, 12, seed=i + 23) for i in range(3))
    cu, pos, has = orc.layout_positions(seqs)
    a = orc.attn3d_oracle_pos(q, k, v, cu, pos, has, (4, 4, 4), 10000.0)
    b = orc.attn3d_oracle_pos(q, k, v, cu, pos, has, (4, 4, 4), 10000.0, origin=(5, -3, 11))
    assert not torch.allclose(a, b, atol=1e-6)


def test_p8_no_rope_equals_library_sdpa():
    total, heads, D = 37, 3, 16
    q, k, v = (rnd(total, heads, D, seed=i + 30).to(F64) for i in range(3))
    mask = torch.ones(total, dtype=torch.uint8)
    mask[[4, 9, 36]] = 0
    got = orc.attn3d_oracle(q, k, v, [(5, 2, 4, 4)], (0, 0, 0), 10000.0, mask)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.permute(1, 0, 2)[None], k.permute(1, 0, 2)[None], v.permute(1, 0, 2)[None],
        attn_mask=(mask != 0)[None, None, None, :])[0].permute(1, 0, 2)
    assert torch.allclose(got, ref, atol=1e-13)
    # prefix-only sequence with rope dims set: still the plain routine (prefix carries no RoPE)
    got = orc.attn3d_oracle(q[:9], k[:9], v[:9], [(9, 0, 1, 1)], (4, 4, 4), 10000.0)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q[:9].permute(1, 0, 2)[None], k[:9].permute(1, 0, 2)[None], v[:9].permute(1, 0, 2)[None])[0].permute(1, 0, 2)
    assert torch.allclose(got, ref, atol=1e-13)


def test_p9_padded_prefix_equals_unpadded():
    T, H, W, D, heads = 2, 3, 4, 12, 2
    Lpad, Lval = 8, 3
    nv = T * H * W
    q, k, v = (rnd(Lpad + nv, heads, D, seed=i + 50) for i in range(3))
    mask = torch.ones(Lpad + nv, dtype=torch.uint8)
    mask[Lval:Lpad] = 0
    padded = orc.attn3d_oracle(q, k, v, [(Lpad, T, H, W)], (4, 4, 4), 10000.0, mask)
    keep = list(range(Lval)) + list(range(Lpad, Lpad + nv))
    tight = orc.attn3d_oracle(q[keep], k[keep], v[keep], [(Lval, T, H, W)], (4, 4, 4), 10000.0)
    assert torch.allclose(padded[keep], tight, atol=1e-13)
    # rows at padded positions are still defined (attend to valid keys) and finite
    assert torch.isfinite(padded).all()


def test_p10_packed_equals_separate():
    seqs = [(2, 1, 2, 3), (4, 2, 2, 2), (0, 1, 1, 5)]
    lens = [8, 12, 5]
    total = sum(lens)
    q, k, v = (rnd(total, 2, 8, seed=i + 60) for i in range(3))
    packed = orc.attn3d_oracle(q, k, v, seqs, (2, 2, 4), 10000.0)
    a = 0
    for s, n in zip(seqs, lens):
        alone = orc.attn3d_oracle(q[a:a + n], k[a:a + n], v[a:a + n], [s], (2, 2, 4), 10000.0)
        assert torch.allclose(packed[a:a + n], alone, atol=1e-14)
        a += n


def test_p11_convex_hull_linearity_constant():
    seqs = [(3, 2, 3, 3)]
    n = 21
    q, k = rnd(n, 2, 8, seed=70), rnd(n, 2, 8, seed=71)
    v = (torch.rand(n, 2, 8, generator=torch.Generator().manual_seed(72)) * 2 - 1).to(torch.bfloat16)
    out = orc.attn3d_oracle(q, k, v, seqs, (2, 4, 2), 10000.0)
    vv = v.to(F64)
    assert (out <= vv.max(0).values[None] + 1e-15).all() and (out >= vv.min(0).values[None] - 1e-15).all()
    v2 = rnd(n, 2, 8, seed=73)
    lin = orc.attn3d_oracle(q, k, 2.0 * vv + 0.5 * v2.to(F64), seqs, (2, 4, 2), 10000.0)
    out2 = orc.attn3d_oracle(q, k, v2, seqs, (2, 4, 2), 10000.0)
    assert torch.allclose(lin, 2.0 * out + 0.5 * out2, atol=1e-13)
    const = orc.attn3d_oracle(q, k, torch.full((n, 2, 8), 0.75, dtype=F64), seqs, (2, 4, 2), 10000.0)
    assert torch.allclose(const, torch.full_like(const, 0.75), atol=1e-15)


def test_p12_p13_independence_and_masked_garbage():
    seqs = [(2, 1, 2, 2), (2, 1, 2, 2)]
    total = 12
    q, k, v = (rnd(total, 3, 8, seed=i + 80) for i in range(3))
    mask = torch.ones(total, dtype=torch.uint8)
    mask[1] = 0
    mask[7] = 0
    base = orc.attn3d_oracle(q, k, v, seqs, (2, 2, 2), 10000.0, mask)
    q2, k2, v2 = q.clone(), k.clone(), v.clone()
    q2[:, 1] += 1
    k2[:, 1] *= 2
    v2[:, 1] -= 3                   # head 1 only
    out = orc.attn3d_oracle(q2, k2, v2, seqs, (2, 2, 2), 10000.0, mask)
    assert torch.equal(out[:, 0], base[:, 0]) and torch.equal(out[:, 2], base[:, 2])
    assert not torch.equal(out[:, 1], base[:, 1])
    k3, v3 = k.clone(), v.clone()
    k3[6:] *= -1.5
    v3[6:] += 9                      # sequence 1 only
    out = orc.attn3d_oracle(q, k3, v3, seqs, (2, 2, 2), 10000.0, mask)
    assert torch.equal(out[:6], base[:6]) and not torch.equal(out[6:], base[6:])
    k4, v4 = k.clone(), v.clone()
    k4[[1, 7]] = 1e4
    v4[[1, 7]] = -777.0              # masked keys: finite garbage
    out = orc.attn3d_oracle(q, k4, v4, seqs, (2, 2, 2), 10000.0, mask)
    assert torch.equal(out, base)
    # mask polarity: zero means "do not attend"
    allz = orc.attn3d_oracle(q, k, v, seqs, (2, 2, 2), 10000.0, torch.zeros(total, dtype=torch.uint8))
    assert torch.equal(allz, torch.zeros_like(allz))


def test_p14_scale_tradeoff_and_sqrt_d():
    seqs = [(1, 2, 2, 2)]
    q, k, v = (rnd(9, 2, 8, seed=i + 90).to(F64) for i in range(3))
    a = orc.attn3d_oracle(q, k, v, seqs, (2, 2, 4), 10000.0)
    b = orc.attn3d_oracle(q * 4.0, k / 4.0, v, seqs, (2, 2, 4), 10000.0)
    assert torch.allclose(a, b, atol=1e-13)
    # the scale is 1/sqrt(full head_dim): zero-padding D from 8 to 32 with rope on the first 8
    # must equal scaling q by sqrt(8/32)
    qp = torch.cat([q, torch.zeros(9, 2, 24, dtype=F64)], -1)
    kp = torch.cat([k, torch.zeros(9, 2, 24, dtype=F64)], -1)
    vp = torch.cat([v, torch.zeros(9, 2, 24, dtype=F64)], -1)
    c = orc.attn3d_oracle(qp, kp, vp, seqs, (2, 2, 4), 10000.0)[..., :8]
    d = orc.attn3d_oracle(q * 0.5, k, v, seqs, (2, 2, 4), 10000.0)
    assert torch.allclose(c, d, atol=1e-13)


def test_select_matches_dense_and_row_chunking():
    seqs = [(2, 2, 3, 2), (0, 1, 2, 5)]
    total = 14 + 10
    q, k, v = (rnd(total, 2, 8, seed=i + 100) for i in range(3))
    dense = orc.attn3d_oracle(q, k, v, seqs, (2, 2, 4), 10000.0)
    rows = torch.tensor([0, 3, 9])
    sel = orc.attn3d_oracle(q, k, v, seqs, (2, 2, 4), 10000.0, None, [(1, 1, rows), (0, 0, rows)])
    assert torch.allclose(sel[0], dense[14 + rows, 1], atol=1e-15)
    assert torch.allclose(sel[1], dense[rows, 0], atol=1e-15)
    kr = orc.rope_oracle(k, seqs, (2, 2, 4))
    qr = orc.rope_oracle(q, seqs, (2, 2, 4))
    o = orc.attention_rows(qr[:14, 0], kr[:14, 0], orc.widen(v)[:14, 0], None, 8, row_chunk=3)
    assert torch.allclose(o, dense[:14, 0], atol=1e-14)


def test_half_pairing_differs_and_is_a_permutation_of_adjacent():
    x = rnd(5, 1, 8, seed=3).to(F64)
    pos = torch.tensor([[i, 0, 0] for i in range(5)])
    has = torch.ones(5, dtype=torch.bool)
    adj = orc.rope_rotate(x, pos, has, (8, 0, 0), 10000.0)
    idx = torch.tensor([0, 2, 4, 6, 1, 3, 5, 7])
    half = orc.rope_rotate(x[..., idx], pos, has, (8, 0, 0), 10000.0, pairing="half")
    assert torch.allclose(half, adj[..., idx], atol=1e-15)


def test_widen_is_exact_and_compare_metrics():
    x = torch.tensor([1.0, -0.33203125, 3.0e-39, 65280.0], dtype=torch.bfloat16)
    assert orc.widen(x).tolist() == [float(t) for t in x.float().tolist()]
    ref = torch.tensor([[3.0, 4.0]], dtype=F64)
    got = torch.tensor([[3.0, 4.5]], dtype=torch.float32)
    ma, rl = orc.compare(got, ref)
    assert ma == 0.5 and abs(rl - 0.1) < 1e-15


# ---------------------------------------------------------------- QK normalisation (Section 3.5, group (2))
def test_qk_rms_norm_closed_form_and_invariants():
    # closed form: x = (3, 4): mean square 12.5
    x = torch.tensor([[3.0, 4.0]], dtype=F64)
    g = torch.tensor([2.0, -1.0], dtype=F64)
    y = orc.qk_rms_norm(x, g, 0.0)
    assert torch.allclose(y, torch.tensor([[6.0 / math.sqrt(12.5), -4.0 / math.sqrt(12.5)]], dtype=F64), atol=1e-15)
    y = orc.qk_rms_norm(x, g, 3.5)                       # eps sits inside the square root, next to the mean square
    assert torch.allclose(y, torch.tensor([[6.0 / 4.0, -4.0 / 4.0]], dtype=F64), atol=1e-15)
    # invariants: unit gain gives unit RMS; positive rescaling of a row changes nothing; rows are independent
    x = rnd(7, 3, 16, seed=200).to(F64)
    one = torch.ones(16, dtype=F64)
    y = orc.qk_rms_norm(x, one, 0.0)
    assert torch.allclose((y * y).mean(-1), torch.ones(7, 3, dtype=F64), atol=1e-14)
    assert torch.allclose(orc.qk_rms_norm(x * 37.5, one, 0.0), y, atol=1e-14)
    x2 = x.clone()
    x2[2, 1] *= -3.0
    y2 = orc.qk_rms_norm(x2, one, 0.0)
    assert torch.equal(y2[:2], y[:2]) and torch.allclose(y2[2, 1], -y[2, 1], atol=1e-15) and torch.equal(y2[2, 0], y[2, 0])
    # the gain multiplies element-wise after the normalisation
    g = rnd(16, seed=201).to(F64)
    assert torch.allclose(orc.qk_rms_norm(x, g, 1e-6), orc.qk_rms_norm(x, one, 1e-6) * g, atol=1e-15)


def test_qk_norm_inside_attention_matches_brute_force_and_order():
    seqs = [(2, 1, 2, 3), (0, 2, 1, 2)]
    total, heads, D = 8 + 4, 2, 8
    q, k, v = (rnd(total, heads, D, seed=210 + i) for i in range(3))
    gq, gk = rnd(D, seed=213).float(), rnd(D, seed=214).float()
    eps = 1e-3
    got = orc.attn3d_oracle(q, k, v, seqs, (2, 2, 4), 100.0, None, None, q_gain=gq, k_gain=gk, norm_eps=eps)

    def norm_loops(x, g):
        x = x.to(F64).tolist()
        g = g.to(F64).tolist()
        out = [[[0.0] * D for _ in range(heads)] for _ in range(total)]
        for t in range(total):
            for h in range(heads):
                ms = sum(e * e for e in x[t][h]) / D
                for d in range(D):
                    out[t][h][d] = x[t][h][d] / math.sqrt(ms + eps) * g[d]
        return torch.tensor(out, dtype=F64)

    ref = brute_force(norm_loops(q, gq), norm_loops(k, gk), v, seqs, (2, 2, 4), 100.0)
    assert torch.allclose(got, ref, atol=1e-12)
    # normalise-then-rotate, not the other way round: with a non-constant gain the two differ ...
    rot_then_norm = orc.qk_rms_norm(orc.rope_oracle(k, seqs, (2, 2, 4), 100.0), gk, eps)
    norm_then_rot = orc.rope_oracle(k, seqs, (2, 2, 4), 100.0, gain=gk, norm_eps=eps)
    assert not torch.allclose(rot_then_norm, norm_then_rot, atol=1e-3)
    # ... and with a constant gain they coincide (rotations preserve the mean square)
    c = torch.full((D,), 1.5)
    a = orc.qk_rms_norm(orc.rope_oracle(k, seqs, (2, 2, 4), 100.0), c, eps)
    b = orc.rope_oracle(k, seqs, (2, 2, 4), 100.0, gain=c, norm_eps=eps)
    assert torch.allclose(a, b, atol=1e-14)
    # no gains given: the plain path, bit for bit
    assert torch.equal(orc.attn3d_oracle(q, k, v, seqs, (2, 2, 4), 100.0),
                       orc.attn3d_oracle(q, k, v, seqs, (2, 2, 4), 100.0, q_gain=None, k_gain=None))


# ---------------------------------------------------------------- block-sparse variant (Section 3.4)
def test_block_select_rule_on_hand_made_scores():
    # one query block, scores 0..7: mu = 3.5, sigma = sqrt(5.25) = 2.2913
    sc = torch.arange(8, dtype=F64)[None]
    assert orc.block_select(sc, 1.0, 0, 256, 128).tolist() == [[False] * 6 + [True, True]]       # > 5.79
    assert orc.block_select(sc, 1.5, 0, 256, 128).tolist() == [[False] * 7 + [True]]             # > 6.94
    assert orc.block_select(sc, 0.0, 0, 256, 128).tolist() == [[False] * 4 + [True] * 4]         # > mean
    # constant scores: sigma = 0, nothing is strictly above the mean; the arg-max block is kept
    assert int(orc.block_select(torch.ones(1, 5, dtype=F64), 1.0, 0, 256, 128).sum()) == 1
    # rails: prefix of 130 tokens = KV blocks 0 and 1 always on; query block 0 (holds prefix rows) dense
    sc = torch.tensor([[0.0, 0, 0, 0, 9.0], [0.0, 0, 0, 0, 9.0]], dtype=F64)
    sel = orc.block_select(sc, 1.0, 130, 256, 128)
    assert sel.tolist() == [[True] * 5, [True, True, False, False, True]]
    # the rails follow the block sizes: with 64-token KV blocks the same prefix covers three of them, and with
    # 128-token query blocks both query blocks hold prefix rows
    assert orc.block_select(sc, 1.0, 130, 256, 64).tolist() == [[True] * 5, [True, True, True, False, True]]
    assert orc.block_select(sc, 1.0, 130, 128, 128).tolist() == [[True] * 5, [True] * 5]
    # a larger tau never selects more
    g = torch.Generator().manual_seed(5)
    sc = torch.randn(6, 40, generator=g, dtype=F64)
    a, b, c = (orc.block_select(sc, t, 0, 256, 128) for t in (1.0, 1.25, 1.5))
    assert bool((b <= a).all()) and bool((c <= b).all()) and int(c.sum()) < int(a.sum())


def test_block_scores_are_pooled_logits():
    n, D = 300, 8
    q, k = rnd(n, D, seed=300).to(F64), rnd(n, D, seed=301).to(F64)
    sc = orc.block_scores(q, k, D, 256, 128)
    assert sc.shape == (2, 3)
    # block (1, 2): query rows 256..299, keys 256..299 (ragged tails average over what is there)
    want = float(q[256:].mean(0) @ k[256:].mean(0)) / math.sqrt(D)
    assert abs(float(sc[1, 2]) - want) < 1e-14
    # pooled logits = mean of the full logit block (bilinearity)
    full = (q[:256] @ k[128:256].t()) / math.sqrt(D)
    assert abs(float(sc[0, 1]) - float(full.mean())) < 1e-13
    # other block sizes: 7 query blocks of 50 (no tail), 4 KV blocks of 96 (tail of 12)
    sc = orc.block_scores(q, k, D, 50, 96)
    assert sc.shape == (6, 4)
    full = (q[100:150] @ k[288:].t()) / math.sqrt(D)
    assert abs(float(sc[2, 3]) - float(full.mean())) < 1e-13


def test_sparse_oracle_reduces_to_dense_and_respects_selection():
    seqs = [(130, 2, 10, 26)]                       # 130 + 520 = 650 tokens: 3 query blocks, 6 KV blocks
    n = 650
    q, k, v = (rnd(n, 2, 16, seed=310 + i) for i in range(3))
    dense = orc.attn3d_oracle(q, k, v, seqs, (4, 6, 6), 10000.0)
    # everything selected = dense attention
    full = [[torch.ones(3, 6, dtype=torch.bool) for _ in range(2)]]
    out, _, _ = orc.attn3d_sparse_oracle(q, k, v, seqs, (4, 6, 6), 10000.0, 1.0, 256, 128, selection=full)
    assert torch.allclose(out, dense, atol=1e-13)
    # tau = -inf selects everything as well
    out, used, sc = orc.attn3d_sparse_oracle(q, k, v, seqs, (4, 6, 6), 10000.0, -1e30, 256, 128)
    assert torch.allclose(out, dense, atol=1e-13) and all(bool(u.all()) for u in used[0])
    # a real tau: prefix rails hold, prefix query block equals dense, a dropped block's V does not matter
    out, used, sc = orc.attn3d_sparse_oracle(q, k, v, seqs, (4, 6, 6), 10000.0, 0.5, 256, 128)
    sel = used[0][1]
    assert bool(sel[:, :2].all()) and bool(sel[0].all()) and not bool(sel.all())
    assert torch.allclose(out[:256], dense[:256], atol=1e-13)
    i, j = [(int(a), int(b)) for a, b in zip(*torch.nonzero(~sel, as_tuple=True))][0]
    v2 = v.clone()
    v2[j * 128: (j + 1) * 128, 1] = 50.0
    out2, _, _ = orc.attn3d_sparse_oracle(q, k, v2, seqs, (4, 6, 6), 10000.0, 0.5, 256, 128, selection=used)
    assert torch.equal(out2[i * 256: (i + 1) * 256, 1], out[i * 256: (i + 1) * 256, 1])
    # the block statistic is taken on the rotated operands in fp64, nothing rounded
    qr = orc.rope_oracle(q, seqs, (4, 6, 6), 10000.0)[:, 1]
    kr = orc.rope_oracle(k, seqs, (4, 6, 6), 10000.0)[:, 1]
    assert torch.equal(sc[0][1], orc.block_scores(qr, kr, 16, 256, 128))
    # sampled rows of one (sequence, head) = the same rows of the all-rows result, with and without a given selection
    rows = torch.tensor([0, 255, 256, 300, 511, 512, 649])
    o_s, u_s, sc_s = orc.attn3d_sparse_oracle(q, k, v, seqs, (4, 6, 6), 10000.0, 0.5, 256, 128, select=[(0, 1, rows)])
    # (the library matmul may block 7 rows differently from 256: equal to rounding of fp64, not to the bit)
    assert torch.allclose(o_s[0], out[rows, 1], atol=1e-14) and torch.equal(u_s[0], used[0][1]) and torch.equal(sc_s[0], sc[0][1])
    o_s, _, _ = orc.attn3d_sparse_oracle(q, k, v, seqs, (4, 6, 6), 10000.0, 0.5, 256, 128, selection=[used[0][1]],
                                         select=[(0, 1, rows)])
    assert torch.allclose(o_s[0], out[rows, 1], atol=1e-14)
    # other block sizes give another (valid) approximation: 128-token query blocks select per 128 rows
    out_b, used_b, _ = orc.attn3d_sparse_oracle(q, k, v, seqs, (4, 6, 6), 10000.0, 0.5, 128, 64)
    assert used_b[0][0].shape == (6, 11) and bool(used_b[0][0][:, :3].all()) and bool(used_b[0][0][:2].all())
    assert torch.allclose(out_b[:256], dense[:256], atol=1e-13)
