"""GPU: E4M3 output epilogue and the sequence-parallel exchange kernels (Section 3.2 of the paper).

One GPU stands in for the G ranks: their shards and buffers all live on it and the kernels of the "ranks" run one
after another (nothing waits on anything), which exercises exactly the addresses a real run would use with peer
pointers in place of local ones.  Layout kernels must be bit-exact against the oracle's reference permutations;
the end-to-end result must be the single-device attention."""
import os
from dataclasses import replace

import pytest
import torch

from oracle import attn3d_oracle as orc
from oracle import exchange_oracle as xo
from paper_2609_35110_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_MAX_ABS = 2e-2
TOL_REL_L2 = 5e-3


@pytest.fixture(scope="module")
def B():
    from paper_2609_35110_b200 import binding
    binding._lib()
    return binding


def seq_tuples(w):
    return [(s.text_len, s.T, s.H, s.W) for s in w.seqs]


def oracle_dense(w, inp):
    return orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seq_tuples(w), w.rope_dims, w.theta,
                             None if inp.key_mask is None else inp.key_mask.cpu())


# ------------------------------------------------------------------------------------------ E4M3 epilogue
def in_band(codes, centre, tol):
    """The code space is monotone, so 'the value that was rounded lies within centre -/+ tol' is the same as
    'the code lies between the encodings of centre - tol and centre + tol'."""
    got = xo.e4m3_decode(codes)
    lo = xo.e4m3_decode(xo.e4m3_encode(centre - tol))
    hi = xo.e4m3_decode(xo.e4m3_encode(centre + tol))
    return (got >= lo) & (got <= hi)


def check_e4m3(codes: torch.Tensor, ref: torch.Tensor, bf16_out: torch.Tensor = None):
    """codes: uint8 from the GPU; ref: fp64 oracle rows; bf16_out: the GPU's bf16 forward of the same inputs.

    A float decides an integer here, so the decision is checked in the kernel's precision: the E4M3 epilogue and
    the bf16 epilogue round the SAME fp32 value x, and bf16_out pins x to within 2^-9 relative, so the code must
    lie between the encodings of bf16_out * (1 -/+ 2^-8) -- one code almost everywhere.  Against the fp64 oracle
    the band is the attention's own error (measured max-abs on these inputs is 2e-3; contract 2e-2)."""
    codes = codes.cpu()
    got = xo.e4m3_decode(codes)
    assert not torch.isnan(got).any()
    stats = {}
    if bf16_out is not None:
        b = bf16_out.cpu().double()
        assert bool(in_band(codes, b, b.abs() * 2.0 ** -8 + 1e-30).all()), "E4M3 code is not a rounding of the kernel's value"
        stats["same_as_encoded_bf16"] = (codes == xo.e4m3_encode(b)).double().mean().item()
        assert stats["same_as_encoded_bf16"] > 0.95, stats   # bf16-then-E4M3 double rounding differs ~3 % of the time
    tol = 5e-3 * ref.abs() + 3e-3
    assert bool(in_band(codes, ref, tol).all()), "E4M3 code outside the band allowed by the attention tolerance"
    stats["same_as_encoded_oracle"] = (codes == xo.e4m3_encode(ref)).double().mean().item()
    assert stats["same_as_encoded_oracle"] > 0.8, stats
    # and as numbers: half a step of a 3-bit mantissa, or half a subnormal step, plus the attention tolerance
    assert bool(((got - ref).abs() <= ref.abs() * 2.0 ** -4 + 2.0 ** -10 + tol).all())
    return stats


@pytest.mark.parametrize("name", ["tiny", "lowres", "cfg_batch", "varlen"])
def test_e4m3_output_matches_encoded_oracle(B, name):
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    attn = B.Attn3d.from_workload(w, "cuda")
    n = w.total_tokens * w.heads * w.head_dim
    guard = 4096
    buf = torch.full((n + 2 * guard,), 0x7F, dtype=torch.uint8, device="cuda")      # NaN code: unwritten rows show up
    out = buf[guard:guard + n].view(w.total_tokens, w.heads, w.head_dim)
    B.sol_attn3d_forward_e4m3(attn.plan, inp.q, inp.k, inp.v, out, inp.key_mask)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert bool((buf[:guard] == 0x7F).all()) and bool((buf[-guard:] == 0x7F).all()), "store outside the output tensor"
    # the same call twice gives the same bytes, and the bf16 forward of the same plan still works afterwards
    out2 = torch.empty_like(out)
    B.sol_attn3d_forward_e4m3(attn.plan, inp.q, inp.k, inp.v, out2, inp.key_mask)
    ob = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    print(name, check_e4m3(out, oracle_dense(w, inp), ob))
    attn.close()


def test_e4m3_saturates_and_keeps_signs(B):
    # V = +-1000 everywhere: every output is +-1000 exactly in fp32, far above 448 -> saturated codes 0x7e / 0xfe
    w = wl.shrunk("tiny")
    inp = wl.make_inputs(w, "cuda")
    v = torch.full_like(inp.v, 1000.0)
    v[:, 1::2] = -1000.0
    attn = B.Attn3d.from_workload(w, "cuda")
    out = torch.empty((w.total_tokens, w.heads, w.head_dim), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_forward_e4m3(attn.plan, inp.q, inp.k, v, out, None)
    torch.cuda.synchronize()
    assert bool((out[:, 0::2] == 0x7E).all()) and bool((out[:, 1::2] == 0xFE).all())
    attn.close()


# ------------------------------------------------------------------------------------------ layout kernels
@pytest.mark.parametrize("G,n_local,heads,D", [(2, 300, 8, 128), (4, 77, 8, 64), (8, 33, 40, 128), (1, 10, 3, 64), (3, 0, 6, 64)])
def test_pack_qkv_is_the_reference_permutation(B, G, n_local, heads, D):
    g = torch.Generator(device="cuda").manual_seed(100 + G)
    # Q, K, V as views into one packed QKV buffer (token stride 3*heads*D), as the paper's packed storage
    packed = torch.randn((max(n_local, 1), 3, heads, D), generator=g, device="cuda").to(torch.bfloat16)[:n_local]
    q, k, v = packed[:, 0], packed[:, 1], packed[:, 2]
    hl = heads // G
    send = torch.full((G, n_local, 3, hl, D), -7.0, dtype=torch.bfloat16, device="cuda")
    dummy = torch.zeros(64, dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_pack_qkv(q, k, v, G, [send[r].data_ptr() if n_local else dummy.data_ptr() for r in range(G)], 0)
    torch.cuda.synchronize()
    want = xo.pack_qkv_reference(q.cpu(), k.cpu(), v.cpu(), G)
    assert torch.equal(send.cpu().view(torch.int16), want.view(torch.int16))
    # contiguous inputs give the same bytes
    if n_local:
        send2 = torch.empty_like(send)
        B.sol_attn3d_exchange_pack_qkv(q.contiguous(), k.contiguous(), v.contiguous(), G, [send2[r].data_ptr() for r in range(G)], 0)
        torch.cuda.synchronize()
        assert torch.equal(send2, send)


def test_layout_kernels_beyond_four_gib(B):
    """One rank of a one-way exchange at 150,000 tokens x 40 heads x 128: the packed destination is 4.6 GB, so chunk and
    byte offsets pass 2^32 in the pack, the record pack and the merge.  Every kernel works token by token, so slices of
    tokens (the first, those around the 2^32-byte mark, the last) are compared with the oracle on the same slices."""
    n, heads, D = 150_000, 40, 128
    g = torch.Generator(device="cuda").manual_seed(321)
    q, k, v = (torch.randn((n, heads, D), generator=g, device="cuda", dtype=torch.bfloat16) for _ in range(3))
    send = torch.empty((1, n, 3, heads, D), dtype=torch.bfloat16, device="cuda")
    assert send.numel() * 2 > (1 << 32)
    B.sol_attn3d_exchange_pack_qkv(q, k, v, 1, [send[0].data_ptr()], 0)
    rb = B.sol_attn3d_exchange_record_bytes(B.WIRE_QKV_INT8, D)
    send8 = torch.empty((1, n, heads, rb), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_pack_qkv_int8(q, k, v, 1, [send8[0].data_ptr()], 0)
    # return path: two ranks' results for 440,000 tokens, 4.5 GB in and out
    n2, hl = 440_000, 20
    recv = torch.randint(0, 256, (2, n2, hl, 2 * D), generator=g, device="cuda", dtype=torch.uint8)
    assert recv.numel() > (1 << 32)
    merged = torch.empty((n2, 2 * hl, 2 * D), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_merge_heads(recv, merged, n2, 2 * hl, 2 * D, 2)
    torch.cuda.synchronize()
    mark = (1 << 32) // (3 * heads * D * 2)                    # the token whose packed row straddles byte 2^32
    for t0, t1 in [(0, 64), (mark - 32, mark + 32), (n - 64, n)]:
        qs, ks, vs = q[t0:t1].cpu(), k[t0:t1].cpu(), v[t0:t1].cpu()
        want = xo.pack_qkv_reference(qs, ks, vs, 1)
        assert torch.equal(send[:, t0:t1].cpu().view(torch.int16), want.view(torch.int16)), (t0, t1)
        want8 = xo.qkv_records(qs, ks, vs)
        assert torch.equal(send8[0, t0:t1].cpu(), want8), (t0, t1)
    mark2 = (1 << 32) // (2 * hl * 2 * D)
    for t0, t1 in [(0, 64), (mark2 - 32, mark2 + 32), (n2 - 64, n2)]:
        want = xo.merge_heads_reference(recv[:, t0:t1].cpu())
        assert torch.equal(merged[t0:t1].cpu(), want), (t0, t1)


@pytest.mark.parametrize("G,n_local,heads,record", [(2, 300, 8, 256), (4, 77, 8, 128), (8, 33, 40, 144), (1, 5, 3, 64), (2, 129, 4, 16)])
def test_merge_heads_is_the_reference_permutation(B, G, n_local, heads, record):
    g = torch.Generator(device="cuda").manual_seed(200 + G)
    hl = heads // G
    recv = torch.randint(0, 256, (G, n_local, hl, record), generator=g, device="cuda", dtype=torch.uint8)
    pad = 32                                                    # output rows with a stride larger than dense
    out = torch.full((n_local, heads * record + pad), 0xAB, dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_merge_heads(recv, out, n_local, heads, record, G, out.stride(0))
    torch.cuda.synchronize()
    want = xo.merge_heads_reference(recv.cpu())
    assert torch.equal(out[:, :heads * record].cpu().view(n_local, heads, record), want)
    assert bool((out[:, heads * record:] == 0xAB).all())
    dense = torch.empty((n_local, heads, record), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_merge_heads(recv, dense, n_local, heads, record, G)
    torch.cuda.synchronize()
    assert torch.equal(dense.cpu(), want)


@pytest.mark.parametrize("G,heads,begin,count", [(2, 8, 1, 2), (4, 40, 7, 3), (1, 6, 0, 6), (8, 16, 1, 1)])
def test_head_groups_pack_and_merge_in_place(B, G, heads, begin, count):
    """A head group [begin, begin+count) of every rank's shard: the pack sends exactly those heads, the INT8 pack the
    same records, and the merge drops the group into its place in the full output row."""
    n_local, D = 53, 128
    g = torch.Generator(device="cuda").manual_seed(500 + G)
    q, k, v = (torch.randn((n_local, heads, D), generator=g, device="cuda").to(torch.bfloat16) for _ in range(3))
    hl = heads // G
    sel = torch.cat([torch.arange(r * hl + begin, r * hl + begin + count) for r in range(G)])
    send = torch.empty((G, n_local, 3, count, D), dtype=torch.bfloat16, device="cuda")
    B.sol_attn3d_exchange_pack_qkv(q, k, v, G, [send[r].data_ptr() for r in range(G)], 0, group_begin=begin, group_heads=count)
    torch.cuda.synchronize()
    want = xo.pack_qkv_reference(q.cpu()[:, sel], k.cpu()[:, sel], v.cpu()[:, sel], G)
    assert torch.equal(send.cpu().view(torch.int16), want.view(torch.int16))
    rb = B.sol_attn3d_exchange_record_bytes(B.WIRE_QKV_INT8, D)
    send8 = torch.empty((G, n_local, count, rb), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_pack_qkv_int8(q, k, v, G, [send8[r].data_ptr() for r in range(G)], 0, group_begin=begin, group_heads=count)
    torch.cuda.synchronize()
    rec = xo.qkv_records(q.cpu()[:, sel], k.cpu()[:, sel], v.cpu()[:, sel])
    for r in range(G):
        assert torch.equal(send8[r].cpu(), rec[:, r * count:(r + 1) * count])
    # merge: what the ranks return for this group lands at heads r*hl + begin .. of the full rows; the rest stays
    record = 2 * D
    recv = torch.randint(0, 256, (G, n_local, count, record), generator=g, device="cuda", dtype=torch.uint8)
    full = torch.full((n_local, heads, record), 0xAB, dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_merge_heads(recv, full.data_ptr() + begin * record, n_local, G * count, record, G, heads * record,
                                      out_rank_stride_bytes=hl * record)
    torch.cuda.synchronize()
    exp = torch.full((n_local, heads, record), 0xAB, dtype=torch.uint8)
    exp[:, sel] = xo.merge_heads_reference(recv.cpu())
    assert torch.equal(full.cpu(), exp)


def test_exchange_entry_points_reject_bad_arguments(B):
    x = torch.zeros((4, 6, 64), dtype=torch.bfloat16, device="cuda")
    dst = torch.zeros(4 * 3 * 6 * 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.SolAttn3dError):
        B.sol_attn3d_exchange_pack_qkv(x, x, x, 4, [dst.data_ptr()] * 4, 0)                 # 6 heads, 4 ranks
    with pytest.raises(B.SolAttn3dError):
        B.sol_attn3d_exchange_pack_qkv(x, x, x, 2, [dst.data_ptr(), dst.data_ptr() + 2], 0)  # misaligned destination
    r = torch.zeros((2, 4, 3, 40), dtype=torch.uint8, device="cuda")
    o = torch.zeros((4, 6, 40), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SolAttn3dError):
        B.sol_attn3d_exchange_merge_heads(r, o, 4, 6, 40, 2)                                # record not a multiple of 16


# ------------------------------------------------------------------------------------------ the whole exchange
def virtual_ranks_forward(B, w, inp, G, fmt, peer_style):
    """All G ranks on this GPU, one after another.  Returns the per-rank merged outputs [n_r, heads, D]."""
    total, heads, D = w.total_tokens, w.heads, w.head_dim
    hl = heads // G
    ranges = xo.shard_ranges(total, G)
    tok_begin = [a for a, _ in ranges] + [total]
    out_dtype = torch.uint8 if fmt == B.OUT_E4M3 else torch.bfloat16
    qkv = [torch.full((total, 3, hl, D), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(G)]
    # (1) QKV exchange
    if peer_style:
        for s, (a, b) in enumerate(ranges):                    # rank s stores straight into every owner's buffer
            B.sol_attn3d_exchange_pack_qkv(inp.q[a:b], inp.k[a:b], inp.v[a:b], G, [t.data_ptr() for t in qkv], a)
    else:
        for s, (a, b) in enumerate(ranges):
            send = torch.empty((G, b - a, 3, hl, D), dtype=torch.bfloat16, device="cuda")
            B.sol_attn3d_exchange_pack_qkv(inp.q[a:b], inp.k[a:b], inp.v[a:b], G,
                                           [send[r].data_ptr() if b > a else qkv[0].data_ptr() for r in range(G)], 0)
            for r in range(G):                                 # the all-to-all, by hand
                qkv[r][a:b] = send[r]
    for r in range(G):                                         # every rank now holds its head shard of everything
        for wh, full in enumerate((inp.q, inp.k, inp.v)):
            assert torch.equal(qkv[r][:, wh], full[:, r * hl:(r + 1) * hl])
    # (2) head-sharded attention, (3) output return + merge
    strides = (3 * hl * D, D)
    merged = [torch.full((b - a, heads, D), 0x7F if fmt == B.OUT_E4M3 else float("nan"), dtype=out_dtype, device="cuda")
              for (a, b) in ranges]
    recv = [torch.empty((G, b - a, hl, D), dtype=out_dtype, device="cuda") for (a, b) in ranges]
    for r in range(G):
        attn = B.Attn3d(seq_tuples(w), hl, D, w.rope_dims, w.theta, "cuda", q_strides=strides, k_strides=strides, v_strides=strides)
        qv, kv, vv = qkv[r][:, 0], qkv[r][:, 1], qkv[r][:, 2]
        if peer_style:
            B.sol_attn3d_forward_scatter(attn.plan, qv, kv, vv, inp.key_mask, [m.data_ptr() if m.numel() else 0 for m in merged],
                                         tok_begin, heads, r * hl, fmt)
        else:
            shard = torch.empty((total, hl, D), dtype=out_dtype, device="cuda")
            if fmt == B.OUT_E4M3:
                B.sol_attn3d_forward_e4m3(attn.plan, qv, kv, vv, shard, inp.key_mask)
            else:
                B.sol_attn3d_forward(attn.plan, qv, kv, vv, shard, inp.key_mask)
            for o, (a, b) in enumerate(ranges):                # the all-to-all, by hand
                recv[o][r] = shard[a:b]
        torch.cuda.synchronize()
        assert attn.status() == 0
        attn.close()
    if not peer_style:
        for o, (a, b) in enumerate(ranges):
            B.sol_attn3d_exchange_merge_heads(recv[o], merged[o], b - a, heads, D * merged[o].element_size(), G)
    torch.cuda.synchronize()
    return merged


@pytest.mark.parametrize("name,heads,G", [("tiny", 4, 2), ("lowres", 8, 4), ("lowres", 8, 8), ("cfg_batch", 4, 2), ("varlen", 6, 3)])
@pytest.mark.parametrize("peer_style", [False, True])
def test_exchange_returns_the_single_device_attention(B, name, heads, G, peer_style):
    w = replace(wl.shrunk(name), heads=heads)
    inp = wl.make_inputs(w, "cuda")
    single = B.Attn3d.from_workload(w, "cuda")
    want = single.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    single.close()
    merged = virtual_ranks_forward(B, w, inp, G, B.OUT_BF16, peer_style)
    got = torch.cat(merged, dim=0)
    # heads are independent and, at these sizes (one wave of CTAs), a CTA's arithmetic does not depend on the grid
    # around it: bit-identical
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    max_abs, rel_l2 = orc.compare(got.cpu(), oracle_dense(w, inp))
    assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2, (max_abs, rel_l2)


@pytest.mark.parametrize("peer_style", [False, True])
def test_exchange_with_e4m3_return(B, peer_style):
    w = replace(wl.shrunk("lowres"), heads=8)
    inp = wl.make_inputs(w, "cuda")
    merged = virtual_ranks_forward(B, w, inp, 4, B.OUT_E4M3, peer_style)
    got = torch.cat(merged, dim=0)
    check_e4m3(got, oracle_dense(w, inp))
    single = B.Attn3d.from_workload(w, "cuda")
    want = torch.empty((w.total_tokens, w.heads, w.head_dim), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_forward_e4m3(single.plan, inp.q, inp.k, inp.v, want, inp.key_mask)
    torch.cuda.synchronize()
    assert torch.equal(got, want)
    single.close()


def test_scatter_rejects_bad_arguments(B):
    w = wl.shrunk("tiny")
    inp = wl.make_inputs(w, "cuda")
    attn = B.Attn3d.from_workload(w, "cuda")
    total = w.total_tokens
    buf = torch.empty((total, w.heads, w.head_dim), dtype=torch.bfloat16, device="cuda")
    ok = [buf.data_ptr()]
    with pytest.raises(B.SolAttn3dError):
        B.sol_attn3d_forward_scatter(attn.plan, inp.q, inp.k, inp.v, None, ok, [0, total - 1], w.heads, 0)   # does not cover
    with pytest.raises(B.SolAttn3dError):
        B.sol_attn3d_forward_scatter(attn.plan, inp.q, inp.k, inp.v, None, ok, [0, total], w.heads - 1, 0)   # rows too narrow
    with pytest.raises(B.SolAttn3dError):
        B.sol_attn3d_forward_scatter(attn.plan, inp.q, inp.k, inp.v, None, [0], [0, total], w.heads, 0)      # NULL owner with rows
    with pytest.raises(B.SolAttn3dError):
        B.sol_attn3d_forward_scatter(attn.plan, inp.q, inp.k, inp.v, None, ok, [0, total], w.heads, 0, 7)    # unknown format
    B.sol_attn3d_forward_scatter(attn.plan, inp.q, inp.k, inp.v, None, ok, [0, total], w.heads, 0)
    torch.cuda.synchronize()
    want = attn.forward(inp.q, inp.k, inp.v, None)
    torch.cuda.synchronize()
    assert torch.equal(buf, want)
    attn.close()


def test_sequence_parallel_module_with_one_rank(B):
    """The torch.distributed plumbing itself (NCCL all-to-all with a single rank is a device copy)."""
    import torch.distributed as dist
    from paper_2609_35110_b200.sequence_parallel import SequenceParallelAttn3d
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", str(29400 + os.getpid() % 500))
    created = False
    if not dist.is_initialized():
        dist.init_process_group("nccl", rank=0, world_size=1)
        created = True
    try:
        w = replace(wl.shrunk("cfg_batch"), heads=4)
        inp = wl.make_inputs(w, "cuda")
        single = B.Attn3d.from_workload(w, "cuda")
        want = single.forward(inp.q, inp.k, inp.v, inp.key_mask)
        sp = SequenceParallelAttn3d(seq_tuples(w), w.heads, w.head_dim, w.rope_dims, w.theta)
        got = sp.forward(inp.q, inp.k, inp.v, inp.key_mask)
        torch.cuda.synchronize()
        assert torch.equal(got, want)
        sp8 = SequenceParallelAttn3d(seq_tuples(w), w.heads, w.head_dim, w.rope_dims, w.theta, out_format="e4m3")
        got8 = sp8.forward(inp.q, inp.k, inp.v, inp.key_mask)
        torch.cuda.synchronize()
        check_e4m3(got8, oracle_dense(w, inp))
        # block-INT8 both ways: equals the same kernels called by hand on one rank
        spq = SequenceParallelAttn3d(seq_tuples(w), w.heads, w.head_dim, w.rope_dims, w.theta, out_format="int8", qkv_wire="int8")
        gotq = spq.forward(inp.q, inp.k, inp.v, inp.key_mask)
        torch.cuda.synchronize()
        D = w.head_dim
        rec = torch.empty((w.total_tokens, w.heads, B.sol_attn3d_exchange_record_bytes(B.WIRE_QKV_INT8, D)), dtype=torch.uint8, device="cuda")
        B.sol_attn3d_exchange_pack_qkv_int8(inp.q, inp.k, inp.v, 1, [rec.data_ptr()], 0)
        qkv = torch.empty((w.total_tokens, 3, w.heads, D), dtype=torch.bfloat16, device="cuda")
        B.sol_attn3d_exchange_unpack_qkv_int8(rec, qkv, w.total_tokens, w.heads, D)
        st = (3 * w.heads * D, D)
        a2 = B.Attn3d(seq_tuples(w), w.heads, D, w.rope_dims, w.theta, "cuda", q_strides=st, k_strides=st, v_strides=st)
        o2 = a2.forward(qkv[:, 0], qkv[:, 1], qkv[:, 2], inp.key_mask)
        orec = torch.empty((w.total_tokens, w.heads, B.sol_attn3d_exchange_record_bytes(B.WIRE_OUT_INT8, D)), dtype=torch.uint8, device="cuda")
        B.sol_attn3d_exchange_quantize_out_int8(o2, orec)
        wantq = torch.empty_like(o2)
        B.sol_attn3d_exchange_dequantize_out_int8(orec, wantq)
        torch.cuda.synchronize()
        assert torch.equal(gotq, wantq)
        rel = float(torch.linalg.vector_norm(gotq.double() - want.double()) / torch.linalg.vector_norm(want.double()))
        assert rel < 3e-2, rel
        # head groups with the exchanges on side streams: same bytes as one group, for every wire format
        for kw, ref_out in (({}, got), ({"out_format": "e4m3"}, got8), ({"out_format": "int8", "qkv_wire": "int8"}, gotq)):
            for n_groups in (2, 4):
                spg = SequenceParallelAttn3d(seq_tuples(w), w.heads, w.head_dim, w.rope_dims, w.theta, n_groups=n_groups, **kw)
                for _ in range(2):
                    gg = spg.forward(inp.q, inp.k, inp.v, inp.key_mask)
                    torch.cuda.synchronize()
                    assert torch.equal(gg, ref_out), (kw, n_groups)
                spg.close()
        sp.close(); sp8.close(); spq.close(); a2.close(); single.close()
    finally:
        if created:
            dist.destroy_process_group()


# ------------------------------------------------------------------------------------------ block-INT8 wire formats
@pytest.mark.parametrize("G,n_local,heads,D", [(1, 50, 3, 128), (4, 301, 8, 128), (8, 33, 40, 128), (2, 77, 6, 64), (3, 0, 6, 64)])
def test_int8_qkv_records_are_bit_exact(B, G, n_local, heads, D):
    g = torch.Generator(device="cuda").manual_seed(300 + G)
    packed = torch.randn((max(n_local, 1), 3, heads, D), generator=g, device="cuda")
    packed[:, 1] *= 0.05                                     # different ranges per tensor, as K after QK-norm
    packed[:, 2] *= 30.0
    packed = packed.to(torch.bfloat16)[:n_local]
    if n_local > 2:
        packed[1, 0, 0, :32] = 0                             # an all-zero group
        packed[2, 2, 1, 5] = 127.0 * 64                      # a maximum that sits exactly on a scale (s = 64)
    q, k, v = packed[:, 0], packed[:, 1], packed[:, 2]
    hl = heads // G
    rb = B.sol_attn3d_exchange_record_bytes(B.WIRE_QKV_INT8, D)
    assert rb == xo.qkv_record_bytes(D)
    send = torch.full((G, n_local, hl, rb), 0xEE, dtype=torch.uint8, device="cuda")
    dummy = torch.zeros(64, dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_pack_qkv_int8(q, k, v, G, [send[r].data_ptr() if n_local else dummy.data_ptr() for r in range(G)], 0)
    torch.cuda.synchronize()
    want = xo.qkv_records(q.cpu(), k.cpu(), v.cpu())          # [n, heads, rb]
    for r in range(G):
        assert torch.equal(send[r].cpu(), want[:, r * hl:(r + 1) * hl]), f"records for rank {r}"
    if n_local == 0:
        return
    # receiver: dequantise into the packed [rows][3][hl][D] tensor; exact product, one rounding to bf16
    for r in range(G):
        qkv = torch.full((n_local, 3, hl, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.sol_attn3d_exchange_unpack_qkv_int8(send[r], qkv, n_local, hl, D)
        torch.cuda.synchronize()
        dq = xo.qkv_from_records(want[:, r * hl:(r + 1) * hl].contiguous(), D)
        for wch in range(3):
            assert torch.equal(qkv[:, wch].cpu().view(torch.int16), dq[wch].to(torch.bfloat16).view(torch.int16))
    # and the quantisation error as a number: half a step of the group's scale
    dq_all = xo.qkv_from_records(want, D)
    for wch, x in enumerate((q, k, v)):
        err = (dq_all[wch] - x.cpu().double()).abs().reshape(n_local, heads, D // 32, 32)
        amax = x.cpu().double().abs().reshape(n_local, heads, D // 32, 32).amax(-1, keepdim=True)
        assert bool((err <= amax / 127.0 * 1.125 * 0.5001 + 2.0 ** -17).all())


@pytest.mark.parametrize("n,heads,D", [(200, 5, 128), (77, 40, 128), (64, 3, 64), (0, 4, 128)])
def test_int8_output_records_are_bit_exact(B, n, heads, D):
    g = torch.Generator(device="cuda").manual_seed(400 + n)
    wide = (torch.randn((max(n, 1), heads + 2, D), generator=g, device="cuda") * 0.3).to(torch.bfloat16)[:n]
    rows = wide[:, 1:heads + 1]                               # a strided view: token stride (heads+2)*D
    rb = B.sol_attn3d_exchange_record_bytes(B.WIRE_OUT_INT8, D)
    assert rb == xo.out_record_bytes(D)
    rec = torch.full((max(n, 1), heads, rb), 0xEE, dtype=torch.uint8, device="cuda")[:n]
    B.sol_attn3d_exchange_quantize_out_int8(rows, rec)
    torch.cuda.synchronize()
    want = xo.out_records(rows.cpu())
    assert torch.equal(rec.cpu(), want)
    if n == 0:
        return
    back = torch.full((n, heads, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.sol_attn3d_exchange_dequantize_out_int8(rec, back)
    torch.cuda.synchronize()
    assert torch.equal(back.cpu().view(torch.int16), xo.out_from_records(want, D).to(torch.bfloat16).view(torch.int16))


def int8_pipeline_by_hand(B, w, inp, G):
    """Whole exchange with block-INT8 records both ways, G virtual ranks, every kernel called by hand.  Returns (per-rank
    bf16 rows, per-rank oracle attention of the dequantised inputs)."""
    total, heads, D = w.total_tokens, w.heads, w.head_dim
    hl = heads // G
    ranges = xo.shard_ranges(total, G)
    rb_in = B.sol_attn3d_exchange_record_bytes(B.WIRE_QKV_INT8, D)
    rb_out = B.sol_attn3d_exchange_record_bytes(B.WIRE_OUT_INT8, D)
    recv = [torch.empty((total, hl, rb_in), dtype=torch.uint8, device="cuda") for _ in range(G)]
    for s, (a, b) in enumerate(ranges):                        # peer style: records land in the owners' buffers
        B.sol_attn3d_exchange_pack_qkv_int8(inp.q[a:b], inp.k[a:b], inp.v[a:b], G, [t.data_ptr() for t in recv], a)
    torch.cuda.synchronize()
    want_rec = xo.qkv_records(inp.q.cpu(), inp.k.cpu(), inp.v.cpu())
    strides = (3 * hl * D, D)
    back = [torch.empty((G, b - a, hl, rb_out), dtype=torch.uint8, device="cuda") for (a, b) in ranges]
    ref_shards = []
    for r in range(G):
        assert torch.equal(recv[r].cpu(), want_rec[:, r * hl:(r + 1) * hl])
        qkv = torch.empty((total, 3, hl, D), dtype=torch.bfloat16, device="cuda")
        B.sol_attn3d_exchange_unpack_qkv_int8(recv[r], qkv, total, hl, D)
        attn = B.Attn3d(seq_tuples(w), hl, D, w.rope_dims, w.theta, "cuda", q_strides=strides, k_strides=strides, v_strides=strides)
        shard = attn.forward(qkv[:, 0], qkv[:, 1], qkv[:, 2], inp.key_mask)
        rec = torch.empty((total, hl, rb_out), dtype=torch.uint8, device="cuda")
        B.sol_attn3d_exchange_quantize_out_int8(shard, rec)
        torch.cuda.synchronize()
        assert attn.status() == 0
        attn.close()
        # oracle attention on the dequantised (bf16-rounded) inputs the GPU attention saw
        dq = [x.to(torch.bfloat16) for x in xo.qkv_from_records(want_rec[:, r * hl:(r + 1) * hl].contiguous(), D)]
        ref = orc.attn3d_oracle(dq[0], dq[1], dq[2], seq_tuples(w), w.rope_dims, w.theta,
                                None if inp.key_mask is None else inp.key_mask.cpu())
        max_abs, rel_l2 = orc.compare(shard.cpu(), ref)
        assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2, (max_abs, rel_l2)
        assert torch.equal(rec.cpu(), xo.out_records(shard.cpu()))
        ref_shards.append(ref)
        for o, (a, b) in enumerate(ranges):
            back[o][r] = rec[a:b]
    outs = []
    for o, (a, b) in enumerate(ranges):
        merged = torch.empty((b - a, heads, rb_out), dtype=torch.uint8, device="cuda")
        B.sol_attn3d_exchange_merge_heads(back[o], merged, b - a, heads, rb_out, G)
        rows = torch.empty((b - a, heads, D), dtype=torch.bfloat16, device="cuda")
        B.sol_attn3d_exchange_dequantize_out_int8(merged, rows)
        outs.append(rows)
    torch.cuda.synchronize()
    return outs, ref_shards


def test_exchange_with_int8_wire_formats(B):
    """Whole exchange, 4 virtual ranks, block-INT8 both ways.  Approximate by design, so two checks: the GPU
    pipeline equals the oracle pipeline fed with the same records (attention tolerance), and the end result stays
    within the quantisation error of the unquantised attention."""
    w = replace(wl.shrunk("lowres"), heads=8)
    inp = wl.make_inputs(w, "cuda")
    total, heads, D = w.total_tokens, w.heads, w.head_dim
    outs, ref_shards = int8_pipeline_by_hand(B, w, inp, 4)
    got = torch.cat(outs, 0).cpu().double()
    # against the oracle of the same pipeline: attention error + half an output step
    ref_pipeline = torch.cat(ref_shards, dim=1)
    step = ref_pipeline.abs().reshape(total, heads, D // 32, 32).amax(-1, keepdim=True) / 127.0 * 1.125
    assert bool(((got - ref_pipeline).reshape(total, heads, D // 32, 32).abs() <= 0.5 * step + 2e-3 + 2.0 ** -8 * step * 127).all())
    # against the unquantised attention: a few per cent, as the paper says "approximate"
    exact = oracle_dense(w, replace_mask(inp))
    rel = float(torch.linalg.vector_norm(got - exact) / torch.linalg.vector_norm(exact))
    print("int8 both ways: rel-L2 vs unquantised attention", rel)
    assert rel < 3e-2


def replace_mask(inp):
    class _I:
        pass
    o = _I()
    o.q, o.k, o.v, o.key_mask = inp.q, inp.k, inp.v, None
    return o


# ------------------------------------------------------------------------------------------ full size, sampled rows
def test_full_size_lowres_e4m3_and_scatter_sampled_rows(B):
    """The low-resolution contract shape at full size: E4M3 output, and one rank's shard of a 4-way exchange with
    the scatter epilogue, on sampled rows of two heads against the oracle (same sampling as the bf16 parity test)."""
    w = wl.CONFIGS["lowres"]
    inp = wl.make_inputs(w, "cuda")
    attn = B.Attn3d.from_workload(w, "cuda")
    out8 = torch.full((w.total_tokens, w.heads, w.head_dim), 0x7F, dtype=torch.uint8, device="cuda")
    B.sol_attn3d_forward_e4m3(attn.plan, inp.q, inp.k, inp.v, out8, inp.key_mask)
    out16 = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert not bool((out8 == 0x7F).any()), "an output byte was never written"
    attn.close()
    qc, kc, vc = inp.q.cpu(), inp.k.cpu(), inp.v.cpu()
    select = [(0, h, torch.from_numpy(wl.sample_rows(w, 0, h, 1024))) for h in (0, 15, w.heads - 1)]
    refs = orc.attn3d_oracle(qc, kc, vc, seq_tuples(w), w.rope_dims, w.theta, None, select=select)
    for (_, h, rows), ref in zip(select, refs):
        idx = rows.cuda()
        print("head", h, check_e4m3(out8[idx, h], ref, out16[idx, h]))
    # rank 1 of a 4-way exchange: heads [10, 20) from a packed QKV buffer, rows scattered to four owners
    G, r = 4, 1
    hl = w.heads // G
    qkv = torch.stack((inp.q[:, r * hl:(r + 1) * hl], inp.k[:, r * hl:(r + 1) * hl], inp.v[:, r * hl:(r + 1) * hl]), dim=1).contiguous()
    st = (3 * hl * w.head_dim, w.head_dim)
    shard = B.Attn3d(seq_tuples(w), hl, w.head_dim, w.rope_dims, w.theta, "cuda", q_strides=st, k_strides=st, v_strides=st)
    ranges = xo.shard_ranges(w.total_tokens, G)
    owners = [torch.full((b - a, w.heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda") for (a, b) in ranges]
    B.sol_attn3d_forward_scatter(shard.plan, qkv[:, 0], qkv[:, 1], qkv[:, 2], None, [o.data_ptr() for o in owners],
                                 [a for a, _ in ranges] + [w.total_tokens], w.heads, r * hl)
    torch.cuda.synchronize()
    assert shard.status() == 0
    shard.close()
    got = torch.cat(owners, dim=0)
    # A 10-head plan puts the same (head, query block) in another wave of CTAs than the 40-head plan, and the order
    # in which a CTA walks the key tiles alternates per wave: same sums in another order, equal to rounding.
    a, b = got[:, r * hl:(r + 1) * hl].float(), out16[:, r * hl:(r + 1) * hl].float()
    assert float((a - b).abs().max()) <= 2.0 ** -7 * float(b.abs().max())
    assert float((a == b).float().mean()) > 0.4           # CTAs that walk in the same direction in both plans agree bit for bit
    for (_, h, rows), ref in zip(select, refs):
        if r * hl <= h < (r + 1) * hl:
            max_abs, rel_l2 = orc.compare(got[rows.cuda(), h].cpu(), ref)
            assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2
    assert bool(torch.isnan(got[:, :r * hl].float()).all()) and bool(torch.isnan(got[:, (r + 1) * hl:].float()).all()), \
        "the scatter epilogue wrote outside its head columns"


# ------------------------------------------------------------------------------------------ peer transport, the module's own code
@pytest.mark.parametrize("name,heads,G,fmt", [("lowres", 8, 4, "bf16"), ("varlen", 6, 3, "bf16"), ("cfg_batch", 8, 8, "bf16"),
                                              ("lowres", 8, 2, "e4m3"), ("lowres", 8, 4, "int8"), ("cfg_batch", 4, 2, "int8")])
def test_peer_transport_of_the_module_with_virtual_ranks(B, name, heads, G, fmt):
    """SequenceParallelAttn3d(transport="peer") with all ranks' buffers on this GPU (local_peer_buffers): every rank
    is an instance of the module, and the ranks run its three phases in turn -- all pack, all attend, all read --
    which is the order the barriers of a real run enforce.  Exercises the module's own pointer plumbing (token
    offsets, head offsets, buffer sizes by the largest shard, the slice returned).  Result: each rank's token rows of
    the single-device attention, bit for bit, and equal to the collective transport's kernels called by hand."""
    from paper_2609_35110_b200.sequence_parallel import SequenceParallelAttn3d, local_peer_buffers, shard_ranges
    w = replace(wl.shrunk(name), heads=heads)
    inp = wl.make_inputs(w, "cuda")
    out_dtype = torch.uint8 if fmt == "e4m3" else torch.bfloat16
    int8 = fmt == "int8"                                       # block-INT8 records both ways
    rb_q = B.sol_attn3d_exchange_record_bytes(B.WIRE_QKV_INT8, w.head_dim) if int8 else 0
    rb_o = B.sol_attn3d_exchange_record_bytes(B.WIRE_OUT_INT8, w.head_dim) if int8 else 0
    bufs = local_peer_buffers(w.total_tokens, heads, w.head_dim, G, out_dtype, "cuda", rb_q, rb_o)
    for pb in bufs:                                            # poison: an unwritten element shows
        pb.qkv.view(torch.uint8).fill_(0x7F)
        pb.merged.view(torch.uint8).fill_(0x7F)
    kw = {"qkv_wire": "int8"} if int8 else {}
    ranks = [SequenceParallelAttn3d(seq_tuples(w), heads, w.head_dim, w.rope_dims, w.theta, transport="peer", out_format=fmt,
                                    peer_buffers=bufs[r], **kw) for r in range(G)]
    ranges = shard_ranges(w.total_tokens, G)
    for r, (a, b) in enumerate(ranges):
        assert ranks[r].xp.n_local == b - a
        if b > a:
            ranks[r].peer_pack(inp.q[a:b], inp.k[a:b], inp.v[a:b])
    for r in range(G):
        ranks[r].peer_attend(inp.key_mask)
    torch.cuda.synchronize()
    for r in range(G):
        assert ranks[r].attn.status() == 0
    got = torch.cat([ranks[r].peer_result() for r in range(G)], dim=0)
    assert got.shape[0] == w.total_tokens
    if int8:
        # the same records, kernels and arithmetic as the pipeline called by hand: the same bytes
        by_hand, _ = int8_pipeline_by_hand(B, w, inp, G)
        assert torch.equal(got, torch.cat(by_hand, dim=0))
        for r in ranks:
            r.close()
        return
    single = B.Attn3d.from_workload(w, "cuda")
    if fmt == "e4m3":
        want = torch.empty((w.total_tokens, heads, w.head_dim), dtype=torch.uint8, device="cuda")
        B.sol_attn3d_forward_e4m3(single.plan, inp.q, inp.k, inp.v, want, inp.key_mask)
    else:
        want = single.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    single.close()
    assert torch.equal(got.view(torch.uint8), want.view(torch.uint8))
    by_hand = torch.cat(virtual_ranks_forward(B, w, inp, G, B.OUT_E4M3 if fmt == "e4m3" else B.OUT_BF16, False), dim=0)
    assert torch.equal(got.view(torch.uint8), by_hand.view(torch.uint8))
    if fmt == "bf16":
        max_abs, rel_l2 = orc.compare(got.cpu(), oracle_dense(w, inp))
        assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2
    # forward() of one rank in a one-rank "job" runs the same phases with its (no-op) barriers
    solo_buf = local_peer_buffers(w.total_tokens, heads, w.head_dim, 1, out_dtype, "cuda")[0]
    solo = SequenceParallelAttn3d(seq_tuples(w), heads, w.head_dim, w.rope_dims, w.theta, transport="peer", out_format=fmt,
                                  peer_buffers=solo_buf)
    got1 = solo.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    assert torch.equal(got1.view(torch.uint8), want.view(torch.uint8))
    solo.close()
    for r in ranks:
        r.close()


_PEER_ONE_RANK = r'''
import os, sys
sys.path.insert(0, os.getcwd())
import torch, torch.distributed as dist
from dataclasses import replace
from paper_2609_35110_b200 import binding as B, workloads as wl
from paper_2609_35110_b200.sequence_parallel import SequenceParallelAttn3d
dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
w = replace(wl.shrunk("cfg_batch"), heads=4)
inp = wl.make_inputs(w, "cuda")
seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
single = B.Attn3d.from_workload(w, "cuda")
want = single.forward(inp.q, inp.k, inp.v, inp.key_mask)
want8 = torch.empty(want.shape, dtype=torch.uint8, device="cuda")
B.sol_attn3d_forward_e4m3(single.plan, inp.q, inp.k, inp.v, want8, inp.key_mask)
for fmt, ref in (("bf16", want), ("e4m3", want8)):
    sp = SequenceParallelAttn3d(seqs, w.heads, w.head_dim, w.rope_dims, w.theta, transport="peer", out_format=fmt)
    assert sp.pb.qkv_peers[0] == sp.pb.qkv.data_ptr() and sp.pb.merged_peers[0] == sp.pb.merged.data_ptr()
    for _ in range(2):                                   # twice: the leading barrier protects the buffers of the last call
        got = sp.forward(inp.q, inp.k, inp.v, inp.key_mask)
        torch.cuda.synchronize()
        assert torch.equal(got.view(torch.uint8), ref.view(torch.uint8)), fmt
    assert sp.attn.status() == 0
    sp.close()
dist.destroy_process_group()
print("PEER_ONE_RANK_OK")
'''


def test_peer_transport_with_symmetric_memory_one_rank(B):
    """The real buffer provider of the peer transport: symmetric-memory allocation and rendezvous over an NCCL
    group, peer addresses from the handles, the three stream-ordered barriers.  One rank (this run has one GPU), in a
    child process so that multicast binding is switched off for NCCL and for the symmetric-memory allocator before
    either initialises; the kernels use plain stores through the mapped addresses."""
    import subprocess
    import sys
    env = dict(os.environ, NCCL_NVLS_ENABLE="0", TORCH_SYMM_MEM_DISABLE_MULTICAST="1", MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(29900 + os.getpid() % 90))
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-c", _PEER_ONE_RANK], cwd=root, env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and "PEER_ONE_RANK_OK" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]


# ------------------------------------------------------------------------------------------ wire formats fused into the neighbours
@pytest.mark.parametrize("name", ["tiny", "cfg_batch", "varlen"])
def test_int8_epilogue_equals_quantising_the_bf16_rows(B, name):
    """sol_attn3d_forward_int8: the attention epilogue writes the output records itself.  Byte for byte the records of
    the two-kernel path (bf16 rows, then the record kernel), and of the oracle's record rule applied to those rows;
    the rows are pinned against the attention oracle."""
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    D = w.head_dim
    rb = B.sol_attn3d_exchange_record_bytes(B.WIRE_OUT_INT8, D)
    attn = B.Attn3d.from_workload(w, "cuda")
    rows = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
    two = torch.empty((w.total_tokens, w.heads, rb), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_quantize_out_int8(rows, two)
    fused = torch.full((w.total_tokens + 2, w.heads, rb), 0xAB, dtype=torch.uint8, device="cuda")   # guard rows around
    B.sol_attn3d_forward_int8(attn.plan, inp.q, inp.k, inp.v, fused[1:-1], inp.key_mask)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert bool((fused[0] == 0xAB).all()) and bool((fused[-1] == 0xAB).all())
    assert torch.equal(fused[1:-1], two)
    assert torch.equal(fused[1:-1].cpu(), xo.out_records(rows.cpu()))
    ma, rl = orc.compare(rows.cpu(), oracle_dense(w, inp))
    assert ma <= TOL_MAX_ABS and rl <= TOL_REL_L2
    # scattered to three owners at a head offset, records
    total = w.total_tokens
    tb = [0, total // 3, total // 3, total]
    owners = [torch.full((max(tb[g + 1] - tb[g], 1), w.heads + 1, rb), 0xCD, dtype=torch.uint8, device="cuda") for g in range(3)]
    B.sol_attn3d_forward_scatter(attn.plan, inp.q, inp.k, inp.v, inp.key_mask, [o.data_ptr() for o in owners], tb,
                                 w.heads + 1, 1, B.OUT_INT8)
    torch.cuda.synchronize()
    got = torch.cat([owners[g][: tb[g + 1] - tb[g], 1:] for g in range(3)])
    assert torch.equal(got, two)
    assert all(bool((owners[g][:, 0] == 0xCD).all()) for g in range(3))
    attn.close()


def test_int8_epilogue_writes_zero_records_for_a_sequence_without_keys(B):
    w = wl.Workload(name="dead", seqs=(wl.SeqSpec(40, 0, 1, 1), wl.SeqSpec(3, 2, 5, 7)), heads=2, head_dim=128,
                    rope_dims=(32, 48, 48), seed=11)
    inp = wl.make_inputs(w, "cuda")
    mask = torch.ones(w.total_tokens, dtype=torch.uint8, device="cuda")
    mask[40:] = 0
    attn = B.Attn3d.from_workload(w, "cuda")
    rows = attn.forward(inp.q, inp.k, inp.v, mask)
    rb = B.sol_attn3d_exchange_record_bytes(B.WIRE_OUT_INT8, 128)
    fused = torch.empty((w.total_tokens, w.heads, rb), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_forward_int8(attn.plan, inp.q, inp.k, inp.v, fused, mask)
    torch.cuda.synchronize()
    assert torch.equal(fused.cpu(), xo.out_records(rows.cpu()))
    attn.close()


@pytest.mark.parametrize("name,heads", [("tiny", 4), ("lowres", 5), ("cfg_batch", 2), ("varlen", 3)])
def test_qkv_int8_records_feed_the_attention_directly(B, name, heads):
    """sol_attn3d_forward_qkv_int8: the rotary producer dequantises the records itself.  Bit for bit the result of
    unpacking the records into a bf16 QKV tensor and running the plain forward on its views, for every output format;
    and within the attention tolerance of the oracle run on the oracle's own dequantisation of the oracle's records."""
    w = replace(wl.shrunk(name), heads=heads)
    inp = wl.make_inputs(w, "cuda")
    total, D = w.total_tokens, w.head_dim
    rb_in = B.sol_attn3d_exchange_record_bytes(B.WIRE_QKV_INT8, D)
    rb_out = B.sol_attn3d_exchange_record_bytes(B.WIRE_OUT_INT8, D)
    rec = torch.empty((total, heads, rb_in), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_pack_qkv_int8(inp.q, inp.k, inp.v, 1, [rec.data_ptr()], 0)
    torch.cuda.synchronize()
    assert torch.equal(rec.cpu(), xo.qkv_records(inp.q.cpu(), inp.k.cpu(), inp.v.cpu()))
    # two-kernel path
    qkv = torch.empty((total, 3, heads, D), dtype=torch.bfloat16, device="cuda")
    B.sol_attn3d_exchange_unpack_qkv_int8(rec, qkv, total, heads, D)
    st = (3 * heads * D, D)
    a2 = B.Attn3d(seq_tuples(w), heads, D, w.rope_dims, w.theta, "cuda", q_strides=st, k_strides=st, v_strides=st)
    want = a2.forward(qkv[:, 0], qkv[:, 1], qkv[:, 2], inp.key_mask)
    want8 = torch.empty(want.shape, dtype=torch.uint8, device="cuda")
    B.sol_attn3d_forward_e4m3(a2.plan, qkv[:, 0], qkv[:, 1], qkv[:, 2], want8, inp.key_mask)
    wantr = torch.empty((total, heads, rb_out), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_exchange_quantize_out_int8(want, wantr)
    # fused path, on a plan with the default strides (the records carry their own layout)
    attn = B.Attn3d.from_workload(w, "cuda")
    v_scratch = torch.full((total, heads, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    got = torch.full_like(want, float("nan"))
    B.sol_attn3d_forward_qkv_int8(attn.plan, rec, v_scratch, got, inp.key_mask, B.OUT_BF16)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert torch.equal(v_scratch, qkv[:, 2])
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    got8 = torch.empty_like(want8)
    B.sol_attn3d_forward_qkv_int8(attn.plan, rec, v_scratch, got8, inp.key_mask, B.OUT_E4M3)
    gotr = torch.empty_like(wantr)
    B.sol_attn3d_forward_qkv_int8(attn.plan, rec, v_scratch, gotr, inp.key_mask, B.OUT_INT8)
    torch.cuda.synchronize()
    assert torch.equal(got8, want8) and torch.equal(gotr, wantr)
    # the plain forward still works on the same plan afterwards (the cached V map is re-encoded)
    plain = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    ma, rl = orc.compare(plain.cpu(), oracle_dense(w, inp))
    assert ma <= TOL_MAX_ABS and rl <= TOL_REL_L2
    # oracle: its own records, its own dequantisation (rounded to bf16 as the wire tensor would be), its attention
    dq = [x.to(torch.bfloat16) for x in xo.qkv_from_records(xo.qkv_records(inp.q.cpu(), inp.k.cpu(), inp.v.cpu()), D)]
    ref = orc.attn3d_oracle(dq[0], dq[1], dq[2], seq_tuples(w), w.rope_dims, w.theta,
                            None if inp.key_mask is None else inp.key_mask.cpu())
    ma, rl = orc.compare(got.cpu(), ref)
    assert ma <= TOL_MAX_ABS and rl <= TOL_REL_L2, (ma, rl)
    attn.close(); a2.close()
