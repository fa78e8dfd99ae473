"""More shapes through the same parity check: head_dim 64 with prefix / mask / packing, the plain batch
plan entry, many short sequences, a single head, sequences shorter than one tile."""
import pytest
import torch

from oracle import attn3d_oracle as orc
from paper_2609_35110_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _check(B, w, inp, attn=None):
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
    own = attn is None
    if own:
        attn = B.Attn3d.from_workload(w, "cuda")
    out = torch.full((w.total_tokens, w.heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.sol_attn3d_forward(attn.plan, inp.q, inp.k, inp.v, out, inp.key_mask)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert not bool(torch.isnan(out.float()).any())
    ref = orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seqs, w.rope_dims, w.theta,
                            None if inp.key_mask is None else inp.key_mask.cpu())
    max_abs, rel_l2 = orc.compare(out.cpu(), ref)
    assert max_abs <= 2e-2 and rel_l2 <= 5e-3, (w.name, max_abs, rel_l2)
    if own:
        attn.close()
    return out


def test_head_dim_64_with_prefix_mask_and_packing():
    from paper_2609_35110_b200 import binding as B
    w = wl.Workload(name="d64", seqs=(wl.SeqSpec(100, 3, 7, 9), wl.SeqSpec(64, 5, 6, 11), wl.SeqSpec(0, 1, 5, 5)),
                    heads=5, head_dim=64, rope_dims=(16, 24, 16), seed=31, valid_text=(37, 64, 0))
    _check(B, w, wl.make_inputs(w, "cuda"))


def test_plain_batch_plan_entry():
    from paper_2609_35110_b200 import binding as B
    w = wl.Workload(name="batch3", seqs=tuple(wl.SeqSpec(40, 2, 9, 14) for _ in range(3)), heads=2, head_dim=128,
                    rope_dims=(32, 48, 48), seed=32)
    inp = wl.make_inputs(w, "cuda")
    plan = B.sol_attn3d_plan(3, 2, 128, 2, 9, 14, 40, (32, 48, 48))
    assert B.sol_attn3d_cu_seqlens(plan) == w.cu_seqlens
    ws = torch.empty(B.sol_attn3d_workspace_bytes(plan), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_set_workspace(plan, ws)

    class Holder:                      # same surface as Attn3d for _check
        pass
    h = Holder()
    h.plan = plan
    h.status = lambda: B.sol_attn3d_status(plan)
    # [B, N, heads, D] contiguous is the same memory as the packed [B*N, heads, D]
    _check(B, w, inp, attn=h)
    B.sol_attn3d_destroy(plan)


def test_many_short_sequences_and_single_head():
    from paper_2609_35110_b200 import binding as B
    seqs = tuple(wl.SeqSpec(i % 5, 1 + i % 3, 2 + i % 4, 3 + i % 7) for i in range(24))     # 6 .. 130 tokens each
    w = wl.Workload(name="many", seqs=seqs, heads=1, head_dim=128, rope_dims=(32, 48, 48), seed=33)
    _check(B, w, wl.make_inputs(w, "cuda"))


def test_exactly_one_and_two_tiles_and_partial_rope_d128():
    from paper_2609_35110_b200 import binding as B
    for n_h, n_w in ((8, 16), (16, 16), (16, 17)):                 # 128, 256 and 272 tokens
        w = wl.Workload(name="edge", seqs=(wl.SeqSpec(0, 1, n_h, n_w),), heads=2, head_dim=128,
                        rope_dims=(0, 40, 24), seed=34)
        _check(B, w, wl.make_inputs(w, "cuda"))


def test_forward_can_be_captured_in_a_cuda_graph_and_replayed():
    """The forward enqueues kernels only (no allocation, no synchronisation), so it can be stream-captured once
    and replayed; replays see the tensors' current contents."""
    from paper_2609_35110_b200 import binding as B
    from paper_2609_35110_b200 import workloads as wl
    w = wl.shrunk("cfg_batch")
    inp = wl.make_inputs(w, "cuda")
    attn = B.Attn3d.from_workload(w, "cuda")
    want = attn.forward(inp.q, inp.k, inp.v, inp.key_mask).clone()       # also builds the TMA map of V outside the capture
    out = torch.zeros_like(want)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=s):
        B.sol_attn3d_forward(attn.plan, inp.q, inp.k, inp.v, out, inp.key_mask, stream=torch.cuda.current_stream())
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, want) and attn.status() == 0
    # new contents, same addresses: the replay recomputes
    inp.v.mul_(2.0)
    want2 = attn.forward(inp.q, inp.k, inp.v, inp.key_mask).clone()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, want2) and not torch.equal(want2, want)
    attn.close()


def test_one_very_long_sequence_sampled_rows():
    """262,181 tokens (2,049 key tiles, ragged tail of 37) with one head: index arithmetic far beyond the contract
    sizes (token offsets x strides, tile counts, TMA coordinates), checked on sampled rows."""
    from paper_2609_35110_b200 import binding as B
    w = wl.Workload(name="long", seqs=(wl.SeqSpec(37, 64, 64, 64),), heads=1, head_dim=128, rope_dims=(32, 48, 48), seed=77)
    assert w.total_tokens == 262181
    inp = wl.make_inputs(w, "cuda")
    attn = B.Attn3d.from_workload(w, "cuda")
    out = torch.full((w.total_tokens, 1, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.sol_attn3d_forward(attn.plan, inp.q, inp.k, inp.v, out, None)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert not bool(torch.isnan(out.float()).any())
    rows = torch.from_numpy(wl.sample_rows(w, 0, 0, 256))
    assert int(rows[0]) == 0 and int(rows[-1]) == w.total_tokens - 1
    ref = orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), [(37, 64, 64, 64)], w.rope_dims, w.theta, None,
                            select=[(0, 0, rows)])[0]
    max_abs, rel_l2 = orc.compare(out[rows.cuda(), 0].cpu(), ref)
    print("long:", max_abs, rel_l2)
    assert max_abs <= 2e-2 and rel_l2 <= 5e-3
    attn.close()


def test_tensors_beyond_four_gib_sampled_groups():
    """32 sequences of 4,352 tokens with 128 heads: every one of Q, K, V and the output is 4.56 GB, so byte offsets pass
    2^32 (and element offsets 2^31) in the rotary producer, in the TMA coordinates times strides, and in the epilogue's row
    addresses.  Whole (sequence, head) groups are checked against the oracle, the last one in memory among them."""
    from paper_2609_35110_b200 import binding as B
    spec = wl.SeqSpec(256, 16, 16, 16)
    w = wl.Workload(name="big", seqs=(spec,) * 32, heads=128, head_dim=128, rope_dims=(32, 48, 48), seed=91)
    n_seq = 256 + 16 * 16 * 16
    assert w.total_tokens == 32 * n_seq and w.total_tokens * 128 * 128 * 2 > (1 << 32)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed)
    shape = (w.total_tokens, w.heads, w.head_dim)
    q, k, v = (torch.randn(shape, generator=gen, device="cuda", dtype=torch.bfloat16) for _ in range(3))
    attn = B.Attn3d.from_workload(w, "cuda")
    out = torch.full(shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    B.sol_attn3d_forward(attn.plan, q, k, v, out, None)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert not bool(torch.isnan(out[-n_seq:].float()).any()) and not bool(torch.isnan(out[:n_seq].float()).any())
    for s, h in [(0, 0), (15, 127), (16, 0), (31, 64), (31, 127)]:
        sl = slice(s * n_seq, (s + 1) * n_seq)
        ref = orc.attn3d_oracle(q[sl, h:h + 1].cpu(), k[sl, h:h + 1].cpu(), v[sl, h:h + 1].cpu(), [(256, 16, 16, 16)],
                                w.rope_dims, w.theta, None)
        max_abs, rel_l2 = orc.compare(out[sl, h:h + 1].cpu(), ref)
        assert max_abs <= 2e-2 and rel_l2 <= 5e-3, (s, h, max_abs, rel_l2)
    attn.close()
