"""GPU parity: the CUDA path (through the C-ABI binding) against the fp64 oracle, element by element
on the same seeded inputs.  Tolerances are the contract's: max-abs <= 2e-2 and relative L2 <= 5e-3."""
import os

import pytest
import torch

from oracle import attn3d_oracle as orc
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


def run_gpu(B, w, inp, poison=True):
    attn = B.Attn3d.from_workload(w, "cuda")
    # guard bands around the output catch out-of-bounds stores; NaN poison catches unwritten rows
    n = w.total_tokens * w.heads * w.head_dim
    guard = 4096
    buf = torch.full((n + 2 * guard,), float("nan") if poison else 0.0, dtype=torch.bfloat16, device="cuda")
    buf[:guard] = 7.0
    buf[-guard:] = 7.0
    out = buf[guard:guard + n].view(w.total_tokens, w.heads, w.head_dim)
    attn.forward(inp.q, inp.k, inp.v, inp.key_mask, out=out)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert bool((buf[:guard] == 7.0).all()) and bool((buf[-guard:] == 7.0).all()), "store outside the output tensor"
    attn.close()
    return out


def oracle_dense(w, inp):
    return orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seq_tuples(w), w.rope_dims, w.theta,
                             None if inp.key_mask is None else inp.key_mask.cpu())


# ------------------------------------------------------------------ rotary prologue alone
@pytest.mark.parametrize("name", wl.CONFIG_ORDER)
def test_rope_prologue_matches_oracle(B, name):
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    attn = B.Attn3d.from_workload(w, "cuda")
    q_rot, k_rot = attn.rope_qk(inp.q, inp.k)
    torch.cuda.synchronize()
    for got, x in ((q_rot, inp.q), (k_rot, inp.k)):
        ref = orc.rope_oracle(x.cpu(), seq_tuples(w), w.rope_dims, w.theta)
        ref_b = ref.to(torch.bfloat16)
        g = got.cpu()
        # fp32 rotation from fp32 tables vs fp64: equal after rounding except at rounding boundaries,
        # and never more than one bf16 ulp (2^-7 of the value's binade) away
        assert float((g == ref_b).double().mean()) > 0.999
        err = (g.double() - ref).abs()
        assert bool((err <= ref.abs() * 2.0 ** -7 + 1e-6).all())
    # prefix rows are copied bit for bit
    cu = w.cu_seqlens
    for s, sq in enumerate(w.seqs):
        if sq.text_len:
            assert torch.equal(q_rot[cu[s]:cu[s] + sq.text_len], inp.q[cu[s]:cu[s] + sq.text_len])
    attn.close()


# ------------------------------------------------------------------ whole path, small configs, all rows
@pytest.mark.parametrize("name", wl.CONFIG_ORDER)
def test_forward_matches_oracle_all_rows(B, name):
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    out = run_gpu(B, w, inp)
    assert not bool(torch.isnan(out.float()).any()), "a row was never written"
    ref = oracle_dense(w, inp)
    max_abs, rel_l2 = orc.compare(out.cpu(), ref)
    print(f"{w.name}: max_abs={max_abs:.3e} rel_l2={rel_l2:.3e}")
    assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2
    # per sequence as well (a sequence-local mistake must not hide in the joint norm)
    cu = w.cu_seqlens
    for s in range(w.n_seqs):
        ma, rl = orc.compare(out[cu[s]:cu[s + 1]].cpu(), ref[cu[s]:cu[s + 1]])
        assert ma <= TOL_MAX_ABS and rl <= TOL_REL_L2, (s, ma, rl)


def test_deterministic_and_stream_reuse(B):
    w = wl.shrunk("highres")
    inp = wl.make_inputs(w, "cuda")
    attn = B.Attn3d.from_workload(w, "cuda")
    a = attn.forward(inp.q, inp.k, inp.v).clone()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        b = attn.forward(inp.q, inp.k, inp.v, stream=s)
    s.synchronize()
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    assert attn.status() == 0
    attn.close()


# ------------------------------------------------------------------ closed forms on the GPU
def test_uniform_scores_give_mean_of_valid_v(B):
    w = wl.shrunk("cfg_batch")
    inp = wl.make_inputs(w, "cuda")
    inp.q.zero_()
    out = run_gpu(B, w, inp).cpu().double()
    cu = w.cu_seqlens
    mask = inp.key_mask.cpu() != 0
    for s in range(w.n_seqs):
        v = inp.v[cu[s]:cu[s + 1]].cpu().double()
        mean = v[mask[cu[s]:cu[s + 1]]].mean(0)
        err = (out[cu[s]:cu[s + 1]] - mean[None]).abs().max()
        # P = 1 exactly for every valid key, so only the bf16 rounding of the output remains
        assert float(err) <= float(mean.abs().max()) * 2.0 ** -8 + 1e-6


def test_one_hot_keys_reproduce_v_rows_exactly(B):
    # 2x4x4 grid, D = 64: token n owns pair plane n; q_n = k_n = c e_{2n} so P is the identity
    w = wl.Workload(name="onehot", seqs=(wl.SeqSpec(0, 2, 4, 4),), heads=2, head_dim=64, rope_dims=(16, 24, 24), seed=5)
    inp = wl.make_inputs(w, "cuda")
    q = torch.zeros_like(inp.q)
    for i in range(32):
        q[i, :, 2 * i] = 96.0          # c^2 / sqrt(64) = 1152 > 800
    out = run_gpu(B, w, wl.Inputs(q, q.clone(), inp.v, None))
    assert torch.equal(out, inp.v)


def test_masked_keys_do_not_matter_bitwise(B):
    w = wl.shrunk("cfg_batch")
    inp = wl.make_inputs(w, "cuda")
    a = run_gpu(B, w, inp).clone()
    dead = inp.key_mask == 0
    assert int(dead.sum()) == 512 - 77
    k2, v2 = inp.k.clone(), inp.v.clone()
    k2[dead] = 300.0
    v2[dead] = -1.0e4
    b = run_gpu(B, w, wl.Inputs(inp.q, k2, v2, inp.key_mask))
    assert torch.equal(a, b)


def test_padded_prefix_equals_unpadded_run(B):
    w = wl.shrunk("cfg_batch")
    inp = wl.make_inputs(w, "cuda")
    out = run_gpu(B, w, inp)
    n = w.seqs[1].n_tokens
    keep = torch.cat([torch.arange(77), torch.arange(512, n)]).cuda() + w.cu_seqlens[1]
    w2 = wl.Workload(name="tight", seqs=(wl.SeqSpec(77, 3, 9, 16),), heads=w.heads, head_dim=w.head_dim,
                     rope_dims=w.rope_dims)
    out2 = run_gpu(B, w2, wl.Inputs(inp.q[keep].contiguous(), inp.k[keep].contiguous(), inp.v[keep].contiguous(), None))
    # same math on differently tiled keys: equal up to the bf16 output rounding and accumulation order
    ma, rl = orc.compare(out[keep].cpu(), out2.cpu().double())
    assert rl <= 4e-3 and ma <= 5e-3


def test_packed_equals_separate_runs(B):
    w = wl.shrunk("varlen")
    inp = wl.make_inputs(w, "cuda")
    out = run_gpu(B, w, inp)
    cu = w.cu_seqlens
    for s, sq in enumerate(w.seqs):
        w1 = wl.Workload(name="one", seqs=(sq,), heads=w.heads, head_dim=w.head_dim, rope_dims=w.rope_dims)
        sl = slice(cu[s], cu[s + 1])
        o1 = run_gpu(B, w1, wl.Inputs(inp.q[sl].contiguous(), inp.k[sl].contiguous(), inp.v[sl].contiguous(), None))
        assert torch.equal(o1, out[sl]), f"sequence {s} differs between packed and separate runs"


def test_strided_views_of_a_packed_qkv_buffer(B):
    w = wl.shrunk("lowres")
    inp = wl.make_inputs(w, "cuda")
    qkv = torch.stack([inp.q, inp.k, inp.v], dim=1).contiguous()     # [tokens, 3, heads, D]
    q, k, v = qkv[:, 0], qkv[:, 1], qkv[:, 2]
    st = (3 * w.heads * w.head_dim, w.head_dim)
    attn = B.Attn3d(seq_tuples(w), w.heads, w.head_dim, w.rope_dims, w.theta, "cuda",
                    q_strides=st, k_strides=st, v_strides=st)
    out = attn.forward(q, k, v)
    torch.cuda.synchronize()
    assert attn.status() == 0
    ref = run_gpu(B, w, inp)
    assert torch.equal(out, ref)
    attn.close()


def test_all_keys_masked_gives_zeros_and_prefix_only_sequence(B):
    w = wl.Workload(name="dead", seqs=(wl.SeqSpec(40, 0, 1, 1), wl.SeqSpec(3, 2, 5, 7)), heads=2, head_dim=128,
                    rope_dims=(32, 48, 48), seed=11)
    inp = wl.make_inputs(w, "cuda")
    mask = torch.ones(w.total_tokens, dtype=torch.uint8, device="cuda")
    mask[40:] = 0                                                    # second sequence: no valid key at all
    out = run_gpu(B, w, wl.Inputs(inp.q, inp.k, inp.v, mask))
    assert bool((out[40:] == 0).all())
    ref = orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seq_tuples(w), w.rope_dims, w.theta, mask.cpu())
    ma, rl = orc.compare(out.cpu(), ref)
    assert ma <= TOL_MAX_ABS and rl <= TOL_REL_L2


def test_partial_rope_and_large_logits(B):
    # rotary on 8+16+8 of 64 dims; Q scaled x4 so that the running maximum moves a lot between tiles
    w = wl.Workload(name="partial", seqs=(wl.SeqSpec(7, 3, 11, 13),), heads=3, head_dim=64, rope_dims=(8, 16, 8), seed=21)
    inp = wl.make_inputs(w, "cuda")
    inp.q.mul_(4.0)
    out = run_gpu(B, w, inp)
    ref = oracle_dense(w, inp)
    ma, rl = orc.compare(out.cpu(), ref)
    print(f"partial/large logits: max_abs={ma:.3e} rel_l2={rl:.3e}")
    assert ma <= 5e-2 and rl <= 8e-3     # logits of std 4*sqrt(64)/8: bf16 operand rounding grows with |s|


# ------------------------------------------------------------------ full-size configs, sampled rows
def _rows_per_head(w):
    env = os.environ.get("SOL_PARITY_ROWS")
    return int(env) if env else w.rows_per_head


@pytest.mark.parametrize("name", ["lowres", "highres", "cfg_batch", "varlen"])
def test_full_size_sampled_rows(B, name):
    w = wl.CONFIGS[name]
    inp = wl.make_inputs(w, "cuda")
    out = run_gpu(B, w, inp, poison=False)
    cu = w.cu_seqlens
    q, k, v = inp.q.cpu(), inp.k.cpu(), inp.v.cpu()
    mask = None if inp.key_mask is None else inp.key_mask.cpu()
    o = out.cpu()
    del inp, out
    torch.cuda.empty_cache()
    num = den = 0.0
    worst = 0.0
    count = _rows_per_head(w)
    for s in range(w.n_seqs):
        for h in range(w.heads):
            rows = torch.from_numpy(wl.sample_rows(w, s, h, count))
            ref = orc.attn3d_oracle(q, k, v, seq_tuples(w), w.rope_dims, w.theta, mask, [(s, h, rows)])[0]
            d = o[cu[s] + rows, h].double() - ref
            num += float((d * d).sum())
            den += float((ref * ref).sum())
            worst = max(worst, float(d.abs().max()))
            # every (sequence, head) on its own as well
            assert float(d.abs().max()) <= TOL_MAX_ABS
            assert (float((d * d).sum()) / float((ref * ref).sum())) ** 0.5 <= TOL_REL_L2, (s, h)
    rel = (num / den) ** 0.5
    print(f"{w.name}: rows/(seq,head)={count} max_abs={worst:.3e} rel_l2={rel:.3e}")
    assert worst <= TOL_MAX_ABS and rel <= TOL_REL_L2
