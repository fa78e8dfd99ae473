"""GPU parity of the QK-norm + RoPE producer (fusion group (2) of Section 3.5) and of the forward that
uses it, against the fp64 oracle."""
import pytest
import torch

from oracle import attn3d_oracle as orc
from paper_2609_35110_b200 import workloads as wl

pytestmark = pytest.mark.gpu

EPS = 1e-6


def _gains(D, seed):
    g = torch.Generator().manual_seed(seed)
    gq = (1.0 + 0.3 * torch.randn(D, generator=g)).float()
    gk = (0.5 + 0.2 * torch.randn(D, generator=g)).float()
    return gq, gk


@pytest.mark.parametrize("name", ["tiny", "lowres", "cfg_batch", "varlen"])
def test_producer_matches_oracle(name):
    from paper_2609_35110_b200 import binding as B
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
    gq, gk = _gains(w.head_dim, 7)
    attn = B.Attn3d.from_workload(w, "cuda")
    q_out = torch.empty_like(inp.q)
    k_out = torch.empty_like(inp.k)
    B.sol_attn3d_qknorm_rope(attn.plan, inp.q, inp.k, gq.cuda(), gk.cuda(), EPS, q_out, k_out)
    torch.cuda.synchronize()
    for got, x, g in ((q_out, inp.q, gq), (k_out, inp.k, gk)):
        ref = orc.rope_oracle(x.cpu(), seqs, w.rope_dims, w.theta, gain=g, norm_eps=EPS)
        gcpu = got.cpu()
        assert float((gcpu == ref.to(torch.bfloat16)).double().mean()) > 0.995
        err = (gcpu.double() - ref).abs()
        assert bool((err <= ref.abs() * 2.0 ** -7 + 1e-6).all())      # never more than one bf16 ulp away
    # only one tensor at a time is allowed too
    k_only = torch.empty_like(inp.k)
    B.sol_attn3d_qknorm_rope(attn.plan, None, inp.k, None, gk.cuda(), EPS, None, k_only)
    torch.cuda.synchronize()
    assert torch.equal(k_only, k_out)
    attn.close()


@pytest.mark.parametrize("name", ["tiny", "highres", "cfg_batch", "varlen"])
def test_forward_with_qknorm_matches_oracle(name):
    from paper_2609_35110_b200 import binding as B
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
    gq, gk = _gains(w.head_dim, 11)
    attn = B.Attn3d.from_workload(w, "cuda")
    out = torch.full((w.total_tokens, w.heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.sol_attn3d_forward_qknorm(attn.plan, inp.q, inp.k, inp.v, out, inp.key_mask, gq.cuda(), gk.cuda(), EPS)
    torch.cuda.synchronize()
    assert attn.status() == 0
    ref = orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seqs, w.rope_dims, w.theta,
                            None if inp.key_mask is None else inp.key_mask.cpu(), None,
                            q_gain=gq, k_gain=gk, norm_eps=EPS)
    max_abs, rel_l2 = orc.compare(out.cpu(), ref)
    print(f"{w.name} qknorm: max_abs={max_abs:.3e} rel_l2={rel_l2:.3e}")
    assert max_abs <= 2e-2 and rel_l2 <= 5e-3
    # the plain forward on the same plan afterwards is unaffected
    plain = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    ref0 = orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seqs, w.rope_dims, w.theta,
                             None if inp.key_mask is None else inp.key_mask.cpu())
    ma, rl = orc.compare(plain.cpu(), ref0)
    assert ma <= 2e-2 and rl <= 5e-3
    with pytest.raises(B.SolAttn3dError):
        B._check(B._lib().sol_attn3d_forward_qknorm(attn.plan, inp.q.data_ptr(), inp.k.data_ptr(), inp.v.data_ptr(),
                                                    out.data_ptr(), None, None, None, 1e-6, None), "null gains")
    attn.close()
