"""GPU checks of the block-sparse variant (Section 3.4): the selection against the oracle's rule wherever
the decision is not within rounding of the threshold, and the attention arithmetic against the oracle on
the very selection the GPU made."""
import pytest
import torch

from oracle import attn3d_oracle as orc
from paper_2609_35110_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _run_sparse(B, w, inp, tau):
    attn = B.Attn3d.from_workload(w, "cuda")
    sws = torch.empty(B.sol_attn3d_sparse_workspace_bytes(attn.plan), dtype=torch.uint8, device="cuda")
    out = torch.full((w.total_tokens, w.heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.sol_attn3d_forward_sparse(attn.plan, inp.q, inp.k, inp.v, out, inp.key_mask, tau, sws)
    torch.cuda.synchronize()
    assert attn.status() == 0
    return attn, sws, out


def _gpu_selection(B, attn, sws, w):
    sel = []
    for s, sq in enumerate(w.seqs):
        nq, nk = (sq.n_tokens + 255) // 256, (sq.n_tokens + 127) // 128
        per_head = []
        for h in range(w.heads):
            m = torch.zeros(nq, nk, dtype=torch.bool)
            for i in range(nq):
                m[i, B.sol_attn3d_sparse_selection(attn.plan, sws, s, h, i, nk)] = True
            per_head.append(m)
        sel.append(per_head)
    return sel


@pytest.mark.parametrize("name,tau", [("highres", 1.0), ("highres", 1.5), ("varlen", 1.25), ("cfg_batch", 1.0)])
def test_sparse_forward_matches_oracle(name, tau):
    from paper_2609_35110_b200 import binding as B
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
    attn, sws, out = _run_sparse(B, w, inp, tau)
    gpu_sel = _gpu_selection(B, attn, sws, w)
    mask = None if inp.key_mask is None else inp.key_mask.cpu()
    # (1) the oracle's own selection: identical wherever the score is not within rounding of the threshold
    _, ora_sel, scores = orc.attn3d_sparse_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seqs, w.rope_dims, w.theta, tau, mask)
    n_blocks = n_diff = n_on = 0
    for s, sq in enumerate(w.seqs):
        valid = None if mask is None else (mask[w.cu_seqlens[s]: w.cu_seqlens[s + 1]] != 0)
        for h in range(w.heads):
            sc = scores[s][h]
            mu = sc.mean(1, keepdim=True)
            sg = torch.sqrt(((sc - mu) ** 2).mean(1, keepdim=True))
            margin = (sc - (mu + tau * sg)).abs()
            want = ora_sel[s][h].clone()
            if valid is not None:                        # key tiles without a valid key are never listed
                nk = want.shape[1]
                tile_has_key = torch.tensor([bool(valid[j * 128: (j + 1) * 128].any()) for j in range(nk)])
                want &= tile_has_key[None, :]
            clear = margin > 1e-4 * (1.0 + sg)            # fp32 pooling / dot products vs fp64
            # the arg-max rail may pick another block only on an exact tie: treat near-ties as unclear too
            top2 = sc.topk(min(2, sc.shape[1]), dim=1).values
            if sc.shape[1] > 1:
                clear &= ((top2[:, :1] - top2[:, 1:2]) > 1e-5).expand_as(clear) | (sc < top2[:, :1])
            n_blocks += int(clear.numel())
            n_diff += int((gpu_sel[s][h] != want)[clear].sum())
            n_on += int(gpu_sel[s][h].sum())
    assert n_diff == 0, f"{n_diff} block decisions differ from the rule"
    sel_tiles, all_tiles = B.sol_attn3d_sparse_stats(attn.plan, sws)
    assert sel_tiles == n_on and all_tiles >= n_on
    # (2) the attention arithmetic on the GPU's selection
    ref, _, _ = orc.attn3d_sparse_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seqs, w.rope_dims, w.theta, tau, mask,
                                         selection=gpu_sel)
    assert not bool(torch.isnan(out.float()).any())
    max_abs, rel_l2 = orc.compare(out.cpu(), ref)
    print(f"{w.name} tau={tau}: density={sel_tiles / all_tiles:.3f} max_abs={max_abs:.3e} rel_l2={rel_l2:.3e}")
    assert max_abs <= 2e-2 and rel_l2 <= 5e-3
    assert sel_tiles < all_tiles                          # something was actually skipped
    attn.close()


def test_sparse_with_everything_selected_equals_dense_bitwise():
    from paper_2609_35110_b200 import binding as B
    w = wl.shrunk("highres")
    inp = wl.make_inputs(w, "cuda")
    attn, sws, out = _run_sparse(B, w, inp, -1.0e30)       # threshold below every score
    dense = attn.forward(inp.q, inp.k, inp.v)
    torch.cuda.synchronize()
    assert torch.equal(out, dense)
    a, b = B.sol_attn3d_sparse_stats(attn.plan, sws)
    assert a == b
    attn.close()
