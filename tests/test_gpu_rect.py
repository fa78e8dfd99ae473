"""Rectangular attention (fewer queries than keys), the shape that reference-KV caching produces: reference
query rows are skipped, every token still acts as a key."""
import pytest
import torch

from oracle import attn3d_oracle as orc
from paper_2609_35110_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["highres", "varlen", "cfg_batch"])
def test_rect_forward_computes_only_wanted_rows(name):
    from paper_2609_35110_b200 import binding as B
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
    # reference tokens = the first 60 % of each video (queries skipped); text and the rest are queries
    qmask = torch.ones(w.total_tokens, dtype=torch.uint8)
    cu = w.cu_seqlens
    for s, sq in enumerate(w.seqs):
        ref_tokens = int(0.6 * sq.n_video)
        qmask[cu[s] + sq.text_len: cu[s] + sq.text_len + ref_tokens] = 0
    attn = B.Attn3d.from_workload(w, "cuda")
    dense = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
    out = torch.full_like(dense, 7.0)
    B.sol_attn3d_forward_rect(attn.plan, inp.q, inp.k, inp.v, out, inp.key_mask, qmask.cuda())
    torch.cuda.synchronize()
    assert attn.status() == 0
    want = qmask.bool()
    assert torch.equal(out.cpu()[want], dense.cpu()[want])                 # wanted rows: bit-identical to dense
    assert bool((out.cpu()[~want] == 7.0).all())                           # skipped rows: never written
    # and against the oracle on the wanted rows
    sel = []
    for s in range(w.n_seqs):
        rows = torch.nonzero(want[cu[s]:cu[s + 1]]).flatten()
        for h in range(w.heads):
            sel.append((s, h, rows))
    ref = orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seqs, w.rope_dims, w.theta,
                            None if inp.key_mask is None else inp.key_mask.cpu(), sel)
    got = torch.cat([out.cpu()[cu[s] + rows, h] for (s, h, rows) in sel])
    max_abs, rel_l2 = orc.compare(got, torch.cat(ref))
    assert max_abs <= 2e-2 and rel_l2 <= 5e-3
    attn.close()


def test_rect_full_size_low_resolution_stage():
    """The low-resolution-stage shape at full size (25,216 tokens, 40 heads): the first 60 % of the video are
    reference tokens whose query rows are skipped (39 whole query blocks cost nothing, one is partial), plus a few
    scattered skipped rows elsewhere.  Wanted rows equal the dense forward bit for bit, skipped rows are never
    written, and sampled wanted rows match the oracle."""
    from paper_2609_35110_b200 import binding as B
    w = wl.CONFIGS["lowres"]
    inp = wl.make_inputs(w, "cuda")
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
    sq = w.seqs[0]
    qmask = torch.ones(w.total_tokens, dtype=torch.uint8)
    qmask[sq.text_len: sq.text_len + int(0.6 * sq.n_video)] = 0
    qmask[torch.arange(20000, 25216, 97)] = 0
    attn = B.Attn3d.from_workload(w, "cuda")
    dense = attn.forward(inp.q, inp.k, inp.v, None)
    out = torch.full_like(dense, 7.0)
    B.sol_attn3d_forward_rect(attn.plan, inp.q, inp.k, inp.v, out, None, qmask.cuda())
    torch.cuda.synchronize()
    assert attn.status() == 0
    want = qmask.bool().cuda()
    assert torch.equal(out[want], dense[want])
    assert bool((out[~want] == 7.0).all())
    o, q, k, v = out.cpu(), inp.q.cpu(), inp.k.cpu(), inp.v.cpu()
    sel = []
    for h in (0, 21, w.heads - 1):
        rows = torch.from_numpy(wl.sample_rows(w, 0, h, 512))
        sel.append((0, h, rows[qmask[rows].bool()]))
    ref = orc.attn3d_oracle(q, k, v, seqs, w.rope_dims, w.theta, None, sel)
    got = torch.cat([o[rows, h] for (_, h, rows) in sel])
    max_abs, rel_l2 = orc.compare(got, torch.cat(ref))
    assert max_abs <= 2e-2 and rel_l2 <= 5e-3
    attn.close()
