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


# Block sizes of sol_attn3d_forward_sparse as its header documents them; the oracle takes them as arguments.
QBLK, KBLK = 256, 128


def _decision_band(q_rot, k_rot, D, tau):
    """How far from its threshold a block score must be for the GPU's decision to be comparable with the oracle's.

    The oracle takes the block statistic in fp64 on the un-rounded rotated operands; the kernel pools the bf16
    operands it has (each element off by a relative error of at most 2^-9, independent from element to element)
    in fp32.  Per element that is a zero-mean error of variance <= (2^-9 x)^2 / 3; the pooled means and the score
    are linear in those errors, so the score's standard deviation follows in closed form.  A decision is compared
    when the score is more than 6 such standard deviations (its own, plus the threshold's: mu and sigma are
    averages of scores of the same row) plus fp32 summation slack away from the threshold.
    """
    n = q_rot.shape[0]
    nq, nk = (n + QBLK - 1) // QBLK, (n + KBLK - 1) // KBLK
    u2 = (2.0 ** -9) ** 2 / 3.0

    def pooled(x, blk, nb):
        mean = torch.stack([x[i * blk: min(n, (i + 1) * blk)].mean(0) for i in range(nb)])
        var = torch.stack([(x[i * blk: min(n, (i + 1) * blk)] ** 2).sum(0) / float(min(n, (i + 1) * blk) - i * blk) ** 2
                           for i in range(nb)]) * u2
        return mean, var

    qm, qv = pooled(q_rot, QBLK, nq)
    km, kv = pooled(k_rot, KBLK, nk)
    sd = torch.sqrt((qv @ (km ** 2).t() + (qm ** 2) @ kv.t()) / D)              # [nq, nk]
    sc = (qm @ km.t()) / D ** 0.5
    return 6.0 * (sd + (1.0 + abs(tau)) * sd.max(dim=1, keepdim=True).values) + 4e-6 * (1.0 + sc.abs())


def _compare_selection(gpu_sel, q_rot, k_rot, D, tau, text_len, valid):
    """(decisions compared, decisions that differ, blocks the GPU attends) for one (sequence, head)."""
    sc = orc.block_scores(q_rot, k_rot, D, QBLK, KBLK)
    want = orc.block_select(sc, tau, text_len, QBLK, KBLK)
    if valid is not None:                                  # key tiles without a valid key are never listed
        nk = want.shape[1]
        tile_has_key = torch.tensor([bool(valid[j * KBLK: (j + 1) * KBLK].any()) for j in range(nk)])
        want &= tile_has_key[None, :]
    mu = sc.mean(1, keepdim=True)
    sg = torch.sqrt(((sc - mu) ** 2).mean(1, keepdim=True))
    band = _decision_band(q_rot, k_rot, D, tau)
    clear = (sc - (mu + tau * sg)).abs() > band
    # the arg-max rail may pick another block when the two best scores are within rounding: unclear too
    if sc.shape[1] > 1:
        top2 = sc.topk(2, dim=1).values
        tie = (top2[:, :1] - top2[:, 1:2]) <= 2.0 * band.max(dim=1, keepdim=True).values
        clear &= ~(tie & (sc >= top2[:, 1:2]))
    return int(clear.sum()), int((gpu_sel != want)[clear].sum()), int(gpu_sel.sum()), int(clear.numel())


@pytest.mark.parametrize("name,tau", [("highres", 1.0), ("highres", 1.5), ("varlen", 1.25), ("cfg_batch", 1.0)])
def test_sparse_forward_matches_oracle(name, tau):
    from paper_2609_35110_b200 import binding as B
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
    attn, sws, out = _run_sparse(B, w, inp, tau)
    gpu_sel = _gpu_selection(B, attn, sws, w)
    mask = None if inp.key_mask is None else inp.key_mask.cpu()
    # (1) the selection rule: identical wherever the score is not within rounding of the threshold
    n_clear = n_diff = n_on = n_all = 0
    cu = w.cu_seqlens
    for s, sq in enumerate(w.seqs):
        valid = None if mask is None else (mask[cu[s]: cu[s + 1]] != 0)
        q_rot = orc.rope_oracle(inp.q[cu[s]: cu[s + 1]].cpu(), [seqs[s]], w.rope_dims, w.theta)
        k_rot = orc.rope_oracle(inp.k[cu[s]: cu[s + 1]].cpu(), [seqs[s]], w.rope_dims, w.theta)
        for h in range(w.heads):
            c, d, on, al = _compare_selection(gpu_sel[s][h], q_rot[:, h], k_rot[:, h], w.head_dim, tau, sq.text_len, valid)
            n_clear += c; n_diff += d; n_on += on; n_all += al
    assert n_diff == 0, f"{n_diff} block decisions differ from the rule"
    assert n_clear >= 0.8 * n_all, (n_clear, n_all)        # the comparison is not vacuous
    sel_tiles, all_tiles = B.sol_attn3d_sparse_stats(attn.plan, sws)
    assert sel_tiles == n_on and all_tiles >= n_on
    # (2) the attention arithmetic on the GPU's selection
    ref, _, _ = orc.attn3d_sparse_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seqs, w.rope_dims, w.theta, tau, QBLK, KBLK,
                                         mask, selection=gpu_sel)
    assert not bool(torch.isnan(out.float()).any())
    max_abs, rel_l2 = orc.compare(out.cpu(), ref)
    print(f"{w.name} tau={tau}: density={sel_tiles / all_tiles:.3f} compared={n_clear}/{n_all} "
          f"max_abs={max_abs:.3e} rel_l2={rel_l2:.3e}")
    assert max_abs <= 2e-2 and rel_l2 <= 5e-3
    assert sel_tiles < all_tiles                          # something was actually skipped
    attn.close()


@pytest.mark.parametrize("tau", [1.0, 1.5])
def test_sparse_full_size_low_resolution_stage(tau):
    """The low-resolution-stage shape at full size: 25,216 tokens = 99 query blocks x 197 KV blocks per head, 40 heads.
    The selection of three heads is read back and compared with the rule; sampled rows of those heads are compared
    with the oracle's attention over the blocks the GPU selected."""
    from paper_2609_35110_b200 import binding as B
    w = wl.CONFIGS["lowres"]
    inp = wl.make_inputs(w, "cuda")
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
    sq = w.seqs[0]
    nq, nk = (sq.n_tokens + QBLK - 1) // QBLK, (sq.n_tokens + KBLK - 1) // KBLK
    assert (nq, nk) == (99, 197)
    attn, sws, out = _run_sparse(B, w, inp, tau)
    sel_tiles, all_tiles = B.sol_attn3d_sparse_stats(attn.plan, sws)
    assert all_tiles == w.heads * nq * nk and 0 < sel_tiles < all_tiles
    assert not bool(torch.isnan(out.float()).any())
    heads = [0, 17, w.heads - 1]
    q, k, v, o = inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), out.cpu()
    n_clear = n_diff = n_all = 0
    picked, select = [], []
    for h in heads:
        m = torch.zeros(nq, nk, dtype=torch.bool)
        for i in range(nq):
            lst = B.sol_attn3d_sparse_selection(attn.plan, sws, 0, h, i, nk)
            assert lst == sorted(set(lst)) and all(0 <= j < nk for j in lst)      # ascending, no duplicates
            m[i, lst] = True
        q_rot = orc.rope_oracle(q[:, h: h + 1], seqs, w.rope_dims, w.theta)[:, 0]
        k_rot = orc.rope_oracle(k[:, h: h + 1], seqs, w.rope_dims, w.theta)[:, 0]
        c, d, _, al = _compare_selection(m, q_rot, k_rot, w.head_dim, tau, sq.text_len, None)
        n_clear += c; n_diff += d; n_all += al
        assert bool(m[0].all()) and bool(m[:, :2].all())       # rails: prefix query block dense, prefix KV blocks on
        picked.append(m)
        select.append((0, h, torch.from_numpy(wl.sample_rows(w, 0, h, 384))))
    assert n_diff == 0, f"{n_diff} of {n_clear} compared block decisions differ from the rule"
    assert n_clear >= 0.9 * n_all, (n_clear, n_all)
    ref, _, _ = orc.attn3d_sparse_oracle(q, k, v, seqs, w.rope_dims, w.theta, tau, QBLK, KBLK, None,
                                         selection=picked, select=select)
    got = torch.cat([o[rows, h] for (_, h, rows) in select])
    max_abs, rel_l2 = orc.compare(got, torch.cat(ref))
    print(f"lowres full size tau={tau}: density={sel_tiles / all_tiles:.3f} compared={n_clear}/{n_all} "
          f"max_abs={max_abs:.3e} rel_l2={rel_l2:.3e}")
    assert max_abs <= 2e-2 and rel_l2 <= 5e-3
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
