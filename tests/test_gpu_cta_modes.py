"""The two launch modes of the attention kernel at head_dim 128.  By default two CTAs on neighbouring SMs form a pair
that covers 512 query rows: each loads half of every K / V tile and one tcgen05.mma.cta_group::2 of M = 256 works on
both.  SOL_ATTN3D_PAIR=0 (read when a plan is built) keeps the plan on single CTAs of 256 rows, which is also what
the block-sparse variant and head_dim 64 always use.  Both modes get the same parity bar here, on the paths where
they differ: odd and even numbers of 256-row blocks, head ranges, rectangular mode, key masks, the moving softmax
reference, scatter and E4M3 epilogues, and the bounded-wait failure path."""
from dataclasses import replace

import pytest
import torch

from oracle import attn3d_oracle as orc
from paper_2609_35110_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_MAX_ABS = 2e-2
TOL_REL_L2 = 5e-3


@pytest.fixture(params=["pair", "single"])
def PB(request, monkeypatch):
    from paper_2609_35110_b200 import binding
    binding._lib()
    monkeypatch.setenv("SOL_ATTN3D_PAIR", "1" if request.param == "pair" else "0")   # read when a plan is built
    return binding


def _seqs(w):
    return [(s.text_len, s.T, s.H, s.W) for s in w.seqs]


def _oracle(w, inp):
    return orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), _seqs(w), w.rope_dims, w.theta,
                             None if inp.key_mask is None else inp.key_mask.cpu())


@pytest.mark.parametrize("name", ["lowres", "highres", "cfg_batch", "varlen"])
def test_mode_matches_oracle_all_rows(PB, name):
    w = wl.shrunk(name)                                   # 620 / 1156 / 2 x 944 / ragged tokens: odd and even block counts
    inp = wl.make_inputs(w, "cuda")
    attn = PB.Attn3d.from_workload(w, "cuda")
    out = torch.full((w.total_tokens, w.heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    attn.forward(inp.q, inp.k, inp.v, inp.key_mask, out=out)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert not bool(torch.isnan(out.float()).any()), "a row was never written"
    ref = _oracle(w, inp)
    ma, rl = orc.compare(out.cpu(), ref)
    print(f"pair {w.name}: max_abs={ma:.3e} rel_l2={rl:.3e}")
    assert ma <= TOL_MAX_ABS and rl <= TOL_REL_L2
    cu = w.cu_seqlens
    for s in range(w.n_seqs):
        ma, rl = orc.compare(out[cu[s]:cu[s + 1]].cpu(), ref[cu[s]:cu[s + 1]])
        assert ma <= TOL_MAX_ABS and rl <= TOL_REL_L2, (s, ma, rl)
    attn.close()


def test_pair_mode_equals_single_ctas_to_rounding_and_is_deterministic(monkeypatch):
    from paper_2609_35110_b200 import binding as PB
    w = wl.shrunk("highres")
    inp = wl.make_inputs(w, "cuda")
    monkeypatch.setenv("SOL_ATTN3D_PAIR", "1")
    pair = PB.Attn3d.from_workload(w, "cuda")
    a = pair.forward(inp.q, inp.k, inp.v).clone()
    b = pair.forward(inp.q, inp.k, inp.v)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    monkeypatch.setenv("SOL_ATTN3D_PAIR", "0")
    single = PB.Attn3d.from_workload(w, "cuda")
    c = single.forward(inp.q, inp.k, inp.v)
    torch.cuda.synchronize()
    # same products and the same key order inside a tile; the MMA of M = 256 may accumulate in another order
    ma, rl = orc.compare(a.cpu(), c.cpu().double())
    assert rl <= 2e-3 and ma <= 5e-3, (ma, rl)
    pair.close(); single.close()


@pytest.mark.parametrize("direction", ["rising", "falling"])
def test_mode_moving_reference(PB, direction):
    """The logit ramp of the lazy-rescale tests: every tile moves the reference, in both CTAs of every pair."""
    w = wl.Workload(name="ramp_pair", seqs=(wl.SeqSpec(256, 5, 9, 20),), heads=40, head_dim=128, rope_dims=(32, 48, 32), seed=31)
    inp = wl.make_inputs(w, "cuda")
    inp.v.mul_(0.25)
    n_tiles = (w.total_tokens + 127) // 128
    g = [10.0 * (t + 1) for t in range(n_tiles)]
    g = g if direction == "rising" else g[::-1]
    inp.q[:, :, 127] = 8.0
    for t in range(n_tiles):
        inp.k[128 * t: 128 * (t + 1), :, 127] = g[t]
    mask = torch.ones(w.total_tokens, dtype=torch.uint8, device="cuda")
    mask[128 * 3 + 9: 128 * 3 + 90] = 0
    attn = PB.Attn3d.from_workload(w, "cuda")
    before = PB.sol_attn3d_softmax_rescale_count(attn.plan)
    out = attn.forward(inp.q, inp.k, inp.v, mask)
    torch.cuda.synchronize()
    assert attn.status() == 0
    assert PB.sol_attn3d_softmax_rescale_count(attn.plan) - before > 0
    ref = orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), _seqs(w), w.rope_dims, w.theta, mask.cpu())
    ma, rl = orc.compare(out.cpu(), ref)
    assert ma <= TOL_MAX_ABS and rl <= TOL_REL_L2, (ma, rl)
    attn.close()


def test_mode_rect_scatter_e4m3_and_host_groups(PB):
    w = replace(wl.shrunk("cfg_batch"), heads=4)
    inp = wl.make_inputs(w, "cuda")
    attn = PB.Attn3d.from_workload(w, "cuda")
    dense = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    # rectangular: a 512-row block whose second half is unwanted, one that is wholly unwanted
    qmask = torch.ones(w.total_tokens, dtype=torch.uint8, device="cuda")
    qmask[256:512] = 0
    qmask[944 + 512: 944 + 944] = 0
    out = torch.full_like(dense, 7.0)
    PB.sol_attn3d_forward_rect(attn.plan, inp.q, inp.k, inp.v, out, inp.key_mask, qmask)
    torch.cuda.synchronize()
    want = qmask.bool()
    assert torch.equal(out[want], dense[want]) and bool((out[~want] == 7.0).all())
    # scatter to three owners, bf16
    total = w.total_tokens
    tb = [0, 700, 701, total]
    owners = [torch.full((max(tb[g + 1] - tb[g], 1), w.heads + 2, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
              for g in range(3)]
    PB.sol_attn3d_forward_scatter(attn.plan, inp.q, inp.k, inp.v, inp.key_mask, [o.data_ptr() for o in owners], tb,
                                  w.heads + 2, 1)
    torch.cuda.synchronize()
    got = torch.cat([owners[g][: tb[g + 1] - tb[g], 1: 1 + w.heads] for g in range(3)])
    assert torch.equal(got, dense)
    # E4M3 epilogue equals the single-CTA kernel's bytes wherever the bf16 outputs agree
    o8 = torch.empty(dense.shape, dtype=torch.uint8, device="cuda")
    PB.sol_attn3d_forward_e4m3(attn.plan, inp.q, inp.k, inp.v, o8, inp.key_mask)
    torch.cuda.synchronize()
    dec = o8.view(torch.float8_e4m3fn).float()
    assert float((dec - dense.float()).abs().max()) <= 0.07 * float(dense.float().abs().max()) + 1e-3
    # host-buffer forward in head groups (head-range launches of the pair kernel): bit-identical to the device forward
    hq, hk, hv = (t.cpu().pin_memory() for t in (inp.q, inp.k, inp.v))
    hm = inp.key_mask.cpu().pin_memory()
    hout = torch.empty(dense.shape, dtype=dense.dtype).pin_memory()
    staging = torch.empty(PB.sol_attn3d_host_staging_bytes(attn.plan), dtype=torch.uint8, device="cuda")
    PB.sol_attn3d_forward_host(attn.plan, hq, hk, hv, hout, hm, staging, 3)
    torch.cuda.synchronize()
    assert torch.equal(hout, dense.cpu())
    assert attn.status() == 0
    attn.close()


def test_mode_withheld_signal_times_out_and_context_survives(PB, monkeypatch):
    """The failure path at head_dim 128: the MMA issuer of work item 0 withholds one "S is ready" signal; the waits that
    depend on it (of BOTH CTAs of a pair) run out, everyone meets at the final barrier, the kernel returns and reports."""
    w = wl.shrunk("highres")
    inp = wl.make_inputs(w, "cuda")
    monkeypatch.setenv("SOL_ATTN3D_WAIT_LIMIT_MS", "20")
    monkeypatch.setenv("SOL_ATTN3D_FAULT_INJECT", "1")
    bad = PB.Attn3d.from_workload(w, "cuda")
    monkeypatch.delenv("SOL_ATTN3D_FAULT_INJECT")
    monkeypatch.delenv("SOL_ATTN3D_WAIT_LIMIT_MS")
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    bad.forward(inp.q, inp.k, inp.v)
    t1.record()
    torch.cuda.synchronize()
    assert t0.elapsed_time(t1) < 3000.0
    assert bad.status() == PB.ERR_DEVICE_TIMEOUT
    bad.close()
    good = PB.Attn3d.from_workload(w, "cuda")
    out = good.forward(inp.q, inp.k, inp.v)
    torch.cuda.synchronize()
    assert good.status() == 0
    ma, rl = orc.compare(out.cpu(), _oracle(w, inp))
    assert ma <= TOL_MAX_ABS and rl <= TOL_REL_L2
    good.close()
