"""The forward variant for callers that may not allocate device memory.

Some callers of this library run where cudaMalloc is off limits (a plugin inside a framework that
owns all device memory, a real-time loop after start-up).  `sol_attn3d_forward_noalloc` serves them
with a scratch array built into the library instead of a caller workspace.  This file checks, through
the C-ABI binding, that it gives the same output as `sol_attn3d_forward` on two calls in a row (the
second call finds the first call's leftovers in the shared array, including those of a different
plan), that the output also agrees with the fp64 oracle, that calls after the first leave the amount of
free device memory unchanged, and that plans beyond the 32 MiB limit are refused.  Both entry points run
the same kernels on the same schedule, so beyond the tolerance the outputs are required to be equal bit
for bit.  Collected last on purpose.
"""
import pytest
import torch

from oracle import attn3d_oracle as orc
from paper_2609_35110_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_MAX_ABS = 2e-2
TOL_REL_L2 = 5e-3


def _compare(a, b):
    a, b = a.double(), b.double()
    d = a - b
    return float(d.abs().max()), float(torch.linalg.vector_norm(d) / torch.linalg.vector_norm(b))


def test_noalloc_forward_matches_workspace_forward_twice_in_a_row():
    from paper_2609_35110_b200 import binding as B

    cases = []
    for name in ("cfg_batch", "varlen", "tiny"):  # key mask + padding; ragged packed batch; head_dim 64
        w = wl.shrunk(name)
        inp = wl.make_inputs(w, "cuda")
        attn = B.Attn3d.from_workload(w, "cuda")  # existing entry point, caller-provided workspace
        ref = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
        torch.cuda.synchronize()
        assert attn.status() == 0
        seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
        exact = orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seqs, w.rope_dims, w.theta,
                                  None if inp.key_mask is None else inp.key_mask.cpu())
        cases.append((w, inp, attn, ref, exact))

    status = torch.full((1,), 123, dtype=torch.int32, device="cuda")
    # two calls in a row per plan, interleaved with the other plan so that each call starts from
    # scratch contents written for a different problem
    outs = [torch.empty_like(c[3]) for c in cases]  # allocated up front: the loop below must not change free memory
    free_after_first = None
    for rep in range(2):
        for (w, inp, attn, ref, exact), out in zip(cases, outs):
            assert B.sol_attn3d_workspace_bytes(attn.plan) <= 32 << 20
            out.fill_(float("nan"))
            B.sol_attn3d_forward_noalloc(attn.plan, inp.q, inp.k, inp.v, out, inp.key_mask, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert not bool(torch.isnan(out.float()).any())
            max_abs, rel_l2 = _compare(out, ref)
            assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2, (w.name, rep, max_abs, rel_l2)
            assert torch.equal(out, ref), (w.name, rep)          # same kernels, same schedule: same bits
            ma, rl = orc.compare(out.cpu(), exact)
            assert ma <= TOL_MAX_ABS and rl <= TOL_REL_L2, (w.name, rep, ma, rl)
            # the very first call may make the driver load the library's code and its built-in array; from then
            # on the entry point leaves the amount of free device memory alone
            free_now = torch.cuda.mem_get_info()[0]
            if free_after_first is None:
                free_after_first = free_now
            assert free_now == free_after_first, (w.name, rep, free_now, free_after_first)
    # back-to-back on the same plan without a status word
    w, inp, attn, ref, _ = cases[0]
    out1, out2 = torch.empty_like(ref), torch.empty_like(ref)
    B.sol_attn3d_forward_noalloc(attn.plan, inp.q, inp.k, inp.v, out1, inp.key_mask)
    B.sol_attn3d_forward_noalloc(attn.plan, inp.q, inp.k, inp.v, out2, inp.key_mask)
    torch.cuda.synchronize()
    for out in (out1, out2):
        max_abs, rel_l2 = _compare(out, ref)
        assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2
        assert torch.equal(out, ref)
    # a plan without any bound workspace works too
    bare = B.Attn3d.from_workload(w, device=None)
    out3 = torch.empty_like(ref)
    B.sol_attn3d_forward_noalloc(bare.plan, inp.q, inp.k, inp.v, out3, inp.key_mask, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    max_abs, rel_l2 = _compare(out3, ref)
    assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2
    assert torch.equal(out3, ref)
    bare.close()
    for (_, _, attn, _, _) in cases:
        attn.close()


def test_noalloc_refuses_plans_beyond_the_builtin_scratch():
    from paper_2609_35110_b200 import binding as B

    w = wl.CONFIGS["lowres"]                      # needs ~516 MB of scratch
    big = B.Attn3d.from_workload(w, device=None)
    assert B.sol_attn3d_workspace_bytes(big.plan) > 32 << 20
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.SolAttn3dError) as e:
        B.sol_attn3d_forward_noalloc(big.plan, x, x, x, y)      # refused before anything is enqueued
    assert e.value.code == B.ERR_SCRATCH_LIMIT
    big.close()
