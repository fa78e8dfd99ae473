"""The forward variant for callers that may not allocate device memory.

Some callers of this library run where cudaMalloc is off limits (a plugin inside a framework that
owns all device memory, a real-time loop after start-up).  `sol_attn3d_forward_noalloc` serves them
with a scratch array built into the library instead of a caller workspace.  This file checks, through
the C-ABI binding, that it gives the same output as `sol_attn3d_forward` on two calls in a row (the
second call finds the first call's leftovers in the shared array, including those of a different
plan), and that plans beyond the 32 MiB limit are refused.  Collected last on purpose.
"""
import pytest
import torch

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
    for name in ("cfg_batch", "varlen"):          # key mask + padding; ragged packed batch
        w = wl.shrunk(name)
        inp = wl.make_inputs(w, "cuda")
        attn = B.Attn3d.from_workload(w, "cuda")  # existing entry point, caller-provided workspace
        ref = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
        torch.cuda.synchronize()
        assert attn.status() == 0
        cases.append((w, inp, attn, ref))

    status = torch.full((1,), 123, dtype=torch.int32, device="cuda")
    # two calls in a row per plan, interleaved with the other plan so that each call starts from
    # scratch contents written for a different problem
    for rep in range(2):
        for (w, inp, attn, ref) in cases:
            assert B.sol_attn3d_workspace_bytes(attn.plan) <= 32 << 20
            out = torch.full_like(ref, float("nan"))
            B.sol_attn3d_forward_noalloc(attn.plan, inp.q, inp.k, inp.v, out, inp.key_mask, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert not bool(torch.isnan(out.float()).any())
            max_abs, rel_l2 = _compare(out, ref)
            assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2, (w.name, rep, max_abs, rel_l2)
    # back-to-back on the same plan without a status word
    w, inp, attn, ref = cases[0]
    out1, out2 = torch.empty_like(ref), torch.empty_like(ref)
    B.sol_attn3d_forward_noalloc(attn.plan, inp.q, inp.k, inp.v, out1, inp.key_mask)
    B.sol_attn3d_forward_noalloc(attn.plan, inp.q, inp.k, inp.v, out2, inp.key_mask)
    torch.cuda.synchronize()
    for out in (out1, out2):
        max_abs, rel_l2 = _compare(out, ref)
        assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2
    # a plan without any bound workspace works too
    bare = B.Attn3d.from_workload(w, device=None)
    out3 = torch.empty_like(ref)
    B.sol_attn3d_forward_noalloc(bare.plan, inp.q, inp.k, inp.v, out3, inp.key_mask, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    max_abs, rel_l2 = _compare(out3, ref)
    assert max_abs <= TOL_MAX_ABS and rel_l2 <= TOL_REL_L2
    bare.close()
    for (_, _, attn, _) in cases:
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
