"""GPU: sol_attn3d_forward_host (host buffers in, host buffer out, head groups pipelined on internal streams) must
give exactly the bytes of sol_attn3d_forward on device copies, and head-range launches must compose."""
import pytest
import torch

from oracle import attn3d_oracle as orc
from paper_2609_35110_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2609_35110_b200 import binding
    binding._lib()
    return binding


def seq_tuples(w):
    return [(s.text_len, s.T, s.H, s.W) for s in w.seqs]


@pytest.mark.parametrize("name,groups", [("tiny", 0), ("lowres", 2), ("cfg_batch", 0), ("varlen", 3), ("highres", 1), ("varlen", 8)])
def test_host_forward_equals_device_forward(B, name, groups):
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    attn = B.Attn3d.from_workload(w, "cuda")
    want = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    hq, hk, hv = (t.cpu().pin_memory() for t in (inp.q, inp.k, inp.v))
    hmask = None if inp.key_mask is None else inp.key_mask.cpu().pin_memory()
    hout = torch.full(want.shape, float("nan"), dtype=torch.bfloat16).pin_memory()
    staging = torch.empty(B.sol_attn3d_host_staging_bytes(attn.plan), dtype=torch.uint8, device="cuda")
    for rep in range(2):                                   # twice in a row: the staging buffers are reused
        hout.fill_(float("nan"))
        B.sol_attn3d_forward_host(attn.plan, hq, hk, hv, hout, hmask, staging, groups)
        torch.cuda.synchronize()
        assert attn.status() == 0
        assert torch.equal(hout.view(torch.int16), want.cpu().view(torch.int16)), f"rep {rep}"
    ref = orc.attn3d_oracle(hq, hk, hv, seq_tuples(w), w.rope_dims, w.theta, hmask)
    max_abs, rel_l2 = orc.compare(hout, ref)
    assert max_abs <= 2e-2 and rel_l2 <= 5e-3
    # a device forward of the same plan still works afterwards
    again = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    assert torch.equal(again, want)
    attn.close()


@pytest.mark.parametrize("name", ["varlen", "cfg_batch"])
def test_host_forward_as_the_first_call_of_a_plan(B, name):
    """Nothing has run on the plan before: the key-validity bits are built by the first head group's launch set on the
    caller's stream, and the second group's kernels, which run on an internal stream, must come after them."""
    w = wl.shrunk(name)
    inp = wl.make_inputs(w, "cuda")
    attn = B.Attn3d.from_workload(w, "cuda")
    hq, hk, hv = (t.cpu().pin_memory() for t in (inp.q, inp.k, inp.v))
    hmask = None if inp.key_mask is None else inp.key_mask.cpu().pin_memory()
    hout = torch.full(tuple(inp.q.shape), float("nan"), dtype=torch.bfloat16).pin_memory()
    staging = torch.empty(B.sol_attn3d_host_staging_bytes(attn.plan), dtype=torch.uint8, device="cuda")
    B.sol_attn3d_forward_host(attn.plan, hq, hk, hv, hout, hmask, staging, 0)
    torch.cuda.synchronize()
    assert attn.status() == 0
    want = attn.forward(inp.q, inp.k, inp.v, inp.key_mask)
    torch.cuda.synchronize()
    assert torch.equal(hout.view(torch.int16), want.cpu().view(torch.int16))
    attn.close()


def test_host_forward_rejects_bad_arguments(B):
    w = wl.shrunk("tiny")
    inp = wl.make_inputs(w, "cuda")
    attn = B.Attn3d.from_workload(w, "cuda")
    hq, hk, hv = (t.cpu().pin_memory() for t in (inp.q, inp.k, inp.v))
    hout = torch.empty_like(hq).pin_memory()
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SolAttn3dError):
        B.sol_attn3d_forward_host(attn.plan, hq, hk, hv, hout, None, small, 0)
    attn.close()
    D, H = w.head_dim, w.heads
    strided = B.Attn3d(seq_tuples(w), H, D, w.rope_dims, w.theta, "cuda", q_strides=(3 * H * D, D))
    staging = torch.empty(B.sol_attn3d_host_staging_bytes(strided.plan), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SolAttn3dError):
        B.sol_attn3d_forward_host(strided.plan, hq, hk, hv, hout, None, staging, 0)
    strided.close()
