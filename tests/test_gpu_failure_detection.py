"""Failure detection on the device: every wait inside the attention kernel is bounded.  A test hook makes
one CTA withhold a signal (nothing faults, traps or spins forever); the waits that depend on it run into
their limit, the kernel returns, the status word reports the time-out and the context stays usable."""
import os

import pytest
import torch

from oracle import attn3d_oracle as orc
from paper_2609_35110_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_withheld_signal_times_out_and_context_survives(monkeypatch):
    from paper_2609_35110_b200 import binding as B

    w = wl.shrunk("tiny")
    inp = wl.make_inputs(w, "cuda")
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]

    monkeypatch.setenv("SOL_ATTN3D_WAIT_LIMIT_MS", "20")
    monkeypatch.setenv("SOL_ATTN3D_FAULT_INJECT", "1")
    bad = B.Attn3d.from_workload(w, "cuda")                 # the plan reads the two variables when it is built
    monkeypatch.delenv("SOL_ATTN3D_FAULT_INJECT")
    monkeypatch.delenv("SOL_ATTN3D_WAIT_LIMIT_MS")

    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    bad.forward(inp.q, inp.k, inp.v)
    t1.record()
    torch.cuda.synchronize()                                # returns: no wait is unbounded
    assert t0.elapsed_time(t1) < 2000.0
    assert bad.status() == B.ERR_DEVICE_TIMEOUT
    # a later forward on the same plan is refused at the door by every CTA until the status is cleared
    B.sol_attn3d_set_workspace(bad.plan, bad.workspace)      # clears the status word
    assert bad.status() == 0
    bad.close()

    good = B.Attn3d.from_workload(w, "cuda")                # same process, same context
    out = good.forward(inp.q, inp.k, inp.v)
    torch.cuda.synchronize()
    assert good.status() == 0
    ref = orc.attn3d_oracle(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), seqs, w.rope_dims, w.theta)
    max_abs, rel_l2 = orc.compare(out.cpu(), ref)
    assert max_abs <= 2e-2 and rel_l2 <= 5e-3
    good.close()
