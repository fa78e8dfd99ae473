"""CPU tests of the C-ABI library: it loads, exports what the header declares, and its host-side
plan logic (validation, token layout, workspace sizing) is right.  No compute calls."""
import ctypes
import os
import re

import pytest
import torch

from paper_2609_35110_b200 import binding as B
from paper_2609_35110_b200 import build as build_mod
from paper_2609_35110_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    build_mod.build_library()
    return B._lib()


def test_library_exports_every_declared_symbol(built_library):
    header = open(os.path.join(ROOT, "include", "sol_attn3d.h")).read()
    body = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(sol_attn3d_[a-z0-9_]+)\s*\(", body))
    assert {"sol_attn3d_plan", "sol_attn3d_forward", "sol_attn3d_destroy"} <= names
    raw = ctypes.CDLL(B.LIB_PATH)
    for n in sorted(names):
        assert hasattr(raw, n), f"{n} declared in the header but not exported"


def test_plan_rejects_bad_arguments():
    ok = dict(B=1, heads=4, head_dim=64, T=4, H=8, W=8, text_len=0, rope_dims=(16, 24, 24))

    def code(**kw):
        a = dict(ok)
        a.update(kw)
        try:
            p = B.sol_attn3d_plan(**a)
        except B.SolAttn3dError as e:
            return e.code
        B.sol_attn3d_destroy(p)
        return 0

    assert code() == 0
    assert code(B=0) == B.ERR_INVALID_ARG
    assert code(heads=0) == B.ERR_INVALID_ARG
    assert code(T=0) == B.ERR_INVALID_ARG
    assert code(W=-1) == B.ERR_INVALID_ARG
    assert code(text_len=-1) == B.ERR_INVALID_ARG
    assert code(rope_dims=(15, 24, 24)) == B.ERR_INVALID_ARG         # odd
    assert code(rope_dims=(16, 24, 26)) == B.ERR_INVALID_ARG         # sum > head_dim
    assert code(rope_dims=(-2, 24, 24)) == B.ERR_INVALID_ARG
    assert code(head_dim=96) == B.ERR_UNSUPPORTED_SHAPE
    assert code(rope_dims=(0, 0, 0)) == 0                             # no rotary at all is legal
    assert code(rope_dims=(16, 8, 8)) == 0                            # partial rotary


def test_plan_ex_validation_and_strides():
    with pytest.raises(B.SolAttn3dError) as e:
        B.sol_attn3d_plan_ex([], 4, 64, (16, 24, 24))
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.SolAttn3dError) as e:
        B.sol_attn3d_plan_ex([(0, 1, 1, 1)], 4, 64, (16, 24, 24), theta=1.0)
    assert e.value.code == B.ERR_INVALID_ARG
    with pytest.raises(B.SolAttn3dError) as e:                       # token stride of 3 bytes*2: not 16-byte multiple
        B.sol_attn3d_plan_ex([(0, 1, 1, 1)], 4, 64, (16, 24, 24), q_strides=(259, 64))
    assert e.value.code == B.ERR_UNSUPPORTED_SHAPE
    # packed QKV view: token stride 3*heads*D
    p = B.sol_attn3d_plan_ex([(2, 1, 2, 2)], 4, 64, (16, 24, 24), q_strides=(768, 64), k_strides=(768, 64),
                             v_strides=(768, 64))
    B.sol_attn3d_destroy(p)
    # prefix-only sequence (T = 0) is allowed in the extended form, an empty sequence is not
    p = B.sol_attn3d_plan_ex([(5, 0, 1, 1)], 2, 64, (16, 24, 24))
    assert B.sol_attn3d_cu_seqlens(p) == [0, 5]
    B.sol_attn3d_destroy(p)
    with pytest.raises(B.SolAttn3dError):
        B.sol_attn3d_plan_ex([(0, 0, 1, 1)], 2, 64, (16, 24, 24))


def test_cu_seqlens_match_the_contract_configs():
    expect = {"tiny": [0, 256], "lowres": [0, 25216], "highres": [0, 111856],
              "cfg_batch": [0, 112112, 224224], "varlen": [0, 12736, 37952, 95808, 207664]}
    for name, cu in expect.items():
        w = wl.CONFIGS[name]
        a = B.Attn3d.from_workload(w, device=None)
        assert a.cu_seqlens == cu == w.cu_seqlens
        a.close()
    p = B.sol_attn3d_plan(2, 40, 128, 31, 45, 80, 512, (32, 48, 48))
    assert B.sol_attn3d_cu_seqlens(p) == [0, 112112, 224224]
    B.sol_attn3d_destroy(p)


def test_workspace_size_covers_rotated_q_and_k():
    for name in wl.CONFIG_ORDER:
        w = wl.CONFIGS[name]
        a = B.Attn3d.from_workload(w, device=None)
        nbytes = B.sol_attn3d_workspace_bytes(a.plan)
        rot = 2 * w.total_tokens * w.heads * w.head_dim * 2
        assert rot <= nbytes <= rot + (1 << 20) + 64 * (w.total_tokens // 128 + 8)
        assert nbytes % 256 == 0
        a.close()


def test_device_calls_fail_cleanly_without_workspace_or_device():
    p = B.sol_attn3d_plan(1, 4, 64, 4, 8, 8, 0, (16, 24, 24))
    lib = B._lib()
    assert lib.sol_attn3d_forward(p, 16, 32, 48, 64, None, None) == B.ERR_NO_WORKSPACE
    assert lib.sol_attn3d_forward(p, None, 32, 48, 64, None, None) == B.ERR_INVALID_ARG
    assert lib.sol_attn3d_forward(p, 8, 32, 48, 64, None, None) == B.ERR_INVALID_ARG      # misaligned
    assert lib.sol_attn3d_forward(p, 16, 32, 48, 16, None, None) == B.ERR_INVALID_ARG     # out aliases q
    assert lib.sol_attn3d_status(p) == B.ERR_NO_WORKSPACE
    assert lib.sol_attn3d_set_workspace(p, None, 0) == B.ERR_NO_WORKSPACE
    assert lib.sol_attn3d_set_workspace(p, 256 + 8, 1 << 30) == B.ERR_NO_WORKSPACE        # misaligned
    if not torch.cuda.is_available():
        # a plausible pointer on a machine without a GPU: refused before anything is touched
        assert lib.sol_attn3d_set_workspace(p, 1 << 20, 1 << 30) in (B.ERR_NO_DEVICE, B.ERR_CUDA)
    assert B.sol_attn3d_last_launch_count(p) == 0                                         # nothing was enqueued
    assert lib.sol_attn3d_softmax_rescale_count(p, None) == B.ERR_INVALID_ARG
    assert B.sol_attn3d_strerror(B.ERR_DEVICE_TIMEOUT)
    assert lib.sol_attn3d_destroy(None) == 0
    B.sol_attn3d_destroy(p)


def test_workload_recipes():
    w = wl.CONFIGS["cfg_batch"]
    m = wl.make_key_mask(w)
    assert m.shape == (224224,) and int(m[:112112].sum()) == 112112
    assert int(m[112112:112112 + 512].sum()) == 77 and int(m[112112 + 77]) == 0 and int(m[112112 + 512]) == 1
    rows = wl.sample_rows(wl.CONFIGS["highres"], 0, 7)
    assert len(rows) == 4096 and len(set(rows.tolist())) == 4096
    for r in (0, 255, 256, 111855, 111744, 111743):
        assert r in rows
    assert (wl.sample_rows(wl.CONFIGS["highres"], 0, 7) == rows).all()
    assert not (wl.sample_rows(wl.CONFIGS["highres"], 0, 8) == rows).all()
    small = wl.shrunk("lowres")
    inp = wl.make_inputs(small)
    assert inp.q.dtype == torch.bfloat16 and inp.q.shape == (620, 3, 128)
    assert abs(float(inp.k.float().std()) - 0.5) < 0.02 and abs(float(inp.q.float().std()) - 1.0) < 0.03
    v = wl.make_inputs(wl.shrunk("varlen")).v.float()
    assert float(v.min()) >= -1.0 and float(v.max()) <= 1.0 and abs(float(v.mean())) < 0.02
    assert abs(wl.CONFIGS["highres"].flops() - 2.5624e14) / 2.5624e14 < 1e-3
    assert abs(wl.CONFIGS["lowres"].flops() - 1.3022e13) / 1.3022e13 < 1e-3
