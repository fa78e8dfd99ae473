"""ctypes binding of the C-ABI library, one Python function per exported call.

Argument marshalling only: every step of the attention path runs in the CUDA
kernels behind ``libsol_attn3d.so``.  PyTorch appears here only as the owner
of device memory and streams.  There is no CPU fallback: loading fails loudly
if the library has not been built, and device calls fail on a machine without
a B200.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("SOL_ATTN3D_LIB") or os.path.join(_HERE, "libsol_attn3d.so")


class SolAttn3dError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = _lib().sol_attn3d_strerror(code).decode() if _LIB is not None else "?"
        super().__init__(f"{where}: {msg} (code {code})")


class sol_attn3d_desc(ctypes.Structure):
    _fields_ = [
        ("size", ctypes.c_uint32),
        ("n_seqs", ctypes.c_int32),
        ("grids", ctypes.POINTER(ctypes.c_int32)),
        ("text_lens", ctypes.POINTER(ctypes.c_int32)),
        ("heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("rope_dims", ctypes.c_int32 * 3),
        ("theta", ctypes.c_double),
        ("q_strides", ctypes.c_int64 * 2),
        ("k_strides", ctypes.c_int64 * 2),
        ("v_strides", ctypes.c_int64 * 2),
        ("out_strides", ctypes.c_int64 * 2),
    ]


# error codes (mirror include/sol_attn3d.h)
OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED_SHAPE = -2
ERR_NO_WORKSPACE = -3
ERR_NO_DEVICE = -4
ERR_UNSUPPORTED_ARCH = -5
ERR_CUDA = -6
ERR_DEVICE_TIMEOUT = -7
ERR_NO_MEMORY = -8
ERR_SCRATCH_LIMIT = -9
ERR_DEVICE_ASSERT = -10

_LIB = None


def _lib():
    global _LIB
    if _LIB is not None:
        return _LIB
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2609_35110_b200.build` "
            "(there is no CPU fallback for the attention path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    lib.sol_attn3d_plan.argtypes = [ctypes.POINTER(vp), i32, i32, i32, i32, i32, i32, i32, ctypes.POINTER(i32)]
    lib.sol_attn3d_plan.restype = i32
    lib.sol_attn3d_plan_ex.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(sol_attn3d_desc)]
    lib.sol_attn3d_plan_ex.restype = i32
    lib.sol_attn3d_cu_seqlens.argtypes = [vp, ctypes.POINTER(ctypes.POINTER(i64)), ctypes.POINTER(i32)]
    lib.sol_attn3d_cu_seqlens.restype = i32
    lib.sol_attn3d_workspace_bytes.argtypes = [vp]
    lib.sol_attn3d_workspace_bytes.restype = ctypes.c_size_t
    lib.sol_attn3d_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    lib.sol_attn3d_set_workspace.restype = i32
    lib.sol_attn3d_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.sol_attn3d_forward.restype = i32
    lib.sol_attn3d_forward_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sol_attn3d_forward_noalloc.restype = i32
    lib.sol_attn3d_forward_qknorm.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp]
    lib.sol_attn3d_forward_qknorm.restype = i32
    lib.sol_attn3d_qknorm_rope.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp]
    lib.sol_attn3d_qknorm_rope.restype = i32
    lib.sol_attn3d_forward_rect.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sol_attn3d_forward_rect.restype = i32
    lib.sol_attn3d_forward_e4m3.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.sol_attn3d_forward_e4m3.restype = i32
    lib.sol_attn3d_forward_int8.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.sol_attn3d_forward_int8.restype = i32
    lib.sol_attn3d_forward_qkv_int8.argtypes = [vp, vp, vp, vp, vp, i32, vp]
    lib.sol_attn3d_forward_qkv_int8.restype = i32
    lib.sol_attn3d_forward_scatter.argtypes = [vp, vp, vp, vp, vp, i32, ctypes.POINTER(vp), ctypes.POINTER(i64), i32, i32,
                                               i32, vp]
    lib.sol_attn3d_forward_scatter.restype = i32
    lib.sol_attn3d_exchange_pack_qkv.argtypes = [vp, vp, vp, ctypes.POINTER(i64), ctypes.POINTER(i64), ctypes.POINTER(i64),
                                                 i64, i32, i32, i32, i32, i32, ctypes.POINTER(vp), i64, vp]
    lib.sol_attn3d_exchange_pack_qkv.restype = i32
    lib.sol_attn3d_exchange_merge_heads.argtypes = [vp, vp, i64, i32, i32, i32, i64, i64, vp]
    lib.sol_attn3d_exchange_merge_heads.restype = i32
    lib.sol_attn3d_exchange_record_bytes.argtypes = [i32, i32]
    lib.sol_attn3d_exchange_record_bytes.restype = ctypes.c_size_t
    lib.sol_attn3d_exchange_pack_qkv_int8.argtypes = lib.sol_attn3d_exchange_pack_qkv.argtypes
    lib.sol_attn3d_exchange_pack_qkv_int8.restype = i32
    lib.sol_attn3d_exchange_unpack_qkv_int8.argtypes = [vp, vp, i64, i32, i32, vp]
    lib.sol_attn3d_exchange_unpack_qkv_int8.restype = i32
    lib.sol_attn3d_exchange_quantize_out_int8.argtypes = [vp, ctypes.POINTER(i64), i64, i32, i32, vp, vp]
    lib.sol_attn3d_exchange_quantize_out_int8.restype = i32
    lib.sol_attn3d_exchange_dequantize_out_int8.argtypes = [vp, vp, i64, i32, i32, vp]
    lib.sol_attn3d_exchange_dequantize_out_int8.restype = i32
    lib.sol_attn3d_host_staging_bytes.argtypes = [vp]
    lib.sol_attn3d_host_staging_bytes.restype = ctypes.c_size_t
    lib.sol_attn3d_forward_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, i32, vp]
    lib.sol_attn3d_forward_host.restype = i32
    lib.sol_attn3d_sparse_workspace_bytes.argtypes = [vp]
    lib.sol_attn3d_sparse_workspace_bytes.restype = ctypes.c_size_t
    lib.sol_attn3d_forward_sparse.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, ctypes.c_size_t, vp]
    lib.sol_attn3d_forward_sparse.restype = i32
    lib.sol_attn3d_sparse_stats.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_longlong), ctypes.POINTER(ctypes.c_longlong)]
    lib.sol_attn3d_sparse_stats.restype = i32
    lib.sol_attn3d_sparse_selection.argtypes = [vp, vp, i32, i32, i32, ctypes.POINTER(i32), i32, ctypes.POINTER(i32)]
    lib.sol_attn3d_sparse_selection.restype = i32
    lib.sol_attn3d_rope_qk.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.sol_attn3d_rope_qk.restype = i32
    lib.sol_attn3d_status.argtypes = [vp]
    lib.sol_attn3d_status.restype = i32
    lib.sol_attn3d_status_word.argtypes = [vp, ctypes.POINTER(ctypes.c_uint)]
    lib.sol_attn3d_status_word.restype = i32
    lib.sol_attn3d_debug_build.argtypes = []
    lib.sol_attn3d_debug_build.restype = i32
    lib.sol_attn3d_set_profiling.argtypes = [vp, i32]
    lib.sol_attn3d_set_profiling.restype = i32
    lib.sol_attn3d_last_forward_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.sol_attn3d_last_forward_ms.restype = i32
    lib.sol_attn3d_last_launch_count.argtypes = [vp]
    lib.sol_attn3d_last_launch_count.restype = i32
    lib.sol_attn3d_softmax_rescale_count.argtypes = [vp, ctypes.POINTER(ctypes.c_ulonglong)]
    lib.sol_attn3d_softmax_rescale_count.restype = i32
    lib.sol_attn3d_last_cuda_error.argtypes = [vp]
    lib.sol_attn3d_last_cuda_error.restype = i32
    lib.sol_attn3d_strerror.argtypes = [i32]
    lib.sol_attn3d_strerror.restype = ctypes.c_char_p
    lib.sol_attn3d_destroy.argtypes = [vp]
    lib.sol_attn3d_destroy.restype = i32
    _LIB = lib
    return lib


def _check(code: int, where: str) -> None:
    if code != OK:
        raise SolAttn3dError(code, where)


# ----------------------------------------------------------------- 1:1 wrappers
def sol_attn3d_plan(B: int, heads: int, head_dim: int, T: int, H: int, W: int, text_len: int,
                    rope_dims: Sequence[int]) -> ctypes.c_void_p:
    h = ctypes.c_void_p()
    rd = (ctypes.c_int * 3)(*[int(x) for x in rope_dims])
    _check(_lib().sol_attn3d_plan(ctypes.byref(h), B, heads, head_dim, T, H, W, text_len, rd), "sol_attn3d_plan")
    return h


def sol_attn3d_plan_ex(seqs: Sequence[Tuple[int, int, int, int]], heads: int, head_dim: int,
                       rope_dims: Sequence[int], theta: float = 10000.0,
                       q_strides=(0, 0), k_strides=(0, 0), v_strides=(0, 0), out_strides=(0, 0)) -> ctypes.c_void_p:
    """seqs: [(text_len, T, H, W), ...]; strides are (token, head) element strides, 0 = contiguous."""
    n = len(seqs)
    grids = (ctypes.c_int32 * (3 * max(n, 1)))()
    lens = (ctypes.c_int32 * max(n, 1))()
    for i, (L, T, H, W) in enumerate(seqs):
        grids[3 * i], grids[3 * i + 1], grids[3 * i + 2] = T, H, W
        lens[i] = L
    d = sol_attn3d_desc()
    d.size = ctypes.sizeof(sol_attn3d_desc)
    d.n_seqs = n
    d.grids = ctypes.cast(grids, ctypes.POINTER(ctypes.c_int32))
    d.text_lens = ctypes.cast(lens, ctypes.POINTER(ctypes.c_int32))
    d.heads, d.head_dim = heads, head_dim
    for a in range(3):
        d.rope_dims[a] = int(rope_dims[a])
    d.theta = float(theta)
    for name, val in (("q_strides", q_strides), ("k_strides", k_strides), ("v_strides", v_strides),
                      ("out_strides", out_strides)):
        arr = getattr(d, name)
        arr[0], arr[1] = int(val[0]), int(val[1])
    h = ctypes.c_void_p()
    _check(_lib().sol_attn3d_plan_ex(ctypes.byref(h), ctypes.byref(d)), "sol_attn3d_plan_ex")
    return h


def sol_attn3d_cu_seqlens(plan) -> list:
    p = ctypes.POINTER(ctypes.c_int64)()
    n = ctypes.c_int()
    _check(_lib().sol_attn3d_cu_seqlens(plan, ctypes.byref(p), ctypes.byref(n)), "sol_attn3d_cu_seqlens")
    return [int(p[i]) for i in range(n.value + 1)]


def sol_attn3d_workspace_bytes(plan) -> int:
    return int(_lib().sol_attn3d_workspace_bytes(plan))


def sol_attn3d_set_workspace(plan, workspace: torch.Tensor) -> None:
    _check(_lib().sol_attn3d_set_workspace(plan, workspace.data_ptr(), workspace.numel() * workspace.element_size()),
           "sol_attn3d_set_workspace")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def sol_attn3d_forward(plan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                       key_mask: Optional[torch.Tensor] = None, stream=None) -> None:
    for t in (q, k, v, out):
        if not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("q, k, v, out must be CUDA bf16 tensors")
    if key_mask is not None and (not key_mask.is_cuda or key_mask.dtype != torch.uint8 or not key_mask.is_contiguous()):
        raise ValueError("key_mask must be a contiguous CUDA uint8 tensor")
    _check(_lib().sol_attn3d_forward(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(key_mask), _stream(stream)),
           "sol_attn3d_forward")


def sol_attn3d_forward_noalloc(plan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                               key_mask: Optional[torch.Tensor] = None, device_status: Optional[torch.Tensor] = None,
                               stream=None) -> None:
    """Forward without a caller workspace: the scratch is the 32 MiB array inside the library.

    For callers that may not allocate device memory (see include/sol_attn3d.h).  ``device_status`` is an
    optional CUDA int32 tensor with one element that receives the call's status word.  Calls on one
    device must not overlap on the GPU.
    """
    for t in (q, k, v, out):
        if not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("q, k, v, out must be CUDA bf16 tensors")
    if key_mask is not None and (not key_mask.is_cuda or key_mask.dtype != torch.uint8 or not key_mask.is_contiguous()):
        raise ValueError("key_mask must be a contiguous CUDA uint8 tensor")
    if device_status is not None and (not device_status.is_cuda or device_status.element_size() != 4):
        raise ValueError("device_status must be a CUDA tensor of 4-byte elements")
    _check(_lib().sol_attn3d_forward_noalloc(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(key_mask),
                                             _ptr(device_status), _stream(stream)), "sol_attn3d_forward_noalloc")


def sol_attn3d_forward_rect(plan, q, k, v, out, key_mask, query_mask: torch.Tensor, stream=None) -> None:
    """Rectangular forward: only rows with query_mask != 0 are computed and written; all tokens are keys."""
    for t in (q, k, v, out):
        if not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("q, k, v, out must be CUDA bf16 tensors")
    if not query_mask.is_cuda or query_mask.dtype != torch.uint8 or not query_mask.is_contiguous():
        raise ValueError("query_mask must be a contiguous CUDA uint8 tensor")
    _check(_lib().sol_attn3d_forward_rect(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(key_mask), _ptr(query_mask),
                                          _stream(stream)), "sol_attn3d_forward_rect")


def sol_attn3d_host_staging_bytes(plan) -> int:
    return int(_lib().sol_attn3d_host_staging_bytes(plan))


def sol_attn3d_forward_host(plan, q_host: torch.Tensor, k_host: torch.Tensor, v_host: torch.Tensor, out_host: torch.Tensor,
                            key_mask_host: Optional[torch.Tensor], staging: torch.Tensor, n_groups: int = 0, stream=None) -> None:
    """Forward on host tensors (pinned bf16, dense [tokens, heads, D]) through a device staging buffer; copies of one
    head group overlap the kernels of another.  Synchronise the stream before reading out_host."""
    for t in (q_host, k_host, v_host, out_host):
        if t.is_cuda or t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise ValueError("host tensors must be contiguous CPU bf16 tensors")
    if key_mask_host is not None and (key_mask_host.is_cuda or key_mask_host.dtype != torch.uint8 or not key_mask_host.is_contiguous()):
        raise ValueError("key_mask_host must be a contiguous CPU uint8 tensor")
    if not staging.is_cuda:
        raise ValueError("staging must be a CUDA tensor")
    _check(_lib().sol_attn3d_forward_host(plan, _ptr(q_host), _ptr(k_host), _ptr(v_host), _ptr(out_host), _ptr(key_mask_host),
                                          _ptr(staging), staging.numel() * staging.element_size(), n_groups, _stream(stream)),
           "sol_attn3d_forward_host")


OUT_BF16, OUT_E4M3, OUT_INT8 = 0, 1, 2
MAX_RANKS = 8


def sol_attn3d_forward_e4m3(plan, q, k, v, out_e4m3: torch.Tensor, key_mask=None, stream=None) -> None:
    """Forward whose epilogue writes one raw E4M3 byte per output element (unit scale)."""
    for t in (q, k, v):
        if not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("q, k, v must be CUDA bf16 tensors")
    if not out_e4m3.is_cuda or out_e4m3.element_size() != 1:
        raise ValueError("out_e4m3 must be a CUDA tensor of one-byte elements")
    _check(_lib().sol_attn3d_forward_e4m3(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(out_e4m3), _ptr(key_mask),
                                          _stream(stream)), "sol_attn3d_forward_e4m3")


def sol_attn3d_forward_int8(plan, q, k, v, out_records: torch.Tensor, key_mask=None, stream=None) -> None:
    """Forward whose epilogue writes block-INT8 output records [tokens, heads, record_bytes] (uint8)."""
    for t in (q, k, v):
        if not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("q, k, v must be CUDA bf16 tensors")
    if not out_records.is_cuda or out_records.element_size() != 1 or not out_records.is_contiguous():
        raise ValueError("out_records must be a contiguous CUDA tensor of one-byte elements")
    _check(_lib().sol_attn3d_forward_int8(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(out_records), _ptr(key_mask),
                                          _stream(stream)), "sol_attn3d_forward_int8")


def sol_attn3d_forward_qkv_int8(plan, qkv_records: torch.Tensor, v_scratch: torch.Tensor, out: torch.Tensor, key_mask=None,
                                out_format: int = OUT_BF16, stream=None) -> None:
    """Forward fed by block-INT8 QKV records [tokens, heads, record_bytes]; v_scratch: bf16 [tokens, heads, D]."""
    if not qkv_records.is_cuda or qkv_records.element_size() != 1 or not qkv_records.is_contiguous():
        raise ValueError("qkv_records must be a contiguous CUDA tensor of one-byte elements")
    if not v_scratch.is_cuda or v_scratch.dtype != torch.bfloat16 or not v_scratch.is_contiguous():
        raise ValueError("v_scratch must be a contiguous CUDA bf16 tensor")
    if not out.is_cuda:
        raise ValueError("out must be a CUDA tensor")
    _check(_lib().sol_attn3d_forward_qkv_int8(plan, _ptr(qkv_records), _ptr(v_scratch), _ptr(out), _ptr(key_mask), out_format,
                                              _stream(stream)), "sol_attn3d_forward_qkv_int8")


def _ptr_array(ptrs: Sequence[int]):
    return (ctypes.c_void_p * len(ptrs))(*[ctypes.c_void_p(int(x)) if x else None for x in ptrs])


def sol_attn3d_forward_scatter(plan, q, k, v, key_mask, dst: Sequence[int], tok_begin: Sequence[int], dst_heads: int,
                               head_offset: int, out_format: int = OUT_BF16, stream=None) -> None:
    """dst: device addresses (ints; this GPU's or peer-mapped) of the token owners' [n_g, dst_heads, D] buffers."""
    for t in (q, k, v):
        if not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("q, k, v must be CUDA bf16 tensors")
    if len(tok_begin) != len(dst) + 1:
        raise ValueError("tok_begin needs len(dst) + 1 entries")
    tb = (ctypes.c_int64 * len(tok_begin))(*[int(x) for x in tok_begin])
    _check(_lib().sol_attn3d_forward_scatter(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(key_mask), len(dst), _ptr_array(dst),
                                             tb, dst_heads, head_offset, out_format, _stream(stream)),
           "sol_attn3d_forward_scatter")


def _strides_of(t: torch.Tensor, head_dim: int):
    """(token, head) element strides of a [tokens, heads, head_dim] tensor whose head_dim axis is contiguous."""
    if t.dim() != 3 or t.shape[2] != head_dim or t.stride(2) != 1:
        raise ValueError("expected [tokens, heads, head_dim] with contiguous head_dim")
    # the stride torch reports for an axis of extent 0 or 1 is arbitrary: use the dense value there
    tok = t.stride(0) if t.shape[0] > 1 else t.shape[1] * head_dim
    head = t.stride(1) if t.shape[1] > 1 else head_dim
    return (ctypes.c_int64 * 2)(tok, head)


def sol_attn3d_exchange_pack_qkv(q, k, v, n_ranks: int, dst: Sequence[int], dst_row0: int = 0, stream=None,
                                 group_begin: int = 0, group_heads: int = 0) -> None:
    """q, k, v: CUDA bf16 [n_local, heads, D] (any token / head strides); dst: n_ranks device addresses.
    group_begin / group_heads: send only that head group of every rank's shard (0, 0 = the whole shard)."""
    n_local, heads, head_dim = q.shape
    for t in (q, k, v):
        if not t.is_cuda or t.dtype != torch.bfloat16 or tuple(t.shape) != (n_local, heads, head_dim):
            raise ValueError("q, k, v must be CUDA bf16 tensors of one shape")
    if len(dst) != n_ranks:
        raise ValueError("one destination per rank")
    _check(_lib().sol_attn3d_exchange_pack_qkv(_ptr(q), _ptr(k), _ptr(v), _strides_of(q, head_dim), _strides_of(k, head_dim),
                                               _strides_of(v, head_dim), n_local, heads, head_dim, n_ranks, group_begin,
                                               group_heads, _ptr_array(dst), dst_row0, _stream(stream)),
           "sol_attn3d_exchange_pack_qkv")


WIRE_QKV_BF16, WIRE_QKV_INT8, WIRE_OUT_BF16, WIRE_OUT_E4M3, WIRE_OUT_INT8 = 0, 1, 2, 3, 4


def sol_attn3d_exchange_record_bytes(kind: int, head_dim: int) -> int:
    n = int(_lib().sol_attn3d_exchange_record_bytes(kind, head_dim))
    if n == 0:
        raise ValueError("unknown wire format or head_dim")
    return n


def sol_attn3d_exchange_pack_qkv_int8(q, k, v, n_ranks: int, dst: Sequence[int], dst_row0: int = 0, stream=None,
                                      group_begin: int = 0, group_heads: int = 0) -> None:
    """As sol_attn3d_exchange_pack_qkv, but the destinations receive block-INT8 records."""
    n_local, heads, head_dim = q.shape
    for t in (q, k, v):
        if not t.is_cuda or t.dtype != torch.bfloat16 or tuple(t.shape) != (n_local, heads, head_dim):
            raise ValueError("q, k, v must be CUDA bf16 tensors of one shape")
    if len(dst) != n_ranks:
        raise ValueError("one destination per rank")
    _check(_lib().sol_attn3d_exchange_pack_qkv_int8(_ptr(q), _ptr(k), _ptr(v), _strides_of(q, head_dim),
                                                    _strides_of(k, head_dim), _strides_of(v, head_dim), n_local, heads,
                                                    head_dim, n_ranks, group_begin, group_heads, _ptr_array(dst), dst_row0,
                                                    _stream(stream)),
           "sol_attn3d_exchange_pack_qkv_int8")


def sol_attn3d_exchange_unpack_qkv_int8(records: torch.Tensor, qkv: torch.Tensor, n_rows: int, heads: int, head_dim: int,
                                        stream=None) -> None:
    if not records.is_cuda or not qkv.is_cuda or qkv.dtype != torch.bfloat16 or not qkv.is_contiguous():
        raise ValueError("records: CUDA bytes; qkv: contiguous CUDA bf16 [rows, 3, heads, D]")
    _check(_lib().sol_attn3d_exchange_unpack_qkv_int8(_ptr(records), _ptr(qkv), n_rows, heads, head_dim, _stream(stream)),
           "sol_attn3d_exchange_unpack_qkv_int8")


def sol_attn3d_exchange_quantize_out_int8(out_rows: torch.Tensor, records: torch.Tensor, stream=None) -> None:
    n_rows, heads, head_dim = out_rows.shape
    if not out_rows.is_cuda or out_rows.dtype != torch.bfloat16 or not records.is_cuda:
        raise ValueError("out_rows: CUDA bf16 [rows, heads, D]; records: CUDA bytes")
    _check(_lib().sol_attn3d_exchange_quantize_out_int8(_ptr(out_rows), _strides_of(out_rows, head_dim), n_rows, heads,
                                                        head_dim, _ptr(records), _stream(stream)),
           "sol_attn3d_exchange_quantize_out_int8")


def sol_attn3d_exchange_dequantize_out_int8(records: torch.Tensor, out_rows: torch.Tensor, stream=None) -> None:
    n_rows, heads, head_dim = out_rows.shape
    if not out_rows.is_cuda or out_rows.dtype != torch.bfloat16 or not out_rows.is_contiguous() or not records.is_cuda:
        raise ValueError("out_rows: contiguous CUDA bf16 [rows, heads, D]; records: CUDA bytes")
    _check(_lib().sol_attn3d_exchange_dequantize_out_int8(_ptr(records), _ptr(out_rows), n_rows, heads, head_dim,
                                                          _stream(stream)), "sol_attn3d_exchange_dequantize_out_int8")


def sol_attn3d_exchange_merge_heads(recv: torch.Tensor, out, n_local: int, heads: int, record_bytes: int,
                                    n_ranks: int, out_tok_stride_bytes: int = 0, stream=None, out_rank_stride_bytes: int = 0) -> None:
    """out: CUDA tensor, or a device address (int) when the rows start inside a larger tensor."""
    if not recv.is_cuda or not recv.is_contiguous():
        raise ValueError("recv must be a contiguous CUDA tensor")
    out_ptr = ctypes.c_void_p(int(out)) if isinstance(out, int) else _ptr(out)
    _check(_lib().sol_attn3d_exchange_merge_heads(_ptr(recv), out_ptr, n_local, heads, record_bytes, n_ranks,
                                                  out_tok_stride_bytes, out_rank_stride_bytes, _stream(stream)),
           "sol_attn3d_exchange_merge_heads")


def sol_attn3d_sparse_workspace_bytes(plan) -> int:
    return int(_lib().sol_attn3d_sparse_workspace_bytes(plan))


def sol_attn3d_forward_sparse(plan, q, k, v, out, key_mask, tau: float, sparse_ws: torch.Tensor, stream=None) -> None:
    """Block-sparse forward (mu + tau*sigma selection of 128-key blocks per 256-row query block)."""
    for t in (q, k, v, out):
        if not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("q, k, v, out must be CUDA bf16 tensors")
    _check(_lib().sol_attn3d_forward_sparse(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(key_mask),
                                            ctypes.c_float(tau), _ptr(sparse_ws),
                                            sparse_ws.numel() * sparse_ws.element_size(), _stream(stream)),
           "sol_attn3d_forward_sparse")


def sol_attn3d_sparse_stats(plan, sparse_ws: torch.Tensor) -> Tuple[int, int]:
    a, b = ctypes.c_longlong(), ctypes.c_longlong()
    _check(_lib().sol_attn3d_sparse_stats(plan, _ptr(sparse_ws), ctypes.byref(a), ctypes.byref(b)), "sol_attn3d_sparse_stats")
    return int(a.value), int(b.value)


def sol_attn3d_sparse_selection(plan, sparse_ws: torch.Tensor, seq: int, head: int, query_block: int, capacity: int) -> list:
    buf = (ctypes.c_int * max(capacity, 1))()
    n = ctypes.c_int()
    _check(_lib().sol_attn3d_sparse_selection(plan, _ptr(sparse_ws), seq, head, query_block, buf, capacity,
                                              ctypes.byref(n)), "sol_attn3d_sparse_selection")
    return [int(buf[i]) for i in range(min(n.value, capacity))]


def _check_gain(g: torch.Tensor, head_dim_hint=None):
    if g is None or not g.is_cuda or g.dtype != torch.float32 or not g.is_contiguous():
        raise ValueError("gains must be contiguous CUDA float32 tensors of head_dim elements")


def sol_attn3d_forward_qknorm(plan, q, k, v, out, key_mask, q_gain: torch.Tensor, k_gain: torch.Tensor, eps: float,
                              stream=None) -> None:
    """Forward with QK RMS-norm (gain vectors of head_dim fp32 values) applied before the rotary embedding."""
    for t in (q, k, v, out):
        if not t.is_cuda or t.dtype != torch.bfloat16:
            raise ValueError("q, k, v, out must be CUDA bf16 tensors")
    _check_gain(q_gain)
    _check_gain(k_gain)
    _check(_lib().sol_attn3d_forward_qknorm(plan, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(key_mask), _ptr(q_gain),
                                            _ptr(k_gain), ctypes.c_float(eps), _stream(stream)),
           "sol_attn3d_forward_qknorm")


def sol_attn3d_qknorm_rope(plan, q, k, q_gain, k_gain, eps: float, q_out, k_out, stream=None) -> None:
    _check(_lib().sol_attn3d_qknorm_rope(plan, _ptr(q), _ptr(k), _ptr(q_gain), _ptr(k_gain), ctypes.c_float(eps),
                                         _ptr(q_out), _ptr(k_out), _stream(stream)), "sol_attn3d_qknorm_rope")


def sol_attn3d_rope_qk(plan, q, k, q_rot, k_rot, stream=None) -> None:
    _check(_lib().sol_attn3d_rope_qk(plan, _ptr(q), _ptr(k), _ptr(q_rot), _ptr(k_rot), _stream(stream)),
           "sol_attn3d_rope_qk")


def sol_attn3d_status(plan) -> int:
    return int(_lib().sol_attn3d_status(plan))


def sol_attn3d_status_word(plan) -> int:
    w = ctypes.c_uint()
    _check(_lib().sol_attn3d_status_word(plan, ctypes.byref(w)), "sol_attn3d_status_word")
    return int(w.value)


def sol_attn3d_debug_build() -> bool:
    return bool(_lib().sol_attn3d_debug_build())


def sol_attn3d_set_profiling(plan, enable: bool) -> None:
    _check(_lib().sol_attn3d_set_profiling(plan, 1 if enable else 0), "sol_attn3d_set_profiling")


def sol_attn3d_last_forward_ms(plan) -> Tuple[float, float, float]:
    ms = (ctypes.c_float * 3)()
    _check(_lib().sol_attn3d_last_forward_ms(plan, ms), "sol_attn3d_last_forward_ms")
    return float(ms[0]), float(ms[1]), float(ms[2])


def sol_attn3d_last_launch_count(plan) -> int:
    return int(_lib().sol_attn3d_last_launch_count(plan))


def sol_attn3d_softmax_rescale_count(plan) -> int:
    n = ctypes.c_ulonglong()
    _check(_lib().sol_attn3d_softmax_rescale_count(plan, ctypes.byref(n)), "sol_attn3d_softmax_rescale_count")
    return int(n.value)


def sol_attn3d_last_cuda_error(plan) -> int:
    return int(_lib().sol_attn3d_last_cuda_error(plan))


def sol_attn3d_strerror(code: int) -> str:
    return _lib().sol_attn3d_strerror(code).decode()


def sol_attn3d_destroy(plan) -> None:
    _check(_lib().sol_attn3d_destroy(plan), "sol_attn3d_destroy")


# ----------------------------------------------------------------- convenience holder
class Attn3d:
    """Owns a plan and its torch-allocated workspace.  ``forward`` = one DiT-block attention."""

    def __init__(self, seqs, heads, head_dim, rope_dims, theta=10000.0, device="cuda", **strides):
        self.seqs = [tuple(int(x) for x in s) for s in seqs]
        self.heads, self.head_dim = heads, head_dim
        self.plan = sol_attn3d_plan_ex(self.seqs, heads, head_dim, rope_dims, theta, **strides)
        self.cu_seqlens = sol_attn3d_cu_seqlens(self.plan)
        self.total_tokens = self.cu_seqlens[-1]
        self.workspace = None
        if device is not None:
            nbytes = sol_attn3d_workspace_bytes(self.plan)
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
            assert self.workspace.data_ptr() % 256 == 0
            sol_attn3d_set_workspace(self.plan, self.workspace)

    @classmethod
    def from_workload(cls, w, device="cuda"):
        return cls([(s.text_len, s.T, s.H, s.W) for s in w.seqs], w.heads, w.head_dim, w.rope_dims, w.theta, device)

    def forward(self, q, k, v, key_mask=None, out=None, stream=None):
        if out is None:
            out = torch.empty((self.total_tokens, self.heads, self.head_dim), dtype=torch.bfloat16, device=q.device)
        sol_attn3d_forward(self.plan, q, k, v, out, key_mask, stream)
        return out

    def rope_qk(self, q, k, stream=None):
        q_rot = torch.empty((self.total_tokens, self.heads, self.head_dim), dtype=torch.bfloat16, device=q.device)
        k_rot = torch.empty_like(q_rot)
        sol_attn3d_rope_qk(self.plan, q, k, q_rot, k_rot, stream)
        return q_rot, k_rot

    def status(self) -> int:
        return sol_attn3d_status(self.plan)

    def close(self):
        if self.plan is not None:
            sol_attn3d_destroy(self.plan)
            self.plan = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
