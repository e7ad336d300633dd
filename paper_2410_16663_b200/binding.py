"""ctypes binding of ``libfa.so``: the same entry points as ``include/fa.h``, same names.

This layer only marshals arguments (pointers, sizes, the current CUDA stream); every step of
the attention path runs inside the library's kernels.  There is no fallback: if the library is
missing or fails to load, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

FA_OK = 0
FA_ERR_NULL, FA_ERR_SHAPE, FA_ERR_UNSUPPORTED, FA_ERR_ALIGN = -1, -2, -3, -4
FA_ERR_WORKSPACE, FA_ERR_DEVICE, FA_ERR_CUDA, FA_ERR_TIMEOUT = -5, -6, -7, -8
FA_DTYPE_FP16, FA_DTYPE_BF16, FA_DTYPE_FP32 = 0, 1, 2

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libfa.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2410_16663_b200.build` "
                      "(the CUDA library is required; there is no fallback path)")
lib = ctypes.CDLL(_LIB_PATH)

_i, _f, _p, _sz = ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t


class fa_params(ctypes.Structure):
    _fields_ = [("q", _p), ("k", _p), ("v", _p), ("o", _p), ("lse", _p),
                ("B", _i), ("Hq", _i), ("Hkv", _i), ("Sq", _i), ("Skv", _i), ("d", _i),
                ("causal", _i), ("scale", _f), ("dtype", _i), ("o_dtype", _i),
                ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3),
                ("v_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3),
                ("variant", _i)]


_FWD_ARGS = [_p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _f, _p]
lib.fa_forward.restype = _i
lib.fa_forward.argtypes = _FWD_ARGS
lib.fa_forward_bf16.restype = _i
lib.fa_forward_bf16.argtypes = _FWD_ARGS
lib.fa_forward_ex.restype = _i
lib.fa_forward_ex.argtypes = [ctypes.POINTER(fa_params), _p]
lib.fa_forward_fp8.restype = _i
lib.fa_forward_fp8.argtypes = [_p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _f, _f, _f, _f, _i, _p]
lib.fa_forward_proj.restype = _i
lib.fa_forward_proj.argtypes = [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _f, _i, _i, _p, _sz, _p]
lib.fa_forward_proj_workspace_bytes.restype = _sz
lib.fa_forward_proj_workspace_bytes.argtypes = [_i, _i]
lib.fa_decode.restype = _i
lib.fa_decode.argtypes = [_p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _f, _p, _sz, _p]
lib.fa_decode_workspace_bytes.restype = _sz
lib.fa_decode_workspace_bytes.argtypes = [_i, _i, _i, _i, _i]
lib.fa_forward_varlen.restype = _i
lib.fa_forward_varlen.argtypes = [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _i, _f, _i, _p]
class fa_decode_params(ctypes.Structure):
    _fields_ = [("q", _p), ("k", _p), ("v", _p), ("o", _p), ("lse", _p), ("seqlens_k", _p), ("block_table", _p),
                ("B", _i), ("Sq", _i), ("Hq", _i), ("Hkv", _i), ("Skv_max", _i), ("d", _i), ("dtype", _i),
                ("num_pages", _i), ("page_size", _i), ("max_pages", _i), ("table_stride", _i), ("scale", _f),
                ("workspace", _p), ("workspace_bytes", _sz)]


lib.fa_decode_ex.restype = _i
lib.fa_decode_ex.argtypes = [ctypes.POINTER(fa_decode_params), _p]
lib.fa_decode_append.restype = _i
lib.fa_decode_append.argtypes = [_p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _f, _p, _sz, _p]
lib.fa_decode_append_workspace_bytes.restype = _sz
lib.fa_decode_append_workspace_bytes.argtypes = [_i, _i, _i, _i, _i, _i]
lib.fa_decode_fp8.restype = _i
lib.fa_decode_fp8.argtypes = [_p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _f, _f, _f, _p, _sz, _p]
lib.fa_decode_fp8_paged.restype = _i
lib.fa_decode_fp8_paged.argtypes = [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _f, _f, _f, _p, _sz, _p]
lib.fa_decode_fp8_bf16.restype = _i
lib.fa_decode_fp8_bf16.argtypes = lib.fa_decode_fp8.argtypes
lib.fa_decode_fp8_paged_bf16.restype = _i
lib.fa_decode_fp8_paged_bf16.argtypes = lib.fa_decode_fp8_paged.argtypes
lib.fa_forward_varlen_paged.restype = _i
lib.fa_forward_varlen_paged.argtypes = [_p, _p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _i, _i, _i, _i, _f,
                                        _i, _p]
lib.fa_decode_paged.restype = _i
lib.fa_decode_paged.argtypes = [_p, _p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _i, _f, _p, _sz, _p]
lib.fa_decode_noalloc.restype = _i
lib.fa_decode_noalloc.argtypes = [_p, _p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _f, _p]
lib.fa_forward_host.restype = _i
lib.fa_forward_host.argtypes = [_p, _p, _p, _p, _p, _i, _i, _i, _i, _i, _i, _i, _f, _i, _p, _sz, _p]
lib.fa_forward_host_staging_bytes.restype = _sz
lib.fa_forward_host_staging_bytes.argtypes = [_i, _i, _i, _i, _i, _i]
lib.fa_device_status.restype = _i
lib.fa_device_status.argtypes = [ctypes.POINTER(ctypes.c_uint * 2)]
lib.fa_selftest_wait.restype = _i
lib.fa_selftest_wait.argtypes = [ctypes.c_uint, _p, _p]
lib.fa_strerror.restype = ctypes.c_char_p
lib.fa_strerror.argtypes = [_i]
lib.fa_version.restype = _i
lib.fa_last_cuda_error.restype = _i

FA_DECODE_NOALLOC_BYTES = 4 << 20

EXPORTS = ["fa_forward", "fa_forward_bf16", "fa_forward_ex", "fa_forward_fp8", "fa_forward_proj", "fa_forward_proj_workspace_bytes", "fa_decode", "fa_decode_workspace_bytes",
           "fa_decode_noalloc", "fa_decode_paged", "fa_forward_varlen", "fa_decode_fp8", "fa_decode_fp8_paged", "fa_decode_fp8_bf16", "fa_decode_fp8_paged_bf16", "fa_decode_append", "fa_decode_append_workspace_bytes", "fa_decode_ex", "fa_forward_varlen_paged",
           "fa_forward_host", "fa_forward_host_staging_bytes", "fa_device_status", "fa_selftest_wait", "fa_strerror",
           "fa_version", "fa_last_cuda_error"]


class FaError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {fa_strerror(code)} (code {code}, cuda {fa_last_cuda_error()})")


def fa_strerror(code: int) -> str:
    return lib.fa_strerror(int(code)).decode()


def fa_version() -> int:
    return int(lib.fa_version())


def fa_last_cuda_error() -> int:
    return int(lib.fa_last_cuda_error())


def _stream() -> int:
    return int(torch.cuda.current_stream().cuda_stream)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _check(rc: int, what: str, raise_on_error: bool) -> int:
    if rc != FA_OK and raise_on_error:
        raise FaError(rc, what)
    return rc


def fa_forward(q, k, v, o, lse, causal: bool, scale: float, raise_on_error: bool = True) -> int:
    """``fa_forward`` / ``fa_forward_bf16`` on contiguous [B,S,H,d] device tensors (by dtype of q)."""
    B, Sq, Hq, d = q.shape
    _, Skv, Hkv, _ = k.shape
    fn = lib.fa_forward_bf16 if q.dtype == torch.bfloat16 else lib.fa_forward
    rc = fn(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), B, Hq, Hkv, Sq, Skv, d, int(bool(causal)),
            float(scale), _stream())
    return _check(rc, "fa_forward", raise_on_error)


def fa_forward_ex(q, k, v, o, lse, causal: bool, scale: float, variant: int = 0,
                  raise_on_error: bool = True) -> int:
    """``fa_forward_ex``: q/k/v/o are [B,S,H,d] views with any batch/sequence/head strides
    (d contiguous); ``o`` may be fp32 to read the accumulator without the final rounding."""
    B, Sq, Hq, d = q.shape
    _, Skv, Hkv, _ = k.shape
    p = fa_params()
    p.q, p.k, p.v, p.o, p.lse = _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse)
    p.B, p.Hq, p.Hkv, p.Sq, p.Skv, p.d = B, Hq, Hkv, Sq, Skv, d
    p.causal, p.scale = int(bool(causal)), float(scale)
    p.dtype = FA_DTYPE_BF16 if q.dtype == torch.bfloat16 else FA_DTYPE_FP16
    p.o_dtype = FA_DTYPE_FP32 if o.dtype == torch.float32 else p.dtype
    for name, t in (("q_stride", q), ("k_stride", k), ("v_stride", v), ("o_stride", o)):
        arr = getattr(p, name)
        arr[0], arr[1], arr[2] = t.stride(0), t.stride(1), t.stride(2)
    p.variant = int(variant)
    rc = lib.fa_forward_ex(ctypes.byref(p), _stream())
    return _check(rc, "fa_forward_ex", raise_on_error)


def fa_forward_fp8(q, k, v, o, lse, causal: bool, scale: float, q_scale: float, k_scale: float, v_scale: float,
                   raise_on_error: bool = True) -> int:
    """``fa_forward_fp8``: q [B,Sq,Hq,d], k, v [B,Skv,Hkv,d] contiguous device tensors of FP8 e4m3
    (``torch.float8_e4m3fn`` or uint8 bit patterns) with one factor each; o fp16 or bf16."""
    B, Sq, Hq, d = q.shape
    _, Skv, Hkv, _ = k.shape
    dt = FA_DTYPE_BF16 if o.dtype == torch.bfloat16 else FA_DTYPE_FP16
    rc = lib.fa_forward_fp8(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), B, Hq, Hkv, Sq, Skv, d, int(bool(causal)),
                            float(scale), float(q_scale), float(k_scale), float(v_scale), dt, _stream())
    return _check(rc, "fa_forward_fp8", raise_on_error)


def fa_forward_proj_workspace_bytes(B: int, Sq: int) -> int:
    return int(lib.fa_forward_proj_workspace_bytes(B, Sq))


def fa_forward_proj(q, k, v, w_o, o, lse, out, causal: bool, scale: float, fused: bool, workspace=None,
                    raise_on_error: bool = True) -> int:
    """``fa_forward_proj``: attention, then ``out = O.view(B, Sq, Hq*d) @ w_o`` with w_o [Hq*d, d_model];
    one launch (``fused``, needs a workspace of ``fa_forward_proj_workspace_bytes`` bytes) or two."""
    B, Sq, Hq, d = q.shape
    _, Skv, Hkv, _ = k.shape
    dt = FA_DTYPE_BF16 if q.dtype == torch.bfloat16 else FA_DTYPE_FP16
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.fa_forward_proj(_ptr(q), _ptr(k), _ptr(v), _ptr(w_o), _ptr(o), _ptr(lse), _ptr(out), B, Hq, Hkv, Sq, Skv, d,
                             w_o.shape[1], int(bool(causal)), float(scale), dt, int(bool(fused)), _ptr(workspace), wbytes,
                             _stream())
    return _check(rc, "fa_forward_proj", raise_on_error)


def fa_forward_varlen(q, k, v, o, lse, cu_seqlens_q, cu_seqlens_k, max_seqlen_q: int, max_seqlen_k: int,
                      causal: bool, scale: float, raise_on_error: bool = True) -> int:
    """``fa_forward_varlen``: q, o [total_q,Hq,d], k, v [total_k,Hkv,d] contiguous device tensors,
    lse [Hq,total_q] or None, cu_seqlens_* int32 [B+1] on the device."""
    total_q, Hq, d = q.shape
    total_k, Hkv, _ = k.shape
    B = cu_seqlens_q.numel() - 1
    dt = FA_DTYPE_BF16 if q.dtype == torch.bfloat16 else FA_DTYPE_FP16
    rc = lib.fa_forward_varlen(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(cu_seqlens_q),
                               _ptr(cu_seqlens_k), B, Hq, Hkv, total_q, total_k, int(max_seqlen_q),
                               int(max_seqlen_k), d, int(bool(causal)), float(scale), dt, _stream())
    return _check(rc, "fa_forward_varlen", raise_on_error)


def fa_decode_workspace_bytes(B: int, Hq: int, Hkv: int, Skv_max: int, d: int) -> int:
    return int(lib.fa_decode_workspace_bytes(B, Hq, Hkv, Skv_max, d))


def fa_decode(q, k_cache, v_cache, o, lse, seqlens_k, scale: float, workspace,
              raise_on_error: bool = True) -> int:
    """``fa_decode``: q [B,1,Hq,d], caches [B,Smax,Hkv,d], seqlens_k int32 [B] on the device,
    workspace a device byte tensor of at least ``fa_decode_workspace_bytes`` bytes."""
    B, _, Hq, d = q.shape
    _, Smax, Hkv, _ = k_cache.shape
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.fa_decode(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse), _ptr(seqlens_k), B, Hq,
                       Hkv, Smax, d, float(scale), _ptr(workspace), wbytes, _stream())
    return _check(rc, "fa_decode", raise_on_error)


def fa_forward_varlen_paged(q, k_pages, v_pages, block_table, o, lse, cu_seqlens_q, seqlens_k, max_seqlen_q: int,
                            max_seqlen_k: int, causal: bool, scale: float, raise_on_error: bool = True) -> int:
    """``fa_forward_varlen_paged``: q, o [total_q,Hq,d] packed, K and V in page pools [num_pages,page_size,Hkv,d]
    behind block_table int32 [B,stride]; cu_seqlens_q int32 [B+1] and seqlens_k int32 [B] on the device."""
    total_q, Hq, d = q.shape
    num_pages, page_size, Hkv, _ = k_pages.shape
    B = cu_seqlens_q.numel() - 1
    dt = FA_DTYPE_BF16 if q.dtype == torch.bfloat16 else FA_DTYPE_FP16
    rc = lib.fa_forward_varlen_paged(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table), _ptr(o), _ptr(lse),
                                     _ptr(cu_seqlens_q), _ptr(seqlens_k), B, Hq, Hkv, total_q, num_pages, page_size,
                                     block_table.shape[1], block_table.stride(0), int(max_seqlen_q), int(max_seqlen_k), d,
                                     int(bool(causal)), float(scale), dt, _stream())
    return _check(rc, "fa_forward_varlen_paged", raise_on_error)


def fa_decode_ex(q, k, v, o, lse, seqlens_k, scale: float, workspace, block_table=None, max_pages: int = None,
                 raise_on_error: bool = True) -> int:
    """``fa_decode_ex``: fp16 or bf16 (from q's dtype); q, o [B,Sq,Hq,d]; k, v the caches [B,Smax,Hkv,d] or, with a
    block table, the page pools [num_pages,page_size,Hkv,d]."""
    p = fa_decode_params()
    p.q, p.k, p.v, p.o, p.lse = _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse)
    p.seqlens_k, p.block_table = _ptr(seqlens_k), _ptr(block_table)
    p.B, p.Sq, p.Hq, p.d = q.shape
    p.Hkv = k.shape[2]
    p.dtype = FA_DTYPE_BF16 if q.dtype == torch.bfloat16 else FA_DTYPE_FP16
    if block_table is None:
        p.Skv_max = k.shape[1]
    else:
        p.num_pages, p.page_size = k.shape[0], k.shape[1]
        p.max_pages = block_table.shape[1] if max_pages is None else int(max_pages)
        p.table_stride = block_table.stride(0)
    p.scale = float(scale)
    p.workspace = _ptr(workspace)
    p.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.fa_decode_ex(ctypes.byref(p), _stream())
    return _check(rc, "fa_decode_ex", raise_on_error)


def fa_decode_append_workspace_bytes(B: int, Sq: int, Hq: int, Hkv: int, Skv_max: int, d: int) -> int:
    return int(lib.fa_decode_append_workspace_bytes(B, Sq, Hq, Hkv, Skv_max, d))


def fa_decode_append(q, k_cache, v_cache, o, lse, seqlens_k, scale: float, workspace, raise_on_error: bool = True) -> int:
    """``fa_decode_append``: q, o [B,Sq,Hq,d] (the last Sq positions of every sequence), lse [B,Hq,Sq],
    caches [B,Smax,Hkv,d], seqlens_k int32 [B] on the device (lengths including the Sq new tokens)."""
    B, Sq, Hq, d = q.shape
    _, Smax, Hkv, _ = k_cache.shape
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.fa_decode_append(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse), _ptr(seqlens_k), B, Sq, Hq,
                              Hkv, Smax, d, float(scale), _ptr(workspace), wbytes, _stream())
    return _check(rc, "fa_decode_append", raise_on_error)


def fa_decode_fp8(q, k_cache, v_cache, o, lse, seqlens_k, scale: float, k_scale: float, v_scale: float, workspace,
                  raise_on_error: bool = True) -> int:
    """``fa_decode_fp8``: q [B,1,Hq,d] fp16, caches [B,Smax,Hkv,d] of FP8 e4m3 (``torch.float8_e4m3fn`` or
    uint8 bit patterns) with one factor each, seqlens_k int32 [B] on the device."""
    B, _, Hq, d = q.shape
    _, Smax, Hkv, _ = k_cache.shape
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.fa_decode_fp8(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse), _ptr(seqlens_k), B, Hq, Hkv,
                           Smax, d, float(scale), float(k_scale), float(v_scale), _ptr(workspace), wbytes, _stream())
    return _check(rc, "fa_decode_fp8", raise_on_error)


def fa_decode_fp8_bf16(q, k_cache, v_cache, o, lse, seqlens_k, scale: float, k_scale: float, v_scale: float, workspace,
                       raise_on_error: bool = True) -> int:
    """``fa_decode_fp8_bf16``: as ``fa_decode_fp8`` with q and o in bf16."""
    B, _, Hq, d = q.shape
    _, Smax, Hkv, _ = k_cache.shape
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.fa_decode_fp8_bf16(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse), _ptr(seqlens_k), B, Hq, Hkv,
                                Smax, d, float(scale), float(k_scale), float(v_scale), _ptr(workspace), wbytes, _stream())
    return _check(rc, "fa_decode_fp8_bf16", raise_on_error)


def fa_decode_fp8_paged(q, k_pages, v_pages, block_table, o, lse, seqlens_k, scale: float, k_scale: float,
                        v_scale: float, workspace, max_pages: int = None, raise_on_error: bool = True) -> int:
    """``fa_decode_fp8_paged``: as ``fa_decode_paged`` with pools of FP8 e4m3 bytes and one factor per tensor."""
    B, _, Hq, d = q.shape
    num_pages, page_size, Hkv, _ = k_pages.shape
    stride = block_table.stride(0) if block_table.dim() == 2 else block_table.numel() // max(1, B)
    if max_pages is None:
        max_pages = block_table.shape[1]
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.fa_decode_fp8_paged(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table), _ptr(o), _ptr(lse),
                                 _ptr(seqlens_k), B, Hq, Hkv, num_pages, page_size, int(max_pages), int(stride), d,
                                 float(scale), float(k_scale), float(v_scale), _ptr(workspace), wbytes, _stream())
    return _check(rc, "fa_decode_fp8_paged", raise_on_error)


def fa_decode_fp8_paged_bf16(q, k_pages, v_pages, block_table, o, lse, seqlens_k, scale: float, k_scale: float,
                             v_scale: float, workspace, max_pages: int = None, raise_on_error: bool = True) -> int:
    """``fa_decode_fp8_paged_bf16``: as ``fa_decode_fp8_paged`` with q and o in bf16."""
    B, _, Hq, d = q.shape
    num_pages, page_size, Hkv, _ = k_pages.shape
    stride = block_table.stride(0) if block_table.dim() == 2 else block_table.numel() // max(1, B)
    if max_pages is None:
        max_pages = block_table.shape[1]
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.fa_decode_fp8_paged_bf16(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table), _ptr(o), _ptr(lse),
                                      _ptr(seqlens_k), B, Hq, Hkv, num_pages, page_size, int(max_pages), int(stride), d,
                                      float(scale), float(k_scale), float(v_scale), _ptr(workspace), wbytes, _stream())
    return _check(rc, "fa_decode_fp8_paged_bf16", raise_on_error)


def fa_decode_paged(q, k_pages, v_pages, block_table, o, lse, seqlens_k, scale: float, workspace,
                    max_pages: int = None, raise_on_error: bool = True) -> int:
    """``fa_decode_paged``: q [B,1,Hq,d], page pools [num_pages,page_size,Hkv,d], block_table int32
    [B,table_stride] and seqlens_k int32 [B] on the device; workspace of at least
    ``fa_decode_workspace_bytes(B, Hq, Hkv, max_pages * page_size, d)`` bytes."""
    B, _, Hq, d = q.shape
    num_pages, page_size, Hkv, _ = k_pages.shape
    stride = block_table.stride(0) if block_table.dim() == 2 else block_table.numel() // max(1, B)
    if max_pages is None:
        max_pages = block_table.shape[1]
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib.fa_decode_paged(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table), _ptr(o), _ptr(lse),
                             _ptr(seqlens_k), B, Hq, Hkv, num_pages, page_size, int(max_pages), int(stride), d,
                             float(scale), _ptr(workspace), wbytes, _stream())
    return _check(rc, "fa_decode_paged", raise_on_error)


def fa_decode_noalloc(q, k_cache, v_cache, o, lse, seqlens_k, scale: float, raise_on_error: bool = True) -> int:
    """``fa_decode_noalloc``: decode for callers that may not allocate device memory.  Same
    arguments as ``fa_decode`` minus the workspace; the partial results live in a fixed
    ``FA_DECODE_NOALLOC_BYTES`` array inside the library, shared by all calls (do not overlap
    two calls on the GPU).  Problems whose partials do not fit are refused with FA_ERR_WORKSPACE."""
    B, _, Hq, d = q.shape
    _, Smax, Hkv, _ = k_cache.shape
    rc = lib.fa_decode_noalloc(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(o), _ptr(lse), _ptr(seqlens_k), B,
                               Hq, Hkv, Smax, d, float(scale), _stream())
    return _check(rc, "fa_decode_noalloc", raise_on_error)


def fa_forward_host_staging_bytes(B, Hq, Hkv, Sq, Skv, d) -> int:
    return int(lib.fa_forward_host_staging_bytes(B, Hq, Hkv, Sq, Skv, d))


def fa_forward_host(q_host, k_host, v_host, o_host, lse_host, causal: bool, scale: float, staging,
                    raise_on_error: bool = True) -> int:
    """``fa_forward_host``: q/k/v/o/lse are HOST tensors (pinned for asynchronous copies),
    ``staging`` is a device byte tensor of at least ``fa_forward_host_staging_bytes`` bytes."""
    B, Sq, Hq, d = q_host.shape
    _, Skv, Hkv, _ = k_host.shape
    dt = FA_DTYPE_BF16 if q_host.dtype == torch.bfloat16 else FA_DTYPE_FP16
    rc = lib.fa_forward_host(_ptr(q_host), _ptr(k_host), _ptr(v_host), _ptr(o_host), _ptr(lse_host), B, Hq,
                             Hkv, Sq, Skv, d, int(bool(causal)), float(scale), dt, _ptr(staging),
                             staging.numel() * staging.element_size(), _stream())
    return _check(rc, "fa_forward_host", raise_on_error)


def fa_selftest_wait(limit_us: int, gave_up, raise_on_error: bool = True) -> int:
    """``fa_selftest_wait``: one CTA runs a bounded wait that cannot be satisfied; ``gave_up`` is a zeroed
    uint32/int32 device tensor of one element that ends up holding the number of threads that gave up."""
    rc = lib.fa_selftest_wait(int(limit_us), _ptr(gave_up), _stream())
    return _check(rc, "fa_selftest_wait", raise_on_error)


def fa_device_status():
    """Synchronises, then returns (code, where, block) of the device-side status word and clears it."""
    detail = (ctypes.c_uint * 2)(0, 0)
    rc = int(lib.fa_device_status(ctypes.byref(detail)))
    return rc, int(detail[0]), int(detail[1])
