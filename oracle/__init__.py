"""CPU fp64 oracle for standard attention -- TEST INFRASTRUCTURE ONLY.

Thin ctypes front end of ``attention_oracle.c`` (plain C, compiled with gcc on
first use).  It states the paper's definition of standard attention (Section
5.1), its lower-triangular mask (Section 4.1) and the decode-stage form
(Appendix C) and is what the CUDA library is compared against.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the product never does, and this package never imports the
product.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attention_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None

_DTYPE_CODE = {torch.float16: 0, torch.bfloat16: 1, torch.float32: 2, torch.float64: 3}


def build(force: bool = False) -> str:
    """Compile the C oracle into ``liboracle.so`` next to its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
               "-ffp-contract=off", _SRC, "-o", tmp, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            build()
            lib = ctypes.CDLL(_LIB)
            i32, f64, vp = ctypes.c_int, ctypes.c_double, ctypes.c_void_p
            lib.oracle_attention_full.restype = i32
            lib.oracle_attention_full.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32,
                                                  i32, f64, vp, vp, vp, i32]
            lib.oracle_attention_rows.restype = i32
            lib.oracle_attention_rows.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32,
                                                  i32, f64, vp, vp, i32, vp, vp, i32]
            lib.oracle_decode.restype = i32
            lib.oracle_decode.argtypes = [vp, vp, vp, i32, vp, i32, i32, i32, i32, i32, f64, vp,
                                          vp, vp, i32]
            lib.oracle_bruteforce.restype = i32
            lib.oracle_bruteforce.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, f64,
                                              vp, vp]
            lib.oracle_num_threads.restype = i32
            _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the oracle's parallel loops use by default (OpenMP's count)."""
    return int(_load().oracle_num_threads())


def _as_cpu(t) -> torch.Tensor:
    if isinstance(t, np.ndarray):
        t = torch.from_numpy(t)
    if t.device.type != "cpu":
        raise ValueError("the oracle takes host tensors only")
    if t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("expected a [B, S, H, d] tensor with contiguous d")
    return t


def _strides9(q, k, v):
    s = [q.stride(0), q.stride(1), q.stride(2), k.stride(0), k.stride(1), k.stride(2),
         v.stride(0), v.stride(1), v.stride(2)]
    return np.asarray(s, dtype=np.int64)


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"{what} failed with code {rc}")


def _common(q, k, v):
    q, k, v = _as_cpu(q), _as_cpu(k), _as_cpu(v)
    if not (q.dtype == k.dtype == v.dtype) or q.dtype not in _DTYPE_CODE:
        raise ValueError("q, k, v must share one of fp16 / bf16 / fp32 / fp64")
    B, Sq, Hq, d = q.shape
    Bk, Skv, Hkv, dk = k.shape
    if Bk != B or dk != d or tuple(v.shape) != tuple(k.shape):
        raise ValueError("shape mismatch between q, k, v")
    return q, k, v, B, Sq, Hq, Skv, Hkv, d


def attention_full(q, k, v, causal: bool, scale: float, nthreads: int = 0):
    """Standard attention on the whole problem.

    q ``[B,Sq,Hq,d]``, k and v ``[B,Skv,Hkv,d]`` host tensors.  Returns
    ``(O [B,Sq,Hq,d], LSE [B,Hq,Sq])`` as float64 tensors.
    """
    q, k, v, B, Sq, Hq, Skv, Hkv, d = _common(q, k, v)
    O = torch.zeros(B, Sq, Hq, d, dtype=torch.float64)
    LSE = torch.zeros(B, Hq, Sq, dtype=torch.float64)
    st = _strides9(q, k, v)
    rc = _load().oracle_attention_full(q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                       _DTYPE_CODE[q.dtype], B, Hq, Hkv, Sq, Skv, d,
                                       int(bool(causal)), float(scale), st.ctypes.data,
                                       O.data_ptr(), LSE.data_ptr(), int(nthreads))
    _check(rc, "oracle_attention_full")
    return O, LSE


def attention_rows(q, k, v, causal: bool, scale: float, rows, nthreads: int = 0):
    """Standard attention for chosen rows only.

    ``rows`` is an ``[n,3]`` integer array of (b, h, i).  Returns
    ``(O [n,d], LSE [n])`` as float64 tensors.
    """
    q, k, v, B, Sq, Hq, Skv, Hkv, d = _common(q, k, v)
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int32).reshape(-1, 3))
    n = rows.shape[0]
    O = torch.zeros(n, d, dtype=torch.float64)
    LSE = torch.zeros(n, dtype=torch.float64)
    st = _strides9(q, k, v)
    rc = _load().oracle_attention_rows(q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                       _DTYPE_CODE[q.dtype], B, Hq, Hkv, Sq, Skv, d,
                                       int(bool(causal)), float(scale), st.ctypes.data,
                                       rows.ctypes.data, n, O.data_ptr(), LSE.data_ptr(),
                                       int(nthreads))
    _check(rc, "oracle_attention_rows")
    return O, LSE


def attention_varlen(q, k, v, cu_seqlens_q, cu_seqlens_k, causal: bool, scale: float, nthreads: int = 0):
    """Standard attention on a packed batch: sequence b owns rows ``[cu_q[b], cu_q[b+1])`` of q
    ``[total_q,Hq,d]`` and rows ``[cu_k[b], cu_k[b+1])`` of k, v ``[total_k,Hkv,d]``; each
    sequence is one ``attention_full`` problem.  Returns ``(O [total_q,Hq,d], LSE [Hq,total_q])``
    float64.  A sequence without keys, and rows that see no key, give O = 0 and LSE = -inf."""
    q = torch.as_tensor(q)
    k = torch.as_tensor(k)
    v = torch.as_tensor(v)
    cq = np.asarray(cu_seqlens_q, dtype=np.int64).reshape(-1)
    ck = np.asarray(cu_seqlens_k, dtype=np.int64).reshape(-1)
    if cq.shape != ck.shape or cq[0] != 0 or ck[0] != 0 or cq[-1] != q.shape[0] or ck[-1] != k.shape[0]:
        raise ValueError("prefix sums do not match the packed tensors")
    total_q, Hq, d = q.shape
    O = torch.zeros(total_q, Hq, d, dtype=torch.float64)
    LSE = torch.full((Hq, total_q), float("-inf"), dtype=torch.float64)
    for b in range(cq.shape[0] - 1):
        q0, q1, k0, k1 = int(cq[b]), int(cq[b + 1]), int(ck[b]), int(ck[b + 1])
        if q1 < q0 or k1 < k0:
            raise ValueError("prefix sums must not decrease")
        if q1 == q0 or k1 == k0:
            continue
        n_q, n_k = q1 - q0, k1 - k0
        lo = 0
        if causal and n_q > n_k:
            lo = n_q - n_k          # the first lo rows see no key under the bottom-right mask
        Ob, Lb = attention_full(q[q0 + lo:q1].unsqueeze(0).contiguous(), k[k0:k1].unsqueeze(0).contiguous(),
                                v[k0:k1].unsqueeze(0).contiguous(), causal, scale, nthreads)
        O[q0 + lo:q1] = Ob[0]
        LSE[:, q0 + lo:q1] = Lb[0]
    return O, LSE


def attention_varlen_paged(q, k_pages, v_pages, block_table, cu_seqlens_q, seqlens_k, causal: bool, scale: float,
                           nthreads: int = 0):
    """``attention_varlen`` with the keys and values of every sequence read out of page pools
    ``[num_pages, page_size, Hkv, d]``: key j of sequence b is row ``j % page_size`` of page
    ``block_table[b][j // page_size]``.  The keys are first collected, position by position,
    into packed tensors; the result is ``attention_varlen`` on those."""
    k_pages = torch.as_tensor(k_pages)
    v_pages = torch.as_tensor(v_pages)
    table = np.asarray(block_table, dtype=np.int64)
    sk = np.asarray(seqlens_k, dtype=np.int64).reshape(-1)
    num_pages, page_size, Hkv, d = k_pages.shape
    cu_k = np.concatenate([[0], np.cumsum(sk)])
    k = torch.zeros(int(cu_k[-1]), Hkv, d, dtype=k_pages.dtype)
    v = torch.zeros(int(cu_k[-1]), Hkv, d, dtype=v_pages.dtype)
    for b in range(sk.shape[0]):
        for j in range(int(sk[b])):
            page = int(table[b, j // page_size])
            if not 0 <= page < num_pages:
                raise ValueError(f"sequence {b}: key {j} maps to page {page} outside the pool")
            k[int(cu_k[b]) + j] = k_pages[page, j % page_size]
            v[int(cu_k[b]) + j] = v_pages[page, j % page_size]
    return attention_varlen(q, k, v, cu_seqlens_q, cu_k, causal, scale, nthreads)


def decode(q, k_cache, v_cache, seqlens, scale: float, nthreads: int = 0):
    """Decode-stage attention: q ``[B,1,Hq,d]`` over the first ``seqlens[b]`` rows of
    the ``[B,Smax,Hkv,d]`` caches.  Returns ``(O [B,Hq,d], LSE [B,Hq])`` float64."""
    q, k, v, B, Sq, Hq, Smax, Hkv, d = _common(q, k_cache, v_cache)
    if Sq != 1:
        raise ValueError("decode takes one query row per sequence")
    sl = np.ascontiguousarray(np.asarray(seqlens, dtype=np.int32).reshape(-1))
    if sl.shape[0] != B:
        raise ValueError("seqlens must have B entries")
    O = torch.zeros(B, Hq, d, dtype=torch.float64)
    LSE = torch.zeros(B, Hq, dtype=torch.float64)
    st = _strides9(q, k, v)
    rc = _load().oracle_decode(q.data_ptr(), k.data_ptr(), v.data_ptr(), _DTYPE_CODE[q.dtype],
                               sl.ctypes.data, B, Hq, Hkv, Smax, d, float(scale),
                               st.ctypes.data, O.data_ptr(), LSE.data_ptr(), int(nthreads))
    _check(rc, "oracle_decode")
    return O, LSE


def decode_append(q, k_cache, v_cache, seqlens, scale: float, nthreads: int = 0):
    """Decode after ``Sq`` tokens were appended: q ``[B,Sq,Hq,d]`` holds the queries of the LAST
    ``Sq`` positions of every sequence, whose cache ``[B,Smax,Hkv,d]`` has ``seqlens[b]`` valid
    rows including those positions.  Per sequence this is ``attention_full`` with the causal,
    bottom-right aligned mask over the valid prefix.  Returns ``(O [B,Sq,Hq,d], LSE [B,Hq,Sq])``
    float64; a query that sees no key gives O = 0, LSE = -inf."""
    q = torch.as_tensor(q)
    k = torch.as_tensor(k_cache)
    v = torch.as_tensor(v_cache)
    B, Sq, Hq, d = q.shape
    sl = np.asarray(seqlens, dtype=np.int64).reshape(-1)
    O = torch.zeros(B, Sq, Hq, d, dtype=torch.float64)
    LSE = torch.full((B, Hq, Sq), float("-inf"), dtype=torch.float64)
    for b in range(B):
        n = int(sl[b])
        if n == 0:
            continue
        lo = max(0, Sq - n)                  # queries before position 0 see nothing
        Ob, Lb = attention_full(q[b:b + 1, lo:].contiguous(), k[b:b + 1, :n].contiguous(), v[b:b + 1, :n].contiguous(),
                                True, scale, nthreads)
        O[b, lo:] = Ob[0]
        LSE[b, :, lo:] = Lb[0]
    return O, LSE


def e4m3_to_float64(bits):
    """Value of FP8 e4m3 bit patterns (1 sign, 4 exponent, 3 mantissa bits, exponent bias 7, no
    infinities; exponent 15 with mantissa 7 is NaN), written out from the format's definition.
    ``bits``: uint8 tensor.  Returns float64 of the same shape."""
    b = torch.as_tensor(bits).to(torch.int64)
    sign = torch.where((b >> 7) & 1 == 1, -1.0, 1.0).to(torch.float64)
    e = (b >> 3) & 0xF
    mnt = (b & 0x7).to(torch.float64)
    normal = torch.pow(torch.tensor(2.0, dtype=torch.float64), (e - 7).to(torch.float64)) * (1.0 + mnt / 8.0)
    subnormal = (2.0 ** -6) * (mnt / 8.0)
    val = sign * torch.where(e == 0, subnormal, normal)
    nan = (e == 15) & ((b & 0x7) == 7)
    return torch.where(nan, torch.full_like(val, float("nan")), val)


def attention_proj(q, k, v, w_o, causal: bool, scale: float, nthreads: int = 0):
    """Attention followed by the output projection (Section 4.2's fused attention + Linear on one
    device; Appendix C's last step of the attention block): ``O = attention_full(q, k, v)``, then
    ``out[b, i, :] = O16[b, i, :, :].reshape(Hq * d) @ w_o`` in float64, where ``O16`` is O rounded
    to the operands' 16-bit type -- the operator returns O in that type and the projection reads
    what it returns.  ``w_o``: ``[Hq*d, d_model]``.  Returns ``(O, LSE, out)`` float64, O unrounded."""
    O, LSE = attention_full(q, k, v, causal, scale, nthreads)
    q = torch.as_tensor(q)
    w = torch.as_tensor(w_o).to(torch.float64)
    B, Sq, Hq, d = O.shape
    if w.shape[0] != Hq * d:
        raise ValueError("w_o must have Hq * d rows")
    O16 = O.to(q.dtype).to(torch.float64) if q.dtype in (torch.float16, torch.bfloat16) else O
    out = torch.matmul(O16.reshape(B, Sq, Hq * d), w)
    return O, LSE, out


def attention_fp8(q_bits, k_bits, v_bits, causal: bool, scale: float, q_scale: float, k_scale: float,
                  v_scale: float, rows=None, abs_v: bool = False, nthreads: int = 0):
    """Standard attention on FP8 e4m3 operands (Appendix D.2 runs the operator on 8-bit
    operands): ``attention_full`` -- or ``attention_rows`` when ``rows`` is given -- on
    Q = q_scale * value(q_bits), K = k_scale * value(k_bits), V = v_scale * value(v_bits), all
    widened exactly and evaluated in float64.  Nothing here is rounded to 8 bits: the
    probabilities stay float64, so a kernel that rounds them differs by what that rounding costs.
    ``abs_v`` evaluates with |V| in place of V (the weight sum_j P_ij |V_j| that bounds it).
    ``*_bits``: uint8 ``[B,S,H,d]``."""
    q = (e4m3_to_float64(q_bits) * float(q_scale)).contiguous()
    k = (e4m3_to_float64(k_bits) * float(k_scale)).contiguous()
    v = (e4m3_to_float64(v_bits) * float(v_scale)).contiguous()
    if abs_v:
        v = v.abs()
    if rows is None:
        return attention_full(q, k, v, causal, scale, nthreads)
    return attention_rows(q, k, v, causal, scale, rows, nthreads)


def decode_fp8(q, k_bits, v_bits, seqlens, scale: float, k_scale: float, v_scale: float, nthreads: int = 0):
    """Decode-stage attention over an FP8 e4m3 cache: ``decode`` on K = k_scale * value(k_bits),
    V = v_scale * value(v_bits), evaluated in float64 (Appendix D.2 runs the operator on 8-bit
    operands; the widening itself is exact).  ``k_bits``/``v_bits``: uint8 ``[B,Smax,Hkv,d]``.
    Rows at or beyond ``seqlens[b]`` are replaced by zeros first (they may hold NaN patterns and
    are never used)."""
    q = torch.as_tensor(q).to(torch.float64)
    k = e4m3_to_float64(k_bits) * float(k_scale)
    v = e4m3_to_float64(v_bits) * float(v_scale)
    sl = np.asarray(seqlens, dtype=np.int64).reshape(-1)
    for b in range(k.shape[0]):
        k[b, int(sl[b]):] = 0.0
        v[b, int(sl[b]):] = 0.0
    return decode(q, k.contiguous(), v.contiguous(), sl.astype(np.int32), scale, nthreads)


def decode_paged(q, k_pages, v_pages, block_table, seqlens, scale: float, nthreads: int = 0):
    """Decode-stage attention over a paged cache (the decode computation of Appendix C; only
    the addressing differs): key j of sequence b is row ``j % page_size`` of page
    ``block_table[b][j // page_size]`` of the ``[num_pages, page_size, Hkv, d]`` pools.  The
    keys and values of every sequence are first collected, position by position, into
    contiguous caches; the result is then ``decode`` on those.  Positions at or beyond
    ``seqlens[b]`` are filled with zeros (they are never read by ``decode``)."""
    k_pages = torch.as_tensor(k_pages)
    v_pages = torch.as_tensor(v_pages)
    table = np.asarray(block_table, dtype=np.int64)
    sl = np.asarray(seqlens, dtype=np.int64).reshape(-1)
    num_pages, page_size, Hkv, d = k_pages.shape
    B = sl.shape[0]
    Smax = max(1, int(sl.max()) if B else 1)
    k = torch.zeros(B, Smax, Hkv, d, dtype=k_pages.dtype)
    v = torch.zeros(B, Smax, Hkv, d, dtype=v_pages.dtype)
    for b in range(B):
        for j in range(int(sl[b])):
            page = int(table[b, j // page_size])
            if not 0 <= page < num_pages:
                raise ValueError(f"sequence {b}: key {j} maps to page {page} outside the pool")
            k[b, j] = k_pages[page, j % page_size]
            v[b, j] = v_pages[page, j % page_size]
    return decode(q, k, v, sl.astype(np.int32), scale, nthreads)


def bruteforce(q, k, v, causal: bool, scale: float):
    """Extended-precision direct evaluation for tiny inputs (d <= 64): exp(s)/sum exp(s)
    with no max subtraction.  Inputs are converted to contiguous float64."""
    q = torch.as_tensor(q).to(torch.float64).contiguous()
    k = torch.as_tensor(k).to(torch.float64).contiguous()
    v = torch.as_tensor(v).to(torch.float64).contiguous()
    B, Sq, Hq, d = q.shape
    _, Skv, Hkv, _ = k.shape
    O = torch.zeros(B, Sq, Hq, d, dtype=torch.float64)
    LSE = torch.zeros(B, Hq, Sq, dtype=torch.float64)
    rc = _load().oracle_bruteforce(q.data_ptr(), k.data_ptr(), v.data_ptr(), B, Hq, Hkv, Sq,
                                   Skv, d, int(bool(causal)), float(scale), O.data_ptr(),
                                   LSE.data_ptr())
    _check(rc, "oracle_bruteforce")
    return O, LSE
