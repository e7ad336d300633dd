"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def fa():
    from paper_2410_16663_b200 import build
    build.build()
    from paper_2410_16663_b200 import binding
    return binding


def header_functions():
    text = open(os.path.join(ROOT, "include", "fa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fa_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(fa):
    names = header_functions()
    assert "fa_forward" in names and "fa_decode" in names and len(names) >= 10
    for n in names:
        assert hasattr(fa.lib, n), f"{n} declared in include/fa.h but not exported"
    assert sorted(fa.EXPORTS) == sorted(n for n in names)


def test_version_and_strerror(fa):
    assert fa.fa_version() >= 100
    for code in range(0, -9, -1):
        assert fa.fa_strerror(code) and "unknown" not in fa.fa_strerror(code)
    assert "unknown" in fa.fa_strerror(-99)


def _t(*shape, dtype=torch.float16):
    return torch.zeros(*shape, dtype=dtype)


def test_forward_validation_happens_before_any_cuda_call(fa):
    q, k = _t(1, 4, 4, 128), _t(1, 4, 2, 128)
    o = _t(1, 4, 4, 128)
    L = fa.lib
    P = lambda t: t.data_ptr()
    # no-ops
    assert L.fa_forward(P(q), P(k), P(k), P(o), None, 0, 4, 2, 4, 4, 128, 1, 0.1, None) == fa.FA_OK
    assert L.fa_forward(P(q), P(k), P(k), P(o), None, 1, 4, 2, 0, 4, 128, 1, 0.1, None) == fa.FA_OK
    # shapes
    assert L.fa_forward(P(q), P(k), P(k), P(o), None, 1, 3, 2, 4, 4, 128, 1, 0.1, None) == fa.FA_ERR_SHAPE
    assert L.fa_forward(P(q), P(k), P(k), P(o), None, -1, 4, 2, 4, 4, 128, 1, 0.1, None) == fa.FA_ERR_SHAPE
    assert L.fa_forward(P(q), P(k), P(k), P(o), None, 1, 4, 0, 4, 4, 128, 1, 0.1, None) == fa.FA_ERR_SHAPE
    # unsupported
    assert L.fa_forward(P(q), P(k), P(k), P(o), None, 1, 4, 2, 4, 4, 96, 1, 0.1, None) == fa.FA_ERR_UNSUPPORTED
    assert L.fa_forward(P(q), P(k), P(k), P(o), None, 1, 4, 2, 4, 4, 512, 1, 0.1, None) == fa.FA_ERR_UNSUPPORTED
    assert L.fa_forward(P(q), P(k), P(k), P(o), None, 1, 4, 2, 5, 4, 128, 1, 0.1, None) == fa.FA_ERR_UNSUPPORTED
    assert L.fa_forward(P(q), P(k), P(k), P(o), None, 1, 4, 2, 4, 4, 128, 1, -1.0, None) == fa.FA_ERR_UNSUPPORTED
    assert L.fa_forward(P(q), P(k), P(k), P(o), None, 1, 4, 2, 4, 4, 128, 1, float("nan"), None) == fa.FA_ERR_UNSUPPORTED
    # null / alignment
    assert L.fa_forward(None, P(k), P(k), P(o), None, 1, 4, 2, 4, 4, 128, 1, 0.1, None) == fa.FA_ERR_NULL
    assert L.fa_forward(P(q), None, P(k), P(o), None, 1, 4, 2, 4, 4, 128, 1, 0.1, None) == fa.FA_ERR_NULL
    assert L.fa_forward(P(q), P(k), P(k), None, None, 1, 4, 2, 4, 4, 128, 1, 0.1, None) == fa.FA_ERR_NULL
    assert L.fa_forward(P(q) + 2, P(k), P(k), P(o), None, 1, 4, 2, 4, 4, 128, 1, 0.1, None) == fa.FA_ERR_ALIGN
    assert L.fa_forward_bf16(P(q), P(k), P(k), P(o) + 8, None, 1, 4, 2, 4, 4, 128, 1, 0.1, None) == fa.FA_ERR_ALIGN
    assert L.fa_forward_ex(None, None) == fa.FA_ERR_NULL


def test_forward_ex_rejects_bad_strides_and_types(fa):
    q = _t(1, 4, 4, 128)
    p = fa.fa_params()
    p.q = p.k = p.v = p.o = q.data_ptr()
    p.B, p.Hq, p.Hkv, p.Sq, p.Skv, p.d = 1, 4, 4, 4, 4, 128
    p.scale, p.dtype, p.o_dtype = 0.1, fa.FA_DTYPE_FP16, fa.FA_DTYPE_FP16
    p.q_stride[0], p.q_stride[1], p.q_stride[2] = 2048, 512, 100   # head stride not a multiple of 8
    assert fa.lib.fa_forward_ex(ctypes.byref(p), None) == fa.FA_ERR_SHAPE
    p.q_stride[2] = 128
    p.dtype = 7
    assert fa.lib.fa_forward_ex(ctypes.byref(p), None) == fa.FA_ERR_UNSUPPORTED
    p.dtype, p.o_dtype = fa.FA_DTYPE_FP16, fa.FA_DTYPE_BF16
    assert fa.lib.fa_forward_ex(ctypes.byref(p), None) == fa.FA_ERR_UNSUPPORTED
    p.o_dtype, p.variant = fa.FA_DTYPE_FP16, 0


def test_decode_validation_and_workspace_size(fa):
    L = fa.lib
    q, kc, o = _t(2, 1, 8, 128), _t(2, 256, 2, 128), _t(2, 1, 8, 128)
    sl = torch.zeros(2, dtype=torch.int32)
    ws = torch.zeros(1 << 16, dtype=torch.uint8)
    P = lambda t: t.data_ptr()
    need = fa.fa_decode_workspace_bytes(2, 8, 2, 256, 128)
    assert need == 2 * 8 * 1 * 129 * 4
    assert fa.fa_decode_workspace_bytes(2, 8, 2, 256, 64) == 2 * 8 * 1 * 65 * 4    # head dimension 64: its own partials
    assert fa.fa_decode_workspace_bytes(2, 8, 2, 256, 256) == 0 and fa.fa_decode_workspace_bytes(2, 8, 2, 256, 96) == 0
    # large problems use 2048-key chunks
    assert fa.fa_decode_workspace_bytes(64, 32, 32, 32768, 128) == 64 * 32 * 16 * 129 * 4
    args = lambda **kw: None
    assert L.fa_decode(P(q), P(kc), P(kc), P(o), None, P(sl), 2, 8, 3, 256, 128, 0.1, P(ws), need, None) == fa.FA_ERR_SHAPE
    assert L.fa_decode(P(q), P(kc), P(kc), P(o), None, P(sl), 2, 8, 2, 256, 96, 0.1, P(ws), need, None) == fa.FA_ERR_UNSUPPORTED
    assert L.fa_decode(P(q), P(kc), P(kc), P(o), None, None, 2, 8, 2, 256, 128, 0.1, P(ws), need, None) == fa.FA_ERR_NULL
    assert L.fa_decode(P(q), P(kc), P(kc), P(o), None, P(sl), 2, 8, 2, 256, 128, 0.1, P(ws), need - 1, None) == fa.FA_ERR_WORKSPACE
    assert L.fa_decode(P(q), P(kc), P(kc), P(o), None, P(sl), 2, 8, 2, 256, 128, 0.1, None, 0, None) == fa.FA_ERR_WORKSPACE
    assert L.fa_decode(P(q), P(kc), P(kc), P(o), None, P(sl), 2, 8, 2, 256, 128, 0.1, P(ws) + 4, need, None) == fa.FA_ERR_ALIGN
    assert L.fa_decode(P(q), P(kc), P(kc), P(o), None, P(sl), 0, 8, 2, 256, 128, 0.1, P(ws), need, None) == fa.FA_OK


def test_varlen_validation(fa):
    L = fa.lib
    q, k, o = _t(20, 4, 128), _t(30, 2, 128), _t(20, 4, 128)
    cu = torch.zeros(3, dtype=torch.int32)
    P = lambda t: t.data_ptr()
    call = lambda **kw: L.fa_forward_varlen(
        kw.get("q", P(q)), P(k), P(k), P(o), None, kw.get("cu", P(cu)), P(cu), kw.get("B", 2), 4, kw.get("Hkv", 2),
        20, 30, kw.get("max_q", 12), kw.get("max_k", 16), kw.get("d", 128), 1, kw.get("scale", 0.1),
        kw.get("dtype", fa.FA_DTYPE_FP16), None)
    assert call(Hkv=3) == fa.FA_ERR_SHAPE
    assert call(max_q=21) == fa.FA_ERR_SHAPE
    assert call(max_k=31) == fa.FA_ERR_SHAPE
    assert call(d=96) == fa.FA_ERR_UNSUPPORTED and call(d=256) == fa.FA_ERR_UNSUPPORTED   # 128 and 64 are taken
    assert call(dtype=fa.FA_DTYPE_FP32) == fa.FA_ERR_UNSUPPORTED
    assert call(scale=float("nan")) == fa.FA_ERR_UNSUPPORTED
    assert call(cu=None) == fa.FA_ERR_NULL
    assert call(q=None) == fa.FA_ERR_NULL
    assert call(q=P(q) + 8) == fa.FA_ERR_ALIGN
    assert call(cu=P(cu) + 2) == fa.FA_ERR_ALIGN
    assert call(B=0) == fa.FA_OK
    assert call(max_q=0) == fa.FA_OK


def test_decode_ex_validation(fa):
    q, kc, o = _t(2, 1, 8, 128), _t(2, 256, 2, 128), _t(2, 1, 8, 128)
    sl = torch.zeros(2, dtype=torch.int32)
    table = torch.zeros(2, 2, dtype=torch.int32)
    ws = torch.zeros(1 << 16, dtype=torch.uint8)
    assert fa.lib.fa_decode_ex(None, None) == fa.FA_ERR_NULL

    def call(**kw):
        p = fa.fa_decode_params()
        p.q, p.k, p.v, p.o, p.seqlens_k = q.data_ptr(), kc.data_ptr(), kc.data_ptr(), o.data_ptr(), sl.data_ptr()
        p.B, p.Sq, p.Hq, p.Hkv, p.Skv_max, p.d = 2, 1, 8, 2, 256, 128
        p.dtype, p.scale = fa.FA_DTYPE_FP16, 0.1
        p.workspace, p.workspace_bytes = ws.data_ptr(), ws.numel()
        for key, val in kw.items():
            setattr(p, key, val)
        return fa.lib.fa_decode_ex(ctypes.byref(p), None)

    assert call(dtype=fa.FA_DTYPE_FP32) == fa.FA_ERR_UNSUPPORTED
    assert call(Hkv=3) == fa.FA_ERR_SHAPE
    assert call(Sq=65) == fa.FA_ERR_UNSUPPORTED
    assert call(workspace_bytes=8) == fa.FA_ERR_WORKSPACE
    assert call(block_table=table.data_ptr(), num_pages=4, page_size=48, max_pages=2, table_stride=2) == fa.FA_ERR_SHAPE
    assert call(block_table=table.data_ptr(), num_pages=4, page_size=128, max_pages=2, table_stride=1) == fa.FA_ERR_SHAPE
    assert call(B=0) == fa.FA_OK


def test_decode_append_validation(fa):
    L = fa.lib
    q, kc, o = _t(2, 4, 8, 128), _t(2, 256, 2, 128), _t(2, 4, 8, 128)
    sl = torch.zeros(2, dtype=torch.int32)
    ws = torch.zeros(1 << 18, dtype=torch.uint8)
    P = lambda t: t.data_ptr()
    need = fa.fa_decode_append_workspace_bytes(2, 4, 8, 2, 256, 128)
    assert need == 4 * fa.fa_decode_workspace_bytes(2, 8, 2, 256, 128)
    call = lambda **kw: L.fa_decode_append(P(q), P(kc), P(kc), P(o), None, P(sl), kw.get("B", 2), kw.get("Sq", 4), 8,
                                           kw.get("Hkv", 2), kw.get("Smax", 256), 128, 0.1, P(ws), kw.get("wbytes", need), None)
    assert call(Sq=0) == fa.FA_ERR_SHAPE
    assert call(Sq=65) == fa.FA_ERR_UNSUPPORTED
    assert call(Sq=4, Smax=3) == fa.FA_ERR_UNSUPPORTED
    assert call(Hkv=3) == fa.FA_ERR_SHAPE
    assert call(wbytes=need - 1) == fa.FA_ERR_WORKSPACE
    assert call(B=0) == fa.FA_OK


def test_fp8_decode_validation(fa):
    L = fa.lib
    q, o = _t(2, 1, 8, 128), _t(2, 1, 8, 128)
    kc = torch.zeros(2, 256, 2, 128, dtype=torch.uint8)
    sl = torch.zeros(2, dtype=torch.int32)
    ws = torch.zeros(1 << 16, dtype=torch.uint8)
    P = lambda t: t.data_ptr()
    need = fa.fa_decode_workspace_bytes(2, 8, 2, 256, 128)
    for entry in (L.fa_decode_fp8, L.fa_decode_fp8_bf16):   # the bf16 form shares every check
        call = lambda **kw: entry(P(q), P(kc), P(kc), P(o), None, kw.get("sl", P(sl)), kw.get("B", 2), 8,
                                  kw.get("Hkv", 2), 256, kw.get("d", 128), 0.1, kw.get("ks", 1.0), kw.get("vs", 1.0),
                                  P(ws), kw.get("wbytes", need), None)
        assert call(Hkv=3) == fa.FA_ERR_SHAPE
        assert call(d=64) == fa.FA_ERR_UNSUPPORTED
        assert call(ks=0.0) == fa.FA_ERR_UNSUPPORTED
        assert call(vs=float("inf")) == fa.FA_ERR_UNSUPPORTED
        assert call(ks=float("nan")) == fa.FA_ERR_UNSUPPORTED
        assert call(sl=None) == fa.FA_ERR_NULL
        assert call(wbytes=need - 1) == fa.FA_ERR_WORKSPACE
        assert call(B=0) == fa.FA_OK
    table = torch.zeros(2, 1, dtype=torch.int32)
    for entry in (L.fa_decode_fp8_paged, L.fa_decode_fp8_paged_bf16):
        paged = lambda **kw: entry(P(q), P(kc), P(kc), kw.get("table", P(table)), P(o), None, P(sl), 2, 8, 2, 2,
                                   kw.get("page_size", 256), 1, kw.get("stride", 1), 128, 0.1, 1.0, 1.0, P(ws), need, None)
        assert paged(page_size=48) == fa.FA_ERR_SHAPE
        assert paged(stride=0) == fa.FA_ERR_SHAPE
        assert paged(table=None) == fa.FA_ERR_NULL


def test_varlen_paged_validation(fa):
    L = fa.lib
    q, pool, o = _t(20, 4, 128), _t(6, 128, 2, 128), _t(20, 4, 128)
    cu = torch.zeros(3, dtype=torch.int32)
    sk = torch.zeros(2, dtype=torch.int32)
    table = torch.zeros(2, 3, dtype=torch.int32)
    P = lambda t: t.data_ptr()
    call = lambda **kw: L.fa_forward_varlen_paged(
        P(q), P(pool), P(pool), kw.get("table", P(table)), P(o), None, P(cu), P(sk), kw.get("B", 2), 4, 2, 20, 6,
        kw.get("page_size", 128), 3, kw.get("stride", 3), 12, kw.get("max_k", 300), 128, 1, 0.1, fa.FA_DTYPE_FP16, None)
    assert call(page_size=64) == fa.FA_ERR_SHAPE
    assert call(stride=2) == fa.FA_ERR_SHAPE
    assert call(max_k=3 * 128 + 1) == fa.FA_ERR_SHAPE
    assert call(table=None) == fa.FA_ERR_NULL
    assert call(B=0) == fa.FA_OK


def test_paged_decode_validation(fa):
    L = fa.lib
    q, pool, o = _t(2, 1, 8, 128), _t(6, 128, 2, 128), _t(2, 1, 8, 128)
    sl = torch.zeros(2, dtype=torch.int32)
    table = torch.zeros(2, 3, dtype=torch.int32)
    ws = torch.zeros(1 << 16, dtype=torch.uint8)
    P = lambda t: t.data_ptr()
    need = fa.fa_decode_workspace_bytes(2, 8, 2, 3 * 128, 128)
    call = lambda **kw: L.fa_decode_paged(
        P(q), P(pool), P(pool), kw.get("table", P(table)), P(o), None, P(sl), kw.get("B", 2), 8, kw.get("Hkv", 2),
        kw.get("num_pages", 6), kw.get("page_size", 128), kw.get("max_pages", 3), kw.get("stride", 3), 128, 0.1,
        P(ws), kw.get("wbytes", need), None)
    assert call(page_size=48) == fa.FA_ERR_SHAPE        # neither a multiple of the 128-key tile nor 16, 32, 64
    assert call(page_size=8) == fa.FA_ERR_SHAPE
    assert call(page_size=192) == fa.FA_ERR_SHAPE
    assert call(page_size=0) == fa.FA_ERR_SHAPE
    assert call(stride=2) == fa.FA_ERR_SHAPE            # rows of the table overlap
    assert call(num_pages=0) == fa.FA_ERR_SHAPE
    assert call(table=None) == fa.FA_ERR_NULL
    assert call(table=P(table) + 2) == fa.FA_ERR_ALIGN
    assert call(Hkv=3) == fa.FA_ERR_SHAPE
    assert call(wbytes=need - 1) == fa.FA_ERR_WORKSPACE
    assert call(B=0) == fa.FA_OK


def test_host_entry_validation(fa):
    L = fa.lib
    q = _t(1, 4, 4, 128)
    P = lambda t: t.data_ptr()
    need = fa.fa_forward_host_staging_bytes(1, 4, 4, 4, 4, 128)
    assert need >= 4 * (4 * 4 * 128 * 2)
    assert L.fa_forward_host(P(q), P(q), P(q), P(q), None, 1, 4, 4, 4, 4, 128, 1, 0.1, 0, None, 0, None) == fa.FA_ERR_WORKSPACE
    assert L.fa_forward_host(None, P(q), P(q), P(q), None, 1, 4, 4, 4, 4, 128, 1, 0.1, 0, None, 0, None) == fa.FA_ERR_NULL
    assert L.fa_forward_host(P(q), P(q), P(q), P(q), None, 1, 4, 4, 4, 4, 128, 1, 0.1, 5, None, 0, None) == fa.FA_ERR_UNSUPPORTED
    # head dimensions: the ones fa_forward takes, with a staging area that follows d
    up = lambda x: (x + 1023) // 1024 * 1024
    for d in (64, 128, 256):
        assert fa.fa_forward_host_staging_bytes(2, 4, 2, 5, 7, d) == 2 * up(2 * 5 * 4 * d * 2) + 2 * up(2 * 7 * 2 * d * 2) + up(2 * 4 * 5 * 4)
    assert fa.fa_forward_host_staging_bytes(1, 4, 4, 4, 4, 96) == 0
    assert L.fa_forward_host(P(q), P(q), P(q), P(q), None, 1, 4, 4, 4, 4, 96, 1, 0.1, 0, None, 0, None) == fa.FA_ERR_UNSUPPORTED
    assert L.fa_forward_host(P(q), P(q), P(q), P(q), None, 1, 4, 4, 4, 4, 64, 1, 0.1, 0, None, 0, None) == fa.FA_ERR_WORKSPACE


def test_binding_fails_loudly_without_the_library(tmp_path, monkeypatch):
    # the binding has no fallback: a missing library is an ImportError at import time
    import importlib.util
    src = os.path.join(ROOT, "paper_2410_16663_b200", "binding.py")
    dst = tmp_path / "binding_copy.py"
    dst.write_text(open(src).read())
    spec = importlib.util.spec_from_file_location("binding_copy", str(dst))
    mod = importlib.util.module_from_spec(spec)
    with pytest.raises(ImportError):
        spec.loader.exec_module(mod)


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2410_16663_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "oracle/" not in text, f


def test_selftest_wait_validates_before_any_cuda_call(fa):
    c = torch.zeros(4, dtype=torch.int32)
    assert fa.lib.fa_selftest_wait(1000, None, None) == fa.FA_ERR_NULL
    assert fa.lib.fa_selftest_wait(1000, c.data_ptr() + 2, None) == fa.FA_ERR_ALIGN
    assert fa.lib.fa_selftest_wait(0, c.data_ptr(), None) == fa.FA_ERR_UNSUPPORTED
    assert fa.lib.fa_selftest_wait(100001, c.data_ptr(), None) == fa.FA_ERR_UNSUPPORTED


def test_forward_fp8_validation(fa):
    q = torch.zeros(1, 4, 4, 128, dtype=torch.uint8)
    o = torch.zeros(1, 4, 4, 128, dtype=torch.float16)
    P = lambda t: t.data_ptr()
    L = fa.lib.fa_forward_fp8
    ok = dict(B=1, Hq=4, Hkv=2, Sq=4, Skv=4, d=128, causal=1, scale=0.1, qs=0.5, ks=0.5, vs=0.5, od=fa.FA_DTYPE_FP16)
    def call(qp=P(q), kp=P(q), vp=P(q), op=P(o), **kw):
        a = dict(ok); a.update(kw)
        return L(qp, kp, vp, op, None, a["B"], a["Hq"], a["Hkv"], a["Sq"], a["Skv"], a["d"], a["causal"], a["scale"],
                 a["qs"], a["ks"], a["vs"], a["od"], None)
    assert call(B=0) == fa.FA_OK and call(Sq=0) == fa.FA_OK
    assert call(Hq=3) == fa.FA_ERR_SHAPE and call(B=-1) == fa.FA_ERR_SHAPE
    assert call(d=64) == fa.FA_ERR_UNSUPPORTED and call(od=fa.FA_DTYPE_FP32) == fa.FA_ERR_UNSUPPORTED
    assert call(Sq=5) == fa.FA_ERR_UNSUPPORTED                       # causal with more queries than keys
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        assert call(qs=bad) == fa.FA_ERR_UNSUPPORTED and call(ks=bad) == fa.FA_ERR_UNSUPPORTED
        assert call(vs=bad) == fa.FA_ERR_UNSUPPORTED
    assert call(scale=-0.1) == fa.FA_ERR_UNSUPPORTED
    assert call(qp=None) == fa.FA_ERR_NULL and call(op=None) == fa.FA_ERR_NULL and call(kp=None) == fa.FA_ERR_NULL
    assert call(qp=P(q) + 4) == fa.FA_ERR_ALIGN and call(op=P(o) + 2) == fa.FA_ERR_ALIGN


def test_forward_proj_validation(fa):
    q = torch.zeros(1, 4, 4, 128, dtype=torch.float16)
    w = torch.zeros(512, 256, dtype=torch.float16)
    out = torch.zeros(1, 4, 256, dtype=torch.float16)
    ws = torch.zeros(64, dtype=torch.uint8)
    P = lambda t: t.data_ptr()
    L = fa.lib.fa_forward_proj
    def call(qp=P(q), wp=P(w), op=P(q), outp=P(out), wsp=P(ws), wsn=64, **kw):
        a = dict(B=1, Hq=4, Hkv=2, Sq=4, Skv=4, d=128, dm=256, causal=1, scale=0.1, dt=fa.FA_DTYPE_FP16, fused=1)
        a.update(kw)
        return L(qp, P(q), P(q), wp, op, None, outp, a["B"], a["Hq"], a["Hkv"], a["Sq"], a["Skv"], a["d"], a["dm"],
                 a["causal"], a["scale"], a["dt"], a["fused"], wsp, wsn, None)
    assert fa.lib.fa_forward_proj_workspace_bytes(1, 4) == 4 and fa.lib.fa_forward_proj_workspace_bytes(3, 300) == 36
    assert fa.lib.fa_forward_proj_workspace_bytes(0, 4) == 0
    assert call(B=0) == fa.FA_OK and call(Sq=0) == fa.FA_OK
    assert call(Hq=3) == fa.FA_ERR_SHAPE and call(dm=0) == fa.FA_ERR_SHAPE
    assert call(dm=200) == fa.FA_ERR_UNSUPPORTED and call(d=64) == fa.FA_ERR_UNSUPPORTED
    assert call(dt=fa.FA_DTYPE_FP32) == fa.FA_ERR_UNSUPPORTED and call(Sq=5) == fa.FA_ERR_UNSUPPORTED
    assert call(scale=float("nan")) == fa.FA_ERR_UNSUPPORTED
    assert call(qp=None) == fa.FA_ERR_NULL and call(wp=None) == fa.FA_ERR_NULL and call(outp=None) == fa.FA_ERR_NULL
    assert call(outp=P(out) + 16) == fa.FA_ERR_ALIGN and call(wp=P(w) + 2) == fa.FA_ERR_ALIGN
    assert call(wsp=None) == fa.FA_ERR_WORKSPACE and call(wsn=2) == fa.FA_ERR_WORKSPACE
    assert call(wsp=P(ws) + 1) == fa.FA_ERR_ALIGN
