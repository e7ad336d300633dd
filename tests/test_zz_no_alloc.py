"""fa_decode_noalloc: the decode entry point for callers that cannot allocate device memory
(code living inside someone else's memory pool, a serving loop that must never hit the
allocator, a plugin that only receives buffers).  Its partial results go to a fixed array inside
the library instead of a caller workspace, so the test checks two things: the results equal
those of fa_decode, and a second call right after the first (different lengths, so different
slots of the shared array are live) is just as correct, i.e. nothing depends on what the
previous call left behind.  Both calls are also compared with the CPU oracle.  The file name keeps this test last in collection order."""
import pytest
import torch

import oracle
from paper_2410_16663_b200 import inputs as synth
from tests.util import assert_close_to_oracle


@pytest.fixture(scope="module")
def fa():
    from paper_2410_16663_b200 import binding
    return binding


def test_noalloc_refuses_problems_larger_than_its_fixed_scratch(fa):
    # validated before any CUDA call, so this part runs without a GPU as well
    q = torch.zeros(64, 1, 32, 128, dtype=torch.float16)
    need = fa.fa_decode_workspace_bytes(64, 32, 32, 32768, 128)
    assert need > fa.FA_DECODE_NOALLOC_BYTES
    rc = fa.lib.fa_decode_noalloc(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None, q.data_ptr(),
                                  64, 32, 32, 32768, 128, 0.1, None)
    assert rc == fa.FA_ERR_WORKSPACE
    assert fa.lib.fa_decode_noalloc(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), None, q.data_ptr(),
                                    2, 6, 4, 128, 128, 0.1, None) == fa.FA_ERR_SHAPE


def test_noalloc_checks_its_arguments_like_fa_decode_before_any_cuda_call(fa):
    # the same refusals with the same codes as fa_decode, found before the scratch's device address
    # is looked up: this runs on a machine without a GPU or a driver
    buf = torch.zeros(4096, dtype=torch.float16)
    ws = torch.zeros(1 << 16, dtype=torch.uint8)
    ok = buf.data_ptr()
    assert ok % 16 == 0
    cases = [
        dict(q=None),                              # NULL q
        dict(o=None),
        dict(seqlens=None),
        dict(k=None),
        dict(q=ok + 2),                            # misaligned pointers
        dict(v=ok + 8),
        dict(scale=-1.0),                          # negative and non-finite scales
        dict(scale=float("inf")),
        dict(scale=float("nan")),
        dict(Hq=6, Hkv=4),
        dict(d=96),                                # a head dimension other than 128 and 64
        dict(d=256),
        dict(B=70000),
        dict(Skv_max=0),
    ]
    for c in cases:
        a = dict(q=ok, k=ok, v=ok, o=ok, lse=None, seqlens=ok, B=1, Hq=2, Hkv=1, Skv_max=256, d=128, scale=0.1)
        a.update(c)
        rc_ws = fa.lib.fa_decode(a["q"], a["k"], a["v"], a["o"], a["lse"], a["seqlens"], a["B"], a["Hq"], a["Hkv"],
                                 a["Skv_max"], a["d"], a["scale"], ws.data_ptr(), ws.numel(), None)
        rc_na = fa.lib.fa_decode_noalloc(a["q"], a["k"], a["v"], a["o"], a["lse"], a["seqlens"], a["B"], a["Hq"],
                                         a["Hkv"], a["Skv_max"], a["d"], a["scale"], None)
        assert rc_ws < 0 and rc_ws != fa.FA_ERR_CUDA and rc_ws != fa.FA_ERR_DEVICE, (c, rc_ws)
        assert rc_na == rc_ws, (c, rc_na, rc_ws)
    # B == 0 is a successful no-op for both, whatever the pointers
    assert fa.lib.fa_decode_noalloc(None, None, None, None, None, None, 0, 2, 1, 256, 128, 0.1, None) == 0


@pytest.mark.gpu
@pytest.mark.parametrize("d", [128, 64])
def test_noalloc_matches_fa_decode_on_two_calls_in_a_row(fa, d):
    dev = "cuda"
    cfg = synth.DecodeConfig("noalloc", 6, 8, 2, 5000, 1, 5000, d=d, seed=808)
    q, k, v, sl = synth.decode_inputs(cfg, dev, poison=False)  # the second call reads other lengths
    assert fa.fa_decode_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Smax, cfg.d) <= fa.FA_DECODE_NOALLOC_BYTES
    ws = torch.empty(fa.fa_decode_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Smax, cfg.d), dtype=torch.uint8,
                     device=dev)
    lens_a = sl.clone()
    lens_b = torch.tensor([5000, 1, 0, 2049, 300, 4097], dtype=torch.int32)
    qc, kc, vc = q.cpu(), k.cpu(), v.cpu()
    for lens in (lens_a, lens_b):            # two calls in a row on the shared scratch
        sld = lens.to(dev)
        o_ref = torch.empty_like(q)
        l_ref = torch.empty(cfg.B, cfg.Hq, dtype=torch.float32, device=dev)
        fa.fa_decode(q, k, v, o_ref, l_ref, sld, cfg.scale, ws)
        o = torch.full_like(q, float("nan"))
        lse = torch.full((cfg.B, cfg.Hq), float("nan"), dtype=torch.float32, device=dev)
        fa.fa_decode_noalloc(q, k, v, o, lse, sld, cfg.scale)
        torch.cuda.synchronize()
        rc, where, blk = fa.fa_device_status()
        assert rc == 0, (rc, where, blk)
        # the same kernels in the same order on the same inputs: bit for bit what fa_decode gives
        # (a stale partial of the previous call leaking into the merge, however small its weight,
        # would break this)
        assert torch.equal(o, o_ref)
        assert torch.equal(lse, l_ref)
        # and within the library's tolerance of the CPU oracle
        o_orc, l_orc = oracle.decode(qc, kc, vc, lens, cfg.scale)
        assert_close_to_oracle(o[:, 0], lse, o_orc, l_orc, what="fa_decode_noalloc")
