"""fa_decode_noalloc: the decode entry point for callers that cannot allocate device memory
(code living inside someone else's memory pool, a serving loop that must never hit the
allocator, a plugin that only receives buffers).  Its partial results go to a fixed array inside
the library instead of a caller workspace, so the test checks two things: the results equal
those of fa_decode, and a second call right after the first (different lengths, so different
slots of the shared array are live) is just as correct, i.e. nothing depends on what the
previous call left behind.  The file name keeps this test last in collection order."""
import pytest
import torch

from paper_2410_16663_b200 import inputs as synth
from tests.util import TOL_O, TOL_LSE


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


@pytest.mark.gpu
def test_noalloc_matches_fa_decode_on_two_calls_in_a_row(fa):
    dev = "cuda"
    cfg = synth.DecodeConfig("noalloc", 6, 8, 2, 5000, 1, 5000, seed=808)
    q, k, v, sl = synth.decode_inputs(cfg, dev, poison=False)  # the second call reads other lengths
    assert fa.fa_decode_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Smax, cfg.d) <= fa.FA_DECODE_NOALLOC_BYTES
    ws = torch.empty(fa.fa_decode_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Smax, cfg.d), dtype=torch.uint8,
                     device=dev)
    lens_a = sl.clone()
    lens_b = torch.tensor([5000, 1, 0, 2049, 300, 4097], dtype=torch.int32)
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
        assert torch.isfinite(o.float()).all()
        assert float((o.float() - o_ref.float()).abs().max()) <= TOL_O
        same_inf = torch.isneginf(lse) & torch.isneginf(l_ref)
        dl = torch.where(same_inf, torch.zeros_like(lse), (lse - l_ref).abs())
        assert not torch.isnan(dl).any() and float(dl.max()) <= TOL_LSE
