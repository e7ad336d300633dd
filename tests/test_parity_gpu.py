"""Parity of the CUDA library against the CPU oracle, through the C ABI, on seeded inputs.

Small and medium problems are compared element by element against the full oracle; the
benchmark-size configurations are compared on sampled rows the oracle computes one by one.
Tolerances: max|dO| <= 2e-3 and max|dLSE| <= 1e-3 (fp16/bf16 inputs, fp32 accumulation).
With bf16 inputs two format roundings are allowed on top, each bounded exactly from the oracle
(see tests/util.py): 2^-9 * sum_j P_ij |V_j| for the bf16 probabilities fed to the second MMA,
and 2^-8 |O| for a stored bf16 output; the fp32-output mode is gated without the latter."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2410_16663_b200 import inputs as synth
from tests.util import (TOL_O, TOL_LSE, assert_close_to_oracle, guard_alloc, oracle_rows_for, rel_l2_rows)

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def fa():
    from paper_2410_16663_b200 import binding
    return binding


def check_status(fa):
    rc, where, blk = fa.fa_device_status()
    assert rc == 0, f"device status {rc} at {where} block {blk}"


def run_forward(fa, q, k, v, causal, scale, o_dtype=None, variant=0):
    B, Sq, Hq, d = q.shape
    o, chk_o = guard_alloc((B, Sq, Hq, d), o_dtype or q.dtype, DEV)
    lse, chk_l = guard_alloc((B, Hq, Sq), torch.float32, DEV)
    fa.fa_forward_ex(q, k, v, o, lse, causal, scale, variant=variant)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o()
    chk_l()
    return o, lse


def full_case(fa, B, Hq, Hkv, Sq, Skv, causal, dtype, seed, variant=0, scale=None, fp16_ulp=False):
    cfg = synth.PrefillConfig("t", B, Hq, Hkv, Sq, Skv, dtype=dtype, causal=causal, seed=seed)
    q, k, v = synth.prefill_inputs(cfg, "cpu")
    scale = cfg.scale if scale is None else scale
    o_ref, l_ref = oracle.attention_full(q, k, v, causal, scale)
    absv = oracle.attention_full(q, k, v.abs(), causal, scale)[0] if dtype == "bf16" else None
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    what = f"B{B} Hq{Hq} Hkv{Hkv} Sq{Sq} Skv{Skv} causal{int(causal)} {dtype} variant{variant}"
    o, lse = run_forward(fa, qd, kd, vd, causal, scale, variant=variant)
    assert_close_to_oracle(o, lse, o_ref, l_ref, stored_bf16=(dtype == "bf16"), p_absv=absv, what=what,
                           stored_fp16_ulp=fp16_ulp)
    if dtype == "bf16":  # gate on the accumulator, without the rounding of the stored output
        o32, lse32 = run_forward(fa, qd, kd, vd, causal, scale, o_dtype=torch.float32, variant=variant)
        assert_close_to_oracle(o32, lse32, o_ref, l_ref, p_absv=absv, what=what + " fp32-out")
    return o, lse


# ------------------------------------------------------------------ C1: the small benchmark config
@pytest.mark.parametrize("variant", [0, 1, 2, 3, 4])
def test_c1_full_tensor(fa, variant):
    c = synth.C1
    q, k, v = synth.prefill_inputs(c, "cpu")
    o_ref, l_ref = oracle.attention_full(q, k, v, c.causal, c.scale)
    o, lse = run_forward(fa, q.to(DEV), k.to(DEV), v.to(DEV), c.causal, c.scale, variant=variant)
    assert_close_to_oracle(o, lse, o_ref, l_ref, what="C1")
    assert rel_l2_rows(o, o_ref) < 3e-3


def test_c1_plain_entry_points_and_determinism(fa):
    c = synth.C1
    q, k, v = (t.to(DEV) for t in synth.prefill_inputs(c, "cpu"))
    outs = []
    for _ in range(2):
        o = torch.empty_like(q)
        lse = torch.empty(c.B, c.Hq, c.Sq, dtype=torch.float32, device=DEV)
        fa.fa_forward(q, k, v, o, lse, c.causal, c.scale)
        torch.cuda.synchronize()
        outs.append((o, lse))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    o_ex, lse_ex = run_forward(fa, q, k, v, c.causal, c.scale)
    assert torch.equal(outs[0][0], o_ex) and torch.equal(outs[0][1], lse_ex)
    # lse may be NULL
    o2 = torch.empty_like(q)
    fa.fa_forward(q, k, v, o2, None, c.causal, c.scale)
    torch.cuda.synchronize()
    assert torch.equal(o2, outs[0][0])
    check_status(fa)


# ------------------------------------------------------------------ shape grid, full oracle
GRID = [  # (Sq, Skv)
    (1, 1), (2, 2), (17, 17), (127, 127), (128, 128), (129, 129), (255, 255), (256, 256), (257, 257),
    (384, 384), (1000, 1000), (1, 129), (17, 1000), (128, 384), (100, 257), (257, 1000),
]


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("sq,skv", GRID)
def test_shape_grid_fp16(fa, sq, skv, causal):
    full_case(fa, 1, 2, 2, sq, skv, causal, "fp16", seed=sq * 1000 + skv)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("sq,skv", [(1, 1), (129, 129), (257, 1000), (384, 384), (1000, 1000)])
def test_shape_grid_bf16(fa, sq, skv, causal):
    full_case(fa, 1, 2, 1, sq, skv, causal, "bf16", seed=sq * 1000 + skv + 1)


@pytest.mark.parametrize("hq,hkv", [(1, 1), (4, 1), (8, 2), (8, 8), (6, 3)])
def test_head_grouping(fa, hq, hkv):
    full_case(fa, 2, hq, hkv, 200, 333, True, "fp16", seed=hq * 10 + hkv)


@pytest.mark.parametrize("variant", [1, 2, 3])
def test_alternate_kernels_on_ragged_shapes(fa, variant):
    full_case(fa, 2, 4, 2, 257, 1000, True, "fp16", seed=77, variant=variant)
    full_case(fa, 1, 2, 2, 129, 385, False, "bf16", seed=78, variant=variant)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("sq,skv", [(1, 1), (127, 127), (128, 128), (129, 129), (256, 256), (257, 257), (1000, 1000),
                                    (1, 129), (17, 1000), (128, 384), (100, 257), (257, 1000)])
def test_pingpong_kernel_shape_grid(fa, sq, skv, causal):
    full_case(fa, 1, 2, 2, sq, skv, causal, "fp16", seed=sq * 1000 + skv + 7, variant=3)


@pytest.mark.parametrize("causal", [False, True])
def test_default_choice_of_kernel_from_4096_keys_on(fa, causal):
    # fa_forward's own choice (the ping-pong kernel once Skv >= 1024) on a shape the full oracle
    # finishes quickly: few query rows over many keys, rows ending inside a tile, a ragged key tail,
    # bottom-right aligned mask
    full_case(fa, 1, 4, 2, 130, 4200, causal, "fp16", seed=401)
    full_case(fa, 1, 2, 2, 300, 4096, causal, "bf16", seed=402)


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        g = int(rng.choice([1, 1, 2, 4, 8]))
        hkv = int(rng.integers(1, 5))
        B = int(rng.integers(1, 4))
        skv = int(rng.choice([int(rng.integers(1, 400)), int(rng.integers(400, 1400)), int(rng.integers(2048, 2700))]))
        causal = bool(rng.integers(0, 2))
        sq = int(rng.integers(1, skv + 1)) if causal else int(rng.integers(1, 700))
        sq = min(sq, 900)
        if B * hkv * g * sq * skv > 30_000_000:
            continue
        out.append((B, hkv * g, hkv, sq, skv, causal, "fp16" if rng.integers(0, 2) else "bf16"))
    return out


@pytest.mark.parametrize("variant", [3, 4])
def test_random_shapes_both_persistent_kernels(fa, variant):
    # thirty seeded random problems (batch, head grouping, ragged lengths, masks, both 16-bit
    # types) through each persistent kernel, every output element against the oracle
    for i, (B, hq, hkv, sq, skv, causal, dt) in enumerate(_random_shapes(30, seed=2024)):
        full_case(fa, B, hq, hkv, sq, skv, causal, dt, seed=9000 + i, variant=variant)


def test_pingpong_kernel_item_order_in_tile_classes(fa):
    # shapes whose K/V per head are large enough for the launcher to order the items in classes of
    # query tiles: 17 tiles per head (classes of 8, 8 and 1), 33 tiles (16, 16, 1), and without a
    # mask 6 tiles (classes of 4 and 2); every output row must be written exactly once
    full_case(fa, 1, 8, 8, 2100, 2100, True, "fp16", seed=411)
    full_case(fa, 1, 4, 2, 4130, 4130, True, "fp16", seed=412)
    full_case(fa, 2, 16, 16, 700, 2100, False, "fp16", seed=413)


def test_pingpong_kernel_many_items_per_cta(fa):
    # more query tiles than CTAs, of one to five kv steps each: every CTA strings several items
    # together, odd and even step counts, through both warpgroups
    full_case(fa, 2, 160, 8, 640, 640, True, "bf16", seed=91, variant=3)
    full_case(fa, 3, 64, 64, 300, 300, True, "fp16", seed=92, variant=3)
    full_case(fa, 2, 100, 20, 129, 700, False, "fp16", seed=93, variant=3)


def test_pingpong_kernel_peaked_rows_rescale(fa):
    # keys whose norm grows along the sequence: the running max keeps moving, O is rescaled often
    torch.manual_seed(5)
    B, H, S = 1, 2, 1024
    q = torch.randn(B, S, H, 128).half()
    k = (torch.randn(B, S, H, 128) * torch.linspace(0.2, 6.0, S).view(1, S, 1, 1)).half()
    v = torch.randn(B, S, H, 128).half()
    for causal in (False, True):
        o_ref, l_ref = oracle.attention_full(q, k, v, causal, 1.0)
        o, lse = run_forward(fa, q.to(DEV), k.to(DEV), v.to(DEV), causal, 1.0, variant=3)
        assert_close_to_oracle(o, lse, o_ref, l_ref, what=f"peaked causal={causal}", stored_fp16_ulp=True)


def test_scale_zero_and_large_scale(fa):
    full_case(fa, 1, 2, 2, 130, 260, True, "fp16", seed=5, scale=0.0)
    full_case(fa, 1, 2, 2, 130, 260, False, "fp16", seed=6, scale=1.0, fp16_ulp=True)  # peaked softmax


@pytest.mark.parametrize("variant", [0, 3, 4])
def test_bhsd_strided_layout(fa, variant):
    # (the ping-pong kernel writes its 16-bit output through a tensor map built from these strides)
    cfg = synth.PrefillConfig("t", 2, 4, 2, 300, 300, dtype="fp16", causal=True, seed=9)
    q, k, v = synth.prefill_inputs(cfg, "cpu")
    o_ref, l_ref = oracle.attention_full(q, k, v, True, cfg.scale)
    # store as [B,H,S,d] and pass [B,S,H,d] views
    qd = q.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
    kd = k.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
    vd = v.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
    o = torch.empty(2, 4, 300, 128, dtype=torch.float16, device=DEV).permute(0, 2, 1, 3)
    lse = torch.empty(2, 4, 300, dtype=torch.float32, device=DEV)
    fa.fa_forward_ex(qd, kd, vd, o, lse, True, cfg.scale, variant=variant)
    torch.cuda.synchronize()
    check_status(fa)
    assert_close_to_oracle(o, lse, o_ref, l_ref, what="BHSD views")


@pytest.mark.parametrize("variant", [0, 3, 4])
def test_output_aligned_to_16_but_not_32_bytes(fa, variant):
    # rows that start on a 16-byte but not a 32-byte boundary take the 128-bit store path of the
    # paired-tile kernel; the ping-pong kernel's TMA stores need 16 bytes only.  Nothing may be
    # written outside the output: its last query tile has 4 live rows of 128.
    cfg = synth.PrefillConfig("t", 1, 2, 2, 260, 260, dtype="fp16", causal=True, seed=12)
    q, k, v = synth.prefill_inputs(cfg, "cpu")
    o_ref, l_ref = oracle.attention_full(q, k, v, True, cfg.scale)
    n = q.numel()
    buf = torch.full((n + 64,), float("nan"), dtype=torch.float16, device=DEV)
    base = (-buf.data_ptr() // 2) % 16          # elements up to the next 32-byte boundary
    o = buf[base + 8: base + 8 + n].view(1, 260, 2, 128)
    assert o.data_ptr() % 32 == 16
    lse = torch.empty(1, 2, 260, dtype=torch.float32, device=DEV)
    fa.fa_forward_ex(q.to(DEV), k.to(DEV), v.to(DEV), o, lse, True, cfg.scale, variant=variant)
    torch.cuda.synchronize()
    check_status(fa)
    assert_close_to_oracle(o, lse, o_ref, l_ref, what="16-byte aligned output")
    assert torch.isnan(buf[:base + 8]).all() and torch.isnan(buf[base + 8 + n:]).all()


def test_degenerate_sizes(fa):
    q = torch.randn(2, 5, 2, 128, device=DEV).half()
    kv0 = torch.empty(2, 0, 2, 128, dtype=torch.float16, device=DEV)
    o, lse = run_forward(fa, q, kv0, kv0, False, 0.1)       # no keys: O = 0, LSE = -inf
    assert float(o.abs().max()) == 0.0 and torch.isneginf(lse).all()
    # B = 0 and Sq = 0 are no-ops that must not touch the outputs
    o = torch.full((2, 5, 2, 128), 7.0, dtype=torch.float16, device=DEV)
    k = torch.randn(2, 9, 2, 128, device=DEV).half()
    assert fa.lib.fa_forward(q.data_ptr(), k.data_ptr(), k.data_ptr(), o.data_ptr(), None, 0, 2, 2, 5, 9, 128,
                             0, 0.1, None) == 0
    assert fa.lib.fa_forward(q.data_ptr(), k.data_ptr(), k.data_ptr(), o.data_ptr(), None, 2, 2, 2, 0, 9, 128,
                             0, 0.1, None) == 0
    torch.cuda.synchronize()
    assert float((o - 7.0).abs().max()) == 0.0
    check_status(fa)


def test_closed_form_identical_keys_on_gpu(fa):
    # all keys equal: O is the running mean of V, LSE = scale*q.k + ln(n)
    B, H, S = 1, 2, 300
    g = torch.Generator().manual_seed(3)
    q = torch.randn(B, S, H, 128, generator=g).half()
    v = torch.randn(B, S, H, 128, generator=g).half()
    k = torch.randn(B, 1, H, 128, generator=g).half().expand(B, S, H, 128).contiguous()
    o, lse = run_forward(fa, q.to(DEV), k.to(DEV), v.to(DEV), True, 0.05)
    want = v.double().cumsum(dim=1) / torch.arange(1, S + 1, dtype=torch.float64).view(1, S, 1, 1)
    assert float((o.double().cpu() - want).abs().max()) <= TOL_O
    s = 0.05 * (q.double() * k.double()).sum(-1).permute(0, 2, 1)
    want_l = s + torch.log(torch.arange(1, S + 1, dtype=torch.float64)).view(1, 1, S)
    assert float((lse.double().cpu() - want_l).abs().max()) <= TOL_LSE


# ------------------------------------------------------------------ benchmark-size configs, sampled rows
def sampled_case(fa, cfg, n_random, pairs=None, cross_check=False):
    q, k, v = synth.prefill_inputs(cfg, DEV)
    # outputs start as NaN inside NaN guard bands: an element no work item wrote stays NaN
    o, chk_o = guard_alloc(tuple(q.shape), q.dtype, DEV)
    lse, chk_l = guard_alloc((cfg.B, cfg.Hq, cfg.Sq), torch.float32, DEV)
    fa.fa_forward(q, k, v, o, lse, cfg.causal, cfg.scale)    # the launch configuration bench.py times
    torch.cuda.synchronize()
    check_status(fa)
    chk_o()
    chk_l()
    assert not torch.isnan(o).any() and not torch.isnan(lse).any(), f"{cfg.name}: an output element was never written"
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    rows = synth.sample_rows(cfg, n_random, seed=cfg.seed + 99, pairs=pairs)
    bf16 = cfg.dtype == "bf16"
    res = oracle_rows_for(q, k, v, rows, cfg.causal, cfg.scale, with_absv=bf16)
    o_ref, l_ref, absv = res if bf16 else (res[0], res[1], None)
    idx = torch.tensor(rows, device=DEV)
    o_s = o[idx[:, 0], idx[:, 2], idx[:, 1]]
    l_s = lse[idx[:, 0], idx[:, 1], idx[:, 2]]
    assert_close_to_oracle(o_s, l_s, o_ref, l_ref, stored_bf16=bf16, p_absv=absv, what=cfg.name)
    if bf16:
        # gate on the accumulator through the fp32-output mode
        o32 = torch.full((cfg.B, cfg.Sq, cfg.Hq, cfg.d), float("nan"), dtype=torch.float32, device=DEV)
        lse32 = torch.full_like(lse, float("nan"))
        fa.fa_forward_ex(q, k, v, o32, lse32, cfg.causal, cfg.scale)
        torch.cuda.synchronize()
        check_status(fa)
        assert not torch.isnan(o32).any() and not torch.isnan(lse32).any()
        assert_close_to_oracle(o32[idx[:, 0], idx[:, 2], idx[:, 1]], lse32[idx[:, 0], idx[:, 1], idx[:, 2]],
                               o_ref, l_ref, p_absv=absv, what=cfg.name + " fp32-out")
    if cross_check:
        whole_tensor_cross_check(fa, cfg, q, k, v, o, lse)
    return len(rows)


def whole_tensor_cross_check(fa, cfg, q, k, v, o, lse):
    """Every element of the default kernel's O and LSE against a second, much simpler kernel.

    The oracle can only afford sampled rows at these sizes; the simple kernel (one CTA per query
    tile, every stage sequential, P through shared memory) is itself compared with the oracle at
    every element on the small shapes above, so agreement with it over the whole tensor covers the
    rows the sample missed.  Both kernels accumulate in fp32 and differ only in summation order and
    in the reference the exponentials are taken against, so the fp32 outputs are compared at the
    oracle tolerances and the stored 16-bit outputs with one rounding step of the format on top."""
    o2 = torch.full((cfg.B, cfg.Sq, cfg.Hq, cfg.d), float("nan"), dtype=torch.float32, device=DEV)
    l2 = torch.full_like(lse, float("nan"))
    fa.fa_forward_ex(q, k, v, o2, l2, cfg.causal, cfg.scale, variant=2)
    torch.cuda.synchronize()
    check_status(fa)
    assert not torch.isnan(o2).any() and not torch.isnan(l2).any()
    ulp = 2.0 ** -8 if cfg.dtype == "bf16" else 2.0 ** -11
    worst_o, worst_l = 0.0, 0.0
    for b in range(cfg.B):                     # batch by batch: bounds the temporaries
        diff = (o[b].float() - o2[b]).abs() - ulp * o2[b].abs()
        worst_o = max(worst_o, float(diff.max()))
        worst_l = max(worst_l, float((lse[b] - l2[b]).abs().max()))
    assert worst_o <= TOL_O, f"{cfg.name}: whole-tensor max(|dO| - one rounding step) = {worst_o:.3e}"
    assert worst_l <= TOL_LSE, f"{cfg.name}: whole-tensor max|dLSE| = {worst_l:.3e}"


def test_c2_llama7b_prefill_sampled(fa):
    assert sampled_case(fa, synth.C2, 80, cross_check=True) >= 256


@pytest.mark.parametrize("s", [8192, 32768])
def test_c3_long_context_sampled(fa, s):
    assert sampled_case(fa, synth.C3[s], 80, cross_check=(s == 8192)) >= 256


@pytest.mark.parametrize("s", [131072, 262144])
def test_c3_very_long_context_sampled(fa, s):
    cfg = synth.C3[s]
    assert sampled_case(fa, cfg, 20, pairs=[(0, 0), (0, 13), (0, 31)]) >= 64


@pytest.mark.parametrize("causal", [True, False])
def test_long_context_item_order_with_whole_rounds_per_head(fa, causal):
    # from about 56K keys on (148 SMs) the ping-pong kernel goes head by head and gives every head
    # a whole number of rounds of the grid, the last one partly empty: 469 query tiles are three
    # full rounds and one of 25 items, walked in opposite directions for odd and even heads.  A
    # ragged last tile, GQA, every output element written exactly once (NaN pre-fill), sampled
    # rows of every head against the oracle.
    cfg = synth.PrefillConfig("order-60K", 1, 4, 2, 60000, 60000, dtype="bf16", causal=causal,
                              seed=1050 + int(causal))
    assert sampled_case(fa, cfg, 12, pairs=[(0, 0), (0, 1), (0, 2), (0, 3)]) >= 64


def test_c4_gqa_sampled(fa):
    assert sampled_case(fa, synth.C4, 64, cross_check=True) >= 256
    assert sampled_case(fa, synth.C4_NC, 64, cross_check=True) >= 256


# ------------------------------------------------------------------ head dimension 64
def full_case_d64(fa, B, Hq, Hkv, Sq, Skv, causal, dtype, seed, variant=0):
    cfg = synth.PrefillConfig("t", B, Hq, Hkv, Sq, Skv, d=64, dtype=dtype, causal=causal, seed=seed)
    q, k, v = synth.prefill_inputs(cfg, "cpu")
    o_ref, l_ref = oracle.attention_full(q, k, v, causal, cfg.scale)
    absv = oracle.attention_full(q, k, v.abs(), causal, cfg.scale)[0] if dtype == "bf16" else None
    what = f"d64 B{B} Hq{Hq} Hkv{Hkv} Sq{Sq} Skv{Skv} causal{int(causal)} {dtype} variant{variant}"
    o, lse = run_forward(fa, q.to(DEV), k.to(DEV), v.to(DEV), causal, cfg.scale, variant=variant)
    assert_close_to_oracle(o, lse, o_ref, l_ref, stored_bf16=(dtype == "bf16"), p_absv=absv, what=what)
    if dtype == "bf16":
        o32, lse32 = run_forward(fa, q.to(DEV), k.to(DEV), v.to(DEV), causal, cfg.scale, o_dtype=torch.float32,
                                 variant=variant)
        assert_close_to_oracle(o32, lse32, o_ref, l_ref, p_absv=absv, what=what + " fp32-out")


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("sq,skv", [(1, 1), (127, 127), (128, 128), (129, 129), (197, 197), (256, 256), (257, 257),
                                    (1, 129), (17, 1000), (100, 257), (300, 700)])
def test_d64_shape_grid(fa, sq, skv, causal):
    full_case_d64(fa, 2, 3, 3, sq, skv, causal, "fp16", seed=sq * 1000 + skv + 11)


def test_d64_short_sequence_kernel(fa):
    # 128 < Skv <= 256: all keys as one tile, a persistent pipeline over (batch, head, two query
    # tiles).  More items than CTAs, with one or two query tiles each, many query tiles over few
    # keys, causal with fewer queries than keys
    full_case_d64(fa, 30, 12, 12, 197, 197, False, "fp16", seed=81)
    full_case_d64(fa, 40, 6, 2, 100, 130, False, "bf16", seed=82)
    full_case_d64(fa, 3, 4, 4, 700, 256, False, "fp16", seed=83)
    full_case_d64(fa, 5, 8, 8, 150, 255, True, "fp16", seed=84)
    full_case_d64(fa, 2, 2, 1, 256, 256, True, "bf16", seed=85)
    # an odd number of query tiles: the last item of a head has one tile, and the tiles change pairs
    full_case_d64(fa, 7, 9, 3, 300, 200, False, "fp16", seed=86)
    full_case_d64(fa, 50, 4, 4, 190, 197, True, "fp16", seed=87)
    full_case_d64(fa, 9, 4, 4, 640, 197, False, "fp16", seed=88)


@pytest.mark.parametrize("skv", [129, 144, 145, 160, 176, 193, 208, 209, 224, 240, 241])
def test_d64_short_sequence_every_split_of_the_keys(fa, skv):
    # the keys go to the two halves of a row in chunks of 16: every count of chunks from 9 to 16,
    # with and without a ragged last chunk; enough items for every CTA to take several
    full_case_d64(fa, 13, 12, 4, 197, skv, False, "fp16", seed=900 + skv)
    full_case_d64(fa, 2, 3, 3, skv, skv, True, "bf16", seed=700 + skv)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_d64_gqa_and_both_types(fa, dtype):
    full_case_d64(fa, 2, 8, 2, 333, 333, True, dtype, seed=71)
    full_case_d64(fa, 1, 12, 12, 197, 197, False, dtype, seed=72)       # the vision shape, one image
    full_case_d64(fa, 1, 4, 1, 130, 1500, False, dtype, seed=73)        # many kv tiles through the two-slot ring


def test_d64_vision_batch_full_size_sampled(fa):
    # the benchmark's batch of 1024 images: sampled rows against the oracle, everything finite
    cfg = synth.DEIT_B
    q, k, v = synth.prefill_inputs(cfg, DEV)
    o, lse = run_forward(fa, q, k, v, cfg.causal, cfg.scale)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    rows = synth.sample_rows(cfg, 6, seed=5, pairs=[(0, 0), (0, 11), (511, 5), (1023, 0), (1023, 11)])
    o_ref, l_ref = oracle_rows_for(q, k, v, rows, cfg.causal, cfg.scale)
    idx = torch.tensor(rows)
    o_s = o[idx[:, 0], idx[:, 2], idx[:, 1]].view(1, len(rows), 1, cfg.d)
    l_s = lse[idx[:, 0], idx[:, 1], idx[:, 2]].view(1, 1, len(rows))
    assert_close_to_oracle(o_s, l_s, o_ref.view(1, len(rows), 1, cfg.d), l_ref.view(1, 1, len(rows)), what="DeiT-B batch")


def test_d64_is_refused_where_it_is_not_built(fa):
    # of the forced kernel variants only the ping-pong kernel (3) exists for d = 64
    q = torch.zeros(1, 4, 2, 64, dtype=torch.float16, device=DEV)
    o = torch.empty_like(q); lse = torch.empty(1, 2, 4, device=DEV)
    for variant in (1, 2, 4):
        assert fa.fa_forward_ex(q, q, q, o, lse, False, 0.1, variant=variant, raise_on_error=False) == fa.FA_ERR_UNSUPPORTED
    assert fa.fa_forward_ex(q, q, q, o, lse, False, 0.1, variant=3) == fa.FA_OK


@pytest.mark.parametrize("causal", [False, True])
def test_d64_pingpong_kernel_shape_grid(fa, causal):
    # From 512 keys on d = 64 takes the ping-pong kernel (tiles of one 64-element box, O in 64
    # columns of tensor memory).  Its small-item paths are reached by forcing it on short shapes;
    # ragged tiles on both sides, chunked prefill (Sq < Skv), GQA, more items than CTAs.
    for (B, hq, hkv, sq, skv) in [(1, 1, 1, 1, 1), (2, 3, 3, 128, 128), (2, 2, 1, 129, 300), (1, 2, 2, 77, 1500)]:
        full_case_d64(fa, B, hq, hkv, sq, skv, causal, "fp16", seed=sq * 7 + skv, variant=3)
    for (B, hq, hkv, sq, skv) in [(2, 3, 3, 512, 512), (1, 4, 2, 1100, 1100), (3, 5, 5, 513, 2049), (40, 4, 4, 600, 600)]:
        full_case_d64(fa, B, hq, hkv, sq, skv, causal, "fp16", seed=sq * 3 + skv)
    full_case_d64(fa, 1, 4, 1, 2300, 2300, causal, "bf16", seed=97)          # bf16, and its fp32-output mode


def test_d64_long_sequences_full_size_sampled(fa):
    # 8 x 32 heads x 4096 and 2 x 32 x 8192 causal: every element written, sampled rows against the oracle
    for (B, S, seed) in ((8, 4096, 1071), (2, 8192, 1072)):
        cfg = synth.PrefillConfig(f"d64-{S}", B, 32, 32, S, S, d=64, dtype="fp16", causal=True, seed=seed)
        assert sampled_case(fa, cfg, 16, pairs=[(0, 0), (0, 31), (B - 1, 17)]) >= 48


# ------------------------------------------------------------------ head dimension 256
def full_case_d256(fa, B, Hq, Hkv, Sq, Skv, causal, dtype, seed):
    cfg = synth.PrefillConfig("t", B, Hq, Hkv, Sq, Skv, d=256, dtype=dtype, causal=causal, seed=seed)
    q, k, v = synth.prefill_inputs(cfg, "cpu")
    o_ref, l_ref = oracle.attention_full(q, k, v, causal, cfg.scale)
    absv = oracle.attention_full(q, k, v.abs(), causal, cfg.scale)[0] if dtype == "bf16" else None
    what = f"d256 B{B} Hq{Hq} Hkv{Hkv} Sq{Sq} Skv{Skv} causal{int(causal)} {dtype}"
    o, lse = run_forward(fa, q.to(DEV), k.to(DEV), v.to(DEV), causal, cfg.scale)
    assert_close_to_oracle(o, lse, o_ref, l_ref, stored_bf16=(dtype == "bf16"), p_absv=absv, what=what)
    if dtype == "bf16":
        o32, lse32 = run_forward(fa, q.to(DEV), k.to(DEV), v.to(DEV), causal, cfg.scale, o_dtype=torch.float32)
        assert_close_to_oracle(o32, lse32, o_ref, l_ref, p_absv=absv, what=what + " fp32-out")


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("sq,skv", [(1, 1), (127, 127), (128, 128), (129, 129), (300, 300), (1, 129), (17, 1000),
                                    (100, 257), (300, 700)])
def test_d256_shape_grid(fa, sq, skv, causal):
    full_case_d256(fa, 2, 3, 3, sq, skv, causal, "fp16", seed=sq * 1000 + skv + 13)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_d256_gqa_both_types_and_more_ctas_than_sms(fa, dtype):
    full_case_d256(fa, 2, 8, 2, 333, 333, True, dtype, seed=91)
    full_case_d256(fa, 1, 4, 1, 130, 1500, False, dtype, seed=92)     # many kv tiles through the single slots
    full_case_d256(fa, 6, 16, 4, 500, 500, True, dtype, seed=93)      # 384 CTAs on 148 SMs


def test_d256_bench_size_sampled(fa):
    # the benchmark's d = 256 case (2 x 16 heads x 8192, causal): sampled rows against the oracle, everything finite
    cfg = synth.PrefillConfig("d256-8K", 2, 16, 16, 8192, 8192, d=256, dtype="fp16", causal=True, seed=1040)
    q, k, v = synth.prefill_inputs(cfg, DEV)
    o, lse = run_forward(fa, q, k, v, cfg.causal, cfg.scale)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    rows = synth.sample_rows(cfg, 5, seed=6, pairs=[(0, 0), (0, 15), (1, 7), (1, 15)])
    rows += [(0, 3, 0), (1, 3, 8191), (0, 9, 127), (1, 9, 128), (0, 12, 4095)]   # first, last, tile edges
    o_ref, l_ref = oracle_rows_for(q, k, v, rows, cfg.causal, cfg.scale)
    idx = torch.tensor(rows)
    o_s = o[idx[:, 0], idx[:, 2], idx[:, 1]].view(1, len(rows), 1, cfg.d)
    l_s = lse[idx[:, 0], idx[:, 1], idx[:, 2]].view(1, 1, len(rows))
    assert_close_to_oracle(o_s, l_s, o_ref.view(1, len(rows), 1, cfg.d), l_ref.view(1, 1, len(rows)), what="d256 8K")


def test_d256_is_refused_where_it_is_not_built(fa):
    q = torch.zeros(1, 4, 2, 256, dtype=torch.float16, device=DEV)
    o = torch.empty_like(q); lse = torch.empty(1, 2, 4, device=DEV)
    assert fa.fa_forward_ex(q, q, q, o, lse, False, 0.1, variant=1, raise_on_error=False) == fa.FA_ERR_UNSUPPORTED


# ------------------------------------------------------------------ 8-bit operands in prefill
FP8_SCALES = (0.125, 0.25, 0.0625)      # factors of q, k, v


def fp8_allowance(q8, k8, v8, rows, causal, scale, stored_bf16):
    """What rounding the probabilities to FP8 e4m3 may cost, per output element of the given rows
    (b, h, i), from oracle-side quantities only.  The kernel rounds F * 2^(x_ij - m_ref), with F = 2^4
    and the reference m_ref at most 2^4 behind the running row max, to e4m3: a relative rounding of
    at most 2^-4 for values in the normal range and an absolute one of at most 2^-10 below it.
    Carried through O_i = sum_j P_ij V_j / l_i that is at most
        2^-4 * sum_j P_ij |V_j|  +  2^-14 * sum_j |V_j| / L_i ,   L_i = sum_j exp(s_ij - max_j s_ij)
    (visible j only).  The first term comes from the oracle run on |V|; the row max for the second
    is taken from the scores of the row, computed here in float64."""
    qs, ks, vs = FP8_SCALES
    o_abs, _ = oracle.attention_fp8(q8, k8, v8, causal, scale, qs, ks, vs, rows=rows, abs_v=True)
    g = q8.shape[2] // k8.shape[2]
    Sq, Skv = q8.shape[1], k8.shape[1]
    out = torch.zeros_like(o_abs)
    for n, (b, h, i) in enumerate(rows):
        qf = oracle.e4m3_to_float64(q8[b, i, h]) * qs
        kf = oracle.e4m3_to_float64(k8[b, :, h // g]) * ks
        vf = (oracle.e4m3_to_float64(v8[b, :, h // g]) * vs).abs()
        nvis = min(Skv, i + (Skv - Sq) + 1) if causal else Skv
        sc = (kf[:nvis] @ qf) * scale
        L = torch.exp(sc - sc.max()).sum()
        out[n] = 2.0 ** -4 * o_abs[n] + 2.0 ** -14 * vf[:nvis].sum(0) / L
    return out


def fp8_case(fa, B, Hq, Hkv, Sq, Skv, causal, o_dtype, seed, rows=None):
    cfg = synth.PrefillConfig("fp8", B, Hq, Hkv, Sq, Skv, dtype="fp16", causal=causal, seed=seed)
    dev = DEV if rows is not None else "cpu"
    q, k, v = synth.prefill_inputs(cfg, dev)
    qs, ks, vs = FP8_SCALES
    q8, k8, v8 = synth.fp8_operands(q, k, v, qs, ks, vs)
    qd, kd, vd = q8.to(DEV), k8.to(DEV), v8.to(DEV)
    o, chk_o = guard_alloc((B, Sq, Hq, 128), o_dtype, DEV)
    lse, chk_l = guard_alloc((B, Hq, Sq), torch.float32, DEV)
    fa.fa_forward_fp8(qd, kd, vd, o, lse, causal, cfg.scale, qs, ks, vs)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o(); chk_l()
    assert not torch.isnan(o).any() and not torch.isnan(lse).any()
    q8c, k8c, v8c = q8.cpu(), k8.cpu(), v8.cpu()
    if rows is None:
        rows = [(b, h, i) for b in range(B) for h in range(Hq) for i in range(Sq)]
    o_ref, l_ref = oracle.attention_fp8(q8c, k8c, v8c, causal, cfg.scale, qs, ks, vs, rows=rows)
    allow = fp8_allowance(q8c, k8c, v8c, rows, causal, cfg.scale, o_dtype == torch.bfloat16)
    idx = torch.tensor(rows, device=DEV)
    o_s = o[idx[:, 0], idx[:, 2], idx[:, 1]].double().cpu()
    l_s = lse[idx[:, 0], idx[:, 1], idx[:, 2]].double().cpu()
    if o_dtype == torch.bfloat16:
        allow = allow + 2.0 ** -8 * o_ref.abs()
    diff = (o_s - o_ref).abs()
    what = f"fp8 B{B} Hq{Hq} Hkv{Hkv} Sq{Sq} Skv{Skv} causal{int(causal)} {o_dtype}"
    assert float((diff - allow).max()) <= TOL_O, f"{what}: max(|dO| - allowance) = {float((diff - allow).max()):.3e}"
    assert float((l_s - l_ref).abs().max()) <= TOL_LSE, f"{what}: max|dLSE| = {float((l_s - l_ref).abs().max()):.3e}"
    return float(diff.max()), float(allow.max())


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("sq,skv", [(1, 1), (127, 127), (128, 128), (129, 129), (300, 300), (1, 129), (17, 1000), (100, 257),
                                    (257, 1000), (130, 2200)])
def test_fp8_prefill_shape_grid(fa, sq, skv, causal):
    fp8_case(fa, 2, 2, 1, sq, skv, causal, torch.float16, seed=sq * 1000 + skv + 21)


def test_fp8_prefill_gqa_many_items_and_bf16_output(fa):
    fp8_case(fa, 2, 8, 2, 333, 333, True, torch.bfloat16, seed=95)
    fp8_case(fa, 3, 64, 64, 300, 300, True, torch.float16, seed=96)        # several items per CTA
    fp8_case(fa, 1, 4, 4, 700, 1300, False, torch.bfloat16, seed=97)


def test_fp8_prefill_bench_sizes_sampled(fa):
    # C2's shape and the 8K long-context shape with 8-bit operands, sampled rows against the oracle
    for cfg in (synth.C2, synth.C3[8192]):
        rows = synth.sample_rows(cfg, 30, seed=cfg.seed + 7)
        worst, allow = fp8_case(fa, cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Skv, True, torch.float16, seed=cfg.seed + 50, rows=rows)
        print(f"fp8 {cfg.name}: max|dO| {worst:.2e} (largest allowance {allow:.2e})")


# ------------------------------------------------------------------ attention + output projection
def proj_allowance(o_ref, out_ref, w, ulp):
    """Sound bound on |d out| from the attention gate: every element of the 16-bit O the projection
    reads is within TOL_O + 2 ulp |O| of the oracle's rounded O (the gate plus the two roundings),
    which the weights carry into out as sum_k |W_kn| (...); the stored 16-bit out adds ulp |out|."""
    B, Sq, Hq, d = o_ref.shape
    per_k = (TOL_O + 2 * ulp * o_ref.abs()).reshape(B, Sq, Hq * d)
    return torch.matmul(per_k, w.abs()) + ulp * out_ref.abs()


def proj_case(fa, B, Hq, Hkv, Sq, Skv, d_model, causal, dtype, seed, w_kind="dense", rows=None):
    cfg = synth.PrefillConfig("proj", B, Hq, Hkv, Sq, Skv, dtype=dtype, causal=causal, seed=seed)
    q, k, v = synth.prefill_inputs(cfg, "cpu" if rows is None else DEV)
    K = Hq * 128
    gen = torch.Generator().manual_seed(seed + 1)
    if w_kind == "dense":
        w = (torch.randn(K, d_model, generator=gen) / math.sqrt(K)).to(q.dtype)
    else:   # every column has exactly one entry, +-2^e: out[:, n] = +-2^e O[:, src[n]], exact in the accumulator
        src = torch.randint(0, K, (d_model,), generator=gen)
        val = torch.tensor([1.0, -1.0, 0.5, -2.0])[torch.randint(0, 4, (d_model,), generator=gen)]
        w = torch.zeros(K, d_model)
        w[src, torch.arange(d_model)] = val
        w = w.to(q.dtype)
    qd, kd, vd, wd = q.to(DEV), k.to(DEV), v.to(DEV), w.to(DEV)
    ws = torch.empty(max(4, fa.fa_forward_proj_workspace_bytes(B, Sq)), dtype=torch.uint8, device=DEV)
    res = []
    for fused in (True, False):
        o, chk_o = guard_alloc((B, Sq, Hq, 128), q.dtype, DEV)
        lse, chk_l = guard_alloc((B, Hq, Sq), torch.float32, DEV)
        out, chk_out = guard_alloc((B, Sq, d_model), q.dtype, DEV)
        fa.fa_forward_proj(qd, kd, vd, wd, o, lse, out, causal, cfg.scale, fused, ws)
        torch.cuda.synchronize()
        check_status(fa)
        chk_o(); chk_l(); chk_out()
        assert not torch.isnan(o).any() and not torch.isnan(lse).any() and not torch.isnan(out).any()
        res.append((o, lse, out))
    # one launch or two: the same kernels on the same data in the same order
    assert torch.equal(res[0][0], res[1][0]) and torch.equal(res[0][1], res[1][1]) and torch.equal(res[0][2], res[1][2])
    o, lse, out = res[0]
    ulp = 2.0 ** -8 if dtype == "bf16" else 2.0 ** -11
    what = f"proj B{B} Hq{Hq} Hkv{Hkv} Sq{Sq} Skv{Skv} N{d_model} causal{int(causal)} {dtype} {w_kind}"
    if rows is None:
        o_ref, l_ref, out_ref = oracle.attention_proj(q, k, v, w, causal, cfg.scale)
        absv = oracle.attention_full(q, k, v.abs(), causal, cfg.scale)[0] if dtype == "bf16" else None
        assert_close_to_oracle(o, lse, o_ref, l_ref, stored_bf16=(dtype == "bf16"), p_absv=absv, what=what)
        got = out.double().cpu()
    else:
        # sampled (b, i): the oracle on those batch entries' rows, all heads
        got_l, ref_l, oref_l = [], [], []
        for (b, i) in rows:
            r3 = [(0, h, i) for h in range(Hq)]
            orow, _ = oracle.attention_rows(q[b:b + 1].cpu(), k[b:b + 1].cpu(), v[b:b + 1].cpu(), causal, cfg.scale, r3)
            o16 = orow.to(q.dtype).double()
            ref_l.append(o16.reshape(1, K) @ w.double())
            oref_l.append(orow.reshape(1, 1, Hq, 128))
            got_l.append(out[b, i].double().cpu().reshape(1, d_model))
        got, out_ref, o_ref = torch.cat(got_l).unsqueeze(0), torch.cat(ref_l).unsqueeze(0), torch.cat(oref_l, dim=1)
    diff = (got - out_ref).abs()
    allow = proj_allowance(o_ref, out_ref, w.double(), ulp)
    assert float((diff - allow).max()) <= 0.0, f"{what}: max(|d out| - bound) = {float((diff - allow).max()):.3e}"
    # the bound is sound but wide for a dense weight; a dropped head or k-block shows in the row norms
    rel = float(((got - out_ref).norm(dim=-1) / out_ref.norm(dim=-1).clamp_min(1e-30)).max())
    assert rel <= (2e-2 if dtype == "bf16" else 5e-3), f"{what}: relative row error {rel:.3e}"
    return float(diff.max()), rel


@pytest.mark.parametrize("w_kind", ["select", "dense"])
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_attention_with_output_projection_small(fa, dtype, w_kind):
    proj_case(fa, 1, 2, 2, 512, 512, 256, True, dtype, seed=120, w_kind=w_kind)          # C1's attention
    proj_case(fa, 2, 4, 2, 300, 300, 512, True, dtype, seed=121, w_kind=w_kind)          # 4 heads, 512 columns, ragged rows
    proj_case(fa, 1, 4, 1, 130, 1300, 768, False, dtype, seed=122, w_kind=w_kind)


def test_attention_with_output_projection_many_blocks(fa):
    # more projection items than CTAs, several per CTA through both accumulators and around the ring
    proj_case(fa, 3, 8, 8, 700, 700, 1024, True, "fp16", seed=123, w_kind="select")
    proj_case(fa, 3, 8, 8, 700, 700, 1024, True, "fp16", seed=124, w_kind="dense")


def test_attention_with_output_projection_c2_sampled(fa):
    c = synth.C2
    rows = [(0, 0), (0, 127), (0, 128), (1, 1000), (2, 2047), (3, 5), (3, 1029), (1, 255)]
    worst, rel = proj_case(fa, c.B, c.Hq, c.Hkv, c.Sq, c.Skv, 4096, True, "fp16", seed=125, w_kind="dense", rows=rows)
    print(f"C2 + projection to 4096 columns: max|d out| {worst:.2e}, relative row error {rel:.2e}")


# ------------------------------------------------------------------ packed variable-length batches
def varlen_case(fa, cfg, what):
    q, k, v, cu_q, cu_k = synth.varlen_inputs(cfg, "cpu")
    o_ref, l_ref = oracle.attention_varlen(q, k, v, cu_q, cu_k, cfg.causal, cfg.scale)
    absv = oracle.attention_varlen(q, k, v.abs(), cu_q, cu_k, cfg.causal, cfg.scale)[0] if cfg.dtype == "bf16" else None
    o, chk_o = guard_alloc(tuple(q.shape), q.dtype, DEV)
    lse, chk_l = guard_alloc((cfg.Hq, q.shape[0]), torch.float32, DEV)
    fa.fa_forward_varlen(q.to(DEV), k.to(DEV), v.to(DEV), o, lse, cu_q.to(DEV), cu_k.to(DEV),
                         max(cfg.seqlens_q), max(cfg.seqlens_k), cfg.causal, cfg.scale)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o(); chk_l()
    # the comparison helper takes [B,S,H,d] and [B,H,S]: the packed rows as one sequence
    assert_close_to_oracle(o.unsqueeze(0), lse.unsqueeze(0), o_ref.unsqueeze(0), l_ref.unsqueeze(0),
                           stored_bf16=(cfg.dtype == "bf16"), p_absv=None if absv is None else absv.unsqueeze(0), what=what)
    return o, lse


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_varlen_ragged_batch(fa, causal, dtype):
    # lengths on both sides of the 32-row store boxes and the 128-row tiles, an empty sequence,
    # a sequence without keys, chunked prefill (fewer queries than keys), more queries than keys
    # (causal: its first rows see nothing), GQA; every row of O and LSE is compared and the
    # guard bands around both must stay untouched
    lq = (1, 127, 128, 129, 300, 0, 40, 33, 200, 31, 260)
    lk = (1, 127, 128, 129, 300, 0, 700, 0, 90, 31, 515)
    cfg = synth.VarlenConfig("t", 4, 2, lq, lk, dtype=dtype, causal=causal, seed=600 + int(causal))
    varlen_case(fa, cfg, f"varlen ragged causal{int(causal)} {dtype}")


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_varlen_head_dimension_64(fa, dtype):
    # packed batches with d = 64 (the same kernel, tiles of one 64-element box): the ragged batch
    # of the d = 128 test, causal and not, and the same keys behind a block table
    lq = (1, 127, 128, 129, 300, 0, 40, 33, 200, 31, 260)
    lk = (1, 127, 128, 129, 300, 0, 700, 0, 90, 31, 515)
    for causal in (True, False):
        cfg = synth.VarlenConfig("t", 4, 2, lq, lk, d=64, dtype=dtype, causal=causal, seed=640 + int(causal))
        varlen_case(fa, cfg, f"varlen d=64 causal{int(causal)} {dtype}")
    lens = tuple([17, 130, 64, 5] * 30 + [1700])
    cfg = synth.VarlenConfig("t", 2, 1, lens, lens, d=64, dtype=dtype, causal=True, seed=643)
    o_packed, l_packed = varlen_case(fa, cfg, f"varlen d=64 many short + one long {dtype}")
    q, k, v, cu_q, cu_k = synth.varlen_inputs(cfg, "cpu")
    kp, vp, table = synth.paged_from_packed(k, v, lens, 128, seed=9, spare_pages=2, poison=True)
    o = torch.full(tuple(q.shape), float("nan"), dtype=q.dtype, device=DEV)
    lse = torch.full((cfg.Hq, q.shape[0]), float("nan"), dtype=torch.float32, device=DEV)
    fa.fa_forward_varlen_paged(q.to(DEV), kp.to(DEV), vp.to(DEV), table.to(DEV), o, lse, cu_q.to(DEV),
                               torch.tensor(lens, dtype=torch.int32, device=DEV), max(lens), max(lens), True, cfg.scale)
    torch.cuda.synchronize()
    check_status(fa)
    assert torch.equal(o, o_packed) and torch.equal(lse, l_packed)      # the paged form: bit for bit the packed one


def test_varlen_many_short_sequences_and_one_long(fa):
    # more items than CTAs, most of them past the end of their sequence (the launch is sized by
    # the longest sequence): skipped items must not disturb the double buffers
    lens = tuple([17, 130, 64, 5] * 40 + [2500])
    cfg = synth.VarlenConfig("t", 2, 1, lens, lens, dtype="fp16", causal=True, seed=611)
    varlen_case(fa, cfg, "varlen many short + one long")


def test_varlen_equal_lengths_match_the_batched_call_bit_for_bit(fa):
    # C2 as a packed batch must give exactly what fa_forward gives (same kernel arithmetic in the
    # same order; fa_forward on C2 is checked against the oracle elsewhere)
    c = synth.C2
    q, k, v = synth.prefill_inputs(c, DEV)
    o1 = torch.empty_like(q); l1 = torch.empty(c.B, c.Hq, c.Sq, dtype=torch.float32, device=DEV)
    fa.fa_forward(q, k, v, o1, l1, c.causal, c.scale)
    cu = torch.arange(0, (c.B + 1) * c.Sq, c.Sq, dtype=torch.int32, device=DEV)
    o2 = torch.empty(c.B * c.Sq, c.Hq, c.d, dtype=q.dtype, device=DEV)
    l2 = torch.empty(c.Hq, c.B * c.Sq, dtype=torch.float32, device=DEV)
    fa.fa_forward_varlen(q.view(-1, c.Hq, c.d), k.view(-1, c.Hkv, c.d), v.view(-1, c.Hkv, c.d), o2, l2, cu, cu,
                         c.Sq, c.Skv, c.causal, c.scale)
    torch.cuda.synchronize()
    check_status(fa)
    assert torch.equal(o1.view(-1, c.Hq, c.d), o2)
    assert torch.equal(l1, l2.view(c.Hq, c.B, c.Sq).permute(1, 0, 2))


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_varlen_over_a_paged_cache(fa, causal, dtype):
    # chunked prefill against a page pool: each sequence's queries are its last rows, its keys sit
    # in 128- or 256-key pages handed out in random order; unused pages and the rows of a last page
    # past the end of its sequence hold NaN (serving systems do not clear fresh pages: a wrong page
    # would show, and so would a product with a row that is not the sequence's).  Lengths: a key
    # count that ends exactly on a page, one key, more pages than queries, queries = keys, and a
    # sequence with queries but no keys, whose table row is never to be read and holds garbage
    lq = (70, 1, 130, 300, 128, 5, 40)
    lk = (700, 1, 130, 1000, 256, 1500, 0)
    for page in (128, 256):
        cfg = synth.VarlenConfig("t", 4, 2, lq, lk, dtype=dtype, causal=causal, seed=700 + page)
        q, k, v, cu_q, cu_k = synth.varlen_inputs(cfg, "cpu")
        B = len(lq)
        kc = torch.zeros(B, max(lk), cfg.Hkv, 128, dtype=k.dtype); vc = torch.zeros_like(kc)
        for b in range(B):
            kc[b, :lk[b]] = k[int(cu_k[b]):int(cu_k[b + 1])]
            vc[b, :lk[b]] = v[int(cu_k[b]):int(cu_k[b + 1])]
        sk = torch.tensor(lk, dtype=torch.int32)
        kp, vp, table = synth.paged_cache(kc, vc, sk, page, seed=cfg.seed, spare_pages=3, poison=True)
        assert torch.isnan(vp[int(table[0, (lk[0] - 1) // page]), -1]).all()     # page tails stay poisoned
        table[6, :] = torch.tensor([0x7ffffff0, -12345] * table.shape[1])[:table.shape[1]]
        o_ref, l_ref = oracle.attention_varlen_paged(q, kp, vp, table, cu_q, sk, causal, cfg.scale)
        o_chk, l_chk = oracle.attention_varlen(q, k, v, cu_q, cu_k, causal, cfg.scale)
        assert torch.equal(o_ref, o_chk) and torch.equal(l_ref, l_chk)
        absv = oracle.attention_varlen(q, k, v.abs(), cu_q, cu_k, causal, cfg.scale)[0] if dtype == "bf16" else None
        o, chk_o = guard_alloc(tuple(q.shape), q.dtype, DEV)
        lse, chk_l = guard_alloc((cfg.Hq, q.shape[0]), torch.float32, DEV)
        fa.fa_forward_varlen_paged(q.to(DEV), kp.to(DEV), vp.to(DEV), table.to(DEV), o, lse, cu_q.to(DEV), sk.to(DEV),
                                   max(lq), max(lk), causal, cfg.scale)
        torch.cuda.synchronize()
        check_status(fa)
        chk_o(); chk_l()
        assert_close_to_oracle(o.unsqueeze(0), lse.unsqueeze(0), o_ref.unsqueeze(0), l_ref.unsqueeze(0),
                               stored_bf16=(dtype == "bf16"), p_absv=None if absv is None else absv.unsqueeze(0),
                               what=f"varlen paged page{page} causal{int(causal)} {dtype}")


def test_varlen_without_any_keys(fa):
    cfg = synth.VarlenConfig("t", 2, 2, (5, 130), (0, 0), dtype="fp16", causal=False, seed=612)
    q, k, v, cu_q, cu_k = synth.varlen_inputs(cfg, DEV)
    o = torch.full_like(q, float("nan")); lse = torch.full((2, 135), float("nan"), device=DEV)
    fa.fa_forward_varlen(q, k, v, o, lse, cu_q.to(DEV), cu_k.to(DEV), 130, 0, False, cfg.scale)
    torch.cuda.synchronize()
    assert float(o.abs().max()) == 0.0 and torch.isneginf(lse).all()


# ------------------------------------------------------------------ decode
def run_decode(fa, q, k, v, seqlens_dev, scale):
    B, _, Hq, d = q.shape
    Smax, Hkv = k.shape[1], k.shape[2]
    o, chk_o = guard_alloc((B, 1, Hq, d), torch.float16, DEV)
    lse, chk_l = guard_alloc((B, Hq), torch.float32, DEV)
    nbytes = fa.fa_decode_workspace_bytes(B, Hq, Hkv, Smax, d)
    ws, chk_w = guard_alloc((max(nbytes // 4, 4),), torch.float32, DEV)
    fa.fa_decode(q, k, v, o, lse, seqlens_dev, scale, ws)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o(); chk_l(); chk_w()
    return o, lse


@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 4), (8, 2), (8, 1), (6, 2), (16, 1), (17, 1), (40, 2), (7, 1), (10, 2), (9, 1)])
def test_decode_small_full(fa, hq, hkv):
    # (1 to 8 query heads per kv head take the keys-as-rows consumers, 9 and more the heads-as-rows ones)
    cfg = synth.DecodeConfig("t", 5, hq, hkv, 1500, 1, 1500, seed=hq * 31 + hkv)
    q, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=True)
    sl[0], sl[1], sl[2] = 1500, 0, 1          # full, empty, single key
    for b in range(cfg.B):                     # re-poison after editing the lengths
        n = int(sl[b])
        k[b, n:] = float("nan"); v[b, n:] = float("nan")
        if n and torch.isnan(k[b, :n].float()).any():
            g = torch.Generator().manual_seed(b)
            k[b, :n] = torch.randn(n, hkv, 128, generator=g).half()
            v[b, :n] = torch.randn(n, hkv, 128, generator=g).half()
    o_ref, l_ref = oracle.decode(q, k, v, sl, cfg.scale)
    o, lse = run_decode(fa, q.to(DEV), k.to(DEV), v.to(DEV), sl.to(DEV), cfg.scale)
    assert_close_to_oracle(o[:, 0], lse, o_ref, l_ref, what=f"decode {hq}/{hkv}")
    assert float(o[1].abs().max()) == 0.0 and torch.isneginf(lse[1]).all()


def test_decode_chunked_lengths_and_clamping(fa):
    # lengths on both sides of chunk and tile boundaries; a length beyond Smax is clamped
    cfg = synth.DecodeConfig("t", 8, 8, 8, 4096, 1, 4096, seed=321)
    q, k, v, _ = synth.decode_inputs(cfg, "cpu", poison=False)
    # (the chunk length depends on the problem size: 256 to 4096 keys; the lengths straddle each candidate)
    sl = torch.tensor([127, 129, 257, 511, 1025, 2047, 2049, 99999], dtype=torch.int32)
    o_ref, l_ref = oracle.decode(q, k, v, sl.clamp(max=4096), cfg.scale)
    o, lse = run_decode(fa, q.to(DEV), k.to(DEV), v.to(DEV), sl.to(DEV), cfg.scale)
    assert_close_to_oracle(o[:, 0], lse, o_ref, l_ref, what="decode boundaries")
    o2, lse2 = run_decode(fa, q.to(DEV), k.to(DEV), v.to(DEV), sl.to(DEV), cfg.scale)
    assert torch.equal(o, o2) and torch.equal(lse, lse2)      # bit-reproducible


@pytest.mark.parametrize("cfg", [synth.C5_MHA, synth.C5_GQA], ids=["mha", "gqa"])
def test_c5_decode_full_size_sampled(fa, cfg):
    q, k, v, sl = synth.decode_inputs(cfg, DEV, poison=True)
    o, lse = run_decode(fa, q, k, v, sl.to(DEV), cfg.scale)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    g = cfg.Hq // cfg.Hkv
    gen = torch.Generator().manual_seed(cfg.seed + 5)
    order = torch.argsort(sl)
    seqs = {int(order[0]), int(order[-1]), 0, cfg.B - 1}
    seqs.update(int(x) for x in torch.randint(0, cfg.B, (6,), generator=gen))
    for b in sorted(seqs):
        n = int(sl[b])
        heads = {0, g - 1, cfg.Hq - 1, int(torch.randint(0, cfg.Hq, (1,), generator=gen))}
        for h in sorted(heads):
            hk = h // g
            qs = q[b:b + 1, :, h:h + 1].cpu()
            ks = k[b:b + 1, :n, hk:hk + 1].contiguous().cpu()
            vs = v[b:b + 1, :n, hk:hk + 1].contiguous().cpu()
            o_ref, l_ref = oracle.decode(qs, ks, vs, [n], cfg.scale)
            assert_close_to_oracle(o[b, 0, h].view(1, 1, -1), lse[b, h].view(1, 1), o_ref, l_ref,
                                   what=f"{cfg.name} b{b} h{h} n{n}")


# ------------------------------------------------------------------ decode after several appended tokens
def run_decode_append(fa, q, k, v, seqlens_dev, scale):
    B, Sq, Hq, d = q.shape
    Smax, Hkv = k.shape[1], k.shape[2]
    o, chk_o = guard_alloc((B, Sq, Hq, d), torch.float16, DEV)
    lse, chk_l = guard_alloc((B, Hq, Sq), torch.float32, DEV)
    nbytes = fa.fa_decode_append_workspace_bytes(B, Sq, Hq, Hkv, Smax, d)
    ws, chk_w = guard_alloc((max(nbytes // 4, 4),), torch.float32, DEV)
    fa.fa_decode_append(q, k, v, o, lse, seqlens_dev, scale, ws)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o(); chk_l(); chk_w()
    return o, lse


@pytest.mark.parametrize("sq,hq,hkv", [(2, 4, 4), (4, 8, 2), (5, 8, 1), (8, 8, 8), (16, 4, 1), (17, 6, 2), (3, 40, 2), (64, 2, 1),
                                       (2, 8, 2), (3, 4, 2), (7, 3, 3)])
def test_decode_append_small_full(fa, sq, hq, hkv):
    # (up to 8 (token, head) rows per kv head take the keys-as-rows consumers, more the heads-as-rows ones)
    # sq query rows = the last sq positions of each cache; lengths: long, exactly sq, shorter than
    # sq (its first queries see nothing), sq + 1, around a tile and a chunk boundary; NaN past the end
    cfg = synth.DecodeConfig("t", 7, hq, hkv, 3000, 1, 3000, seed=sq * 53 + hq + hkv)
    _, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
    sl[:] = torch.tensor([3000, sq, max(1, sq - 2), sq + 1, 129, 2049, 1500], dtype=torch.int32)
    for b in range(cfg.B):
        k[b, int(sl[b]):] = float("nan")
        v[b, int(sl[b]):] = float("nan")
    gen = torch.Generator().manual_seed(cfg.seed + 3)
    q = torch.randn(cfg.B, sq, hq, 128, generator=gen).half()
    o_ref, l_ref = oracle.decode_append(q, k, v, sl, cfg.scale)
    o, lse = run_decode_append(fa, q.to(DEV), k.to(DEV), v.to(DEV), sl.to(DEV), cfg.scale)
    assert_close_to_oracle(o, lse, o_ref, l_ref, what=f"append decode sq{sq} {hq}/{hkv}")


def test_decode_append_of_one_token_is_decode(fa):
    cfg = synth.DecodeConfig("t", 4, 8, 2, 2500, 1, 2500, seed=977)
    q, k, v, sl = synth.decode_inputs(cfg, DEV, poison=True)
    o1, l1 = run_decode(fa, q, k, v, sl.to(DEV), cfg.scale)
    o2, l2 = run_decode_append(fa, q, k, v, sl.to(DEV), cfg.scale)
    assert torch.equal(o1, o2) and torch.equal(l1, l2.view(cfg.B, cfg.Hq))


def test_decode_append_full_size_sampled(fa):
    # four new tokens per sequence on the GQA decode configuration (64 sequences, up to 32K keys)
    cfg = synth.C5_GQA
    _, k, v, sl = synth.decode_inputs(cfg, DEV, poison=True)
    gen = torch.Generator(device=DEV).manual_seed(cfg.seed + 9)
    q = torch.randn(cfg.B, 4, cfg.Hq, cfg.d, generator=gen, device=DEV).half()
    o, lse = run_decode_append(fa, q, k, v, sl.to(DEV), cfg.scale)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    g = cfg.Hq // cfg.Hkv
    order = torch.argsort(sl)
    for b in sorted({int(order[0]), int(order[-1]), 0, 17, cfg.B - 1}):
        n = int(sl[b])
        for h in (0, g - 1, cfg.Hq - 1):
            hk = h // g
            o_ref, l_ref = oracle.decode_append(q[b:b + 1, :, h:h + 1].cpu(), k[b:b + 1, :n, hk:hk + 1].contiguous().cpu(),
                                                v[b:b + 1, :n, hk:hk + 1].contiguous().cpu(), [n], cfg.scale)
            assert_close_to_oracle(o[b:b + 1, :, h:h + 1], lse[b:b + 1, h:h + 1], o_ref, l_ref, what=f"append b{b} h{h} n{n}")


# ------------------------------------------------------------------ the general decode entry, bf16
@pytest.mark.parametrize("form", ["plain", "append", "paged", "paged-append"])
@pytest.mark.parametrize("dtype", ["bf16", "fp16"])
def test_decode_ex_both_types_all_forms(fa, form, dtype):
    # fa_decode_ex: fp16 and bf16, one or five query rows per sequence, contiguous or paged cache.
    # bf16 is gated like the bf16 prefill: 2e-3 plus the exact bounds of the bf16 probabilities
    # and of the stored bf16 output, both computed from the oracle
    sq = 5 if "append" in form else 1
    cfg = synth.DecodeConfig("t", 5, 8, 2, 2600, 1, 2600, dtype=dtype, seed=1200 + sq)
    _, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
    sl[:] = torch.tensor([2600, 3, 129, 2049, 700], dtype=torch.int32)
    gen = torch.Generator().manual_seed(cfg.seed + 1)
    q = torch.randn(cfg.B, sq, cfg.Hq, 128, generator=gen).to(k.dtype)
    o_ref, l_ref = oracle.decode_append(q, k, v, sl, cfg.scale)
    absv = oracle.decode_append(q, k, v.abs(), sl, cfg.scale)[0] if dtype == "bf16" else None
    o, chk_o = guard_alloc((cfg.B, sq, cfg.Hq, 128), k.dtype, DEV)
    lse, chk_l = guard_alloc((cfg.B, cfg.Hq, sq), torch.float32, DEV)
    if "paged" in form:
        kd, vd, table = synth.paged_cache(k, v, sl, 128, seed=9, spare_pages=2, poison=True)
        table = table.to(DEV)
        smax = table.shape[1] * 128
    else:
        kd, vd, table, smax = k.clone(), v.clone(), None, cfg.Smax
        for b in range(cfg.B):
            kd[b, int(sl[b]):] = float("nan")
            vd[b, int(sl[b]):] = float("nan")
    ws, chk_w = guard_alloc((max(fa.fa_decode_append_workspace_bytes(cfg.B, sq, cfg.Hq, cfg.Hkv, smax, 128) // 4, 4),),
                            torch.float32, DEV)
    fa.fa_decode_ex(q.to(DEV), kd.to(DEV), vd.to(DEV), o, lse, sl.to(DEV), cfg.scale, ws, block_table=table)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o(); chk_l(); chk_w()
    assert_close_to_oracle(o, lse, o_ref, l_ref, stored_bf16=(dtype == "bf16"), p_absv=absv, what=f"decode_ex {form} {dtype}")


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("sq", [1, 3])
def test_decode_with_a_single_chunk_per_sequence(fa, sq, dtype):
    # caches short enough for one chunk: the split kernel writes the result itself and no merge
    # kernel runs; an empty sequence must still get its zeros and -inf.  Also a large batch of
    # 4K-key caches, where the chunk is the whole cache
    for (B, hq, hkv, smax, lens) in [(4, 8, 2, 200, [200, 0, 1, 129]), (130, 4, 1, 4096, None)]:
        cfg = synth.DecodeConfig("t", B, hq, hkv, smax, 1, smax, dtype=dtype, seed=1300 + B + sq)
        _, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
        if lens is not None:
            sl[:] = torch.tensor(lens, dtype=torch.int32)
        sl[0] = smax
        for b in range(B):
            k[b, int(sl[b]):] = float("nan")
            v[b, int(sl[b]):] = float("nan")
        assert fa.fa_decode_workspace_bytes(B, hq, hkv, smax, 128) == B * hq * 129 * 4     # one chunk
        gen = torch.Generator().manual_seed(cfg.seed + 1)
        q = torch.randn(B, sq, hq, 128, generator=gen).to(k.dtype)
        o_ref, l_ref = oracle.decode_append(q, k.nan_to_num(0.0), v.nan_to_num(0.0), sl, cfg.scale)
        absv = oracle.decode_append(q, k.nan_to_num(0.0), v.nan_to_num(0.0).abs(), sl, cfg.scale)[0] if dtype == "bf16" else None
        o, chk_o = guard_alloc((B, sq, hq, 128), k.dtype, DEV)
        lse, chk_l = guard_alloc((B, hq, sq), torch.float32, DEV)
        ws, chk_w = guard_alloc((fa.fa_decode_append_workspace_bytes(B, sq, hq, hkv, smax, 128) // 4,), torch.float32, DEV)
        fa.fa_decode_ex(q.to(DEV), k.to(DEV), v.to(DEV), o, lse, sl.to(DEV), cfg.scale, ws)
        torch.cuda.synchronize()
        check_status(fa)
        chk_o(); chk_l(); chk_w()
        assert_close_to_oracle(o, lse, o_ref, l_ref, stored_bf16=(dtype == "bf16"), p_absv=absv,
                               what=f"single-chunk decode B{B} sq{sq} {dtype}")


# ------------------------------------------------------------------ decode with head dimension 64
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("form", ["plain", "append", "paged", "paged16", "one-chunk"])
def test_decode_head_dimension_64(fa, form, dtype):
    # The 16-bit decode kernel with d = 64 (tiles of one 64-column box, six ring slots): one query
    # row and five (append), contiguous and paged caches (256-key and 16-key pages), many chunks and
    # a single one; lengths: full, empty, one key, ragged around the tile size; NaN past every end.
    sq = 5 if form == "append" else 1
    smax = 640 if form == "one-chunk" else 2560
    cfg = synth.DecodeConfig("t", 6, 8, 2, smax, 1, smax, d=64, dtype=dtype, seed=1400 + len(form))
    _, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
    sl[0], sl[1], sl[2], sl[3] = smax, 0, max(1, sq), 129 + sq
    for b in range(cfg.B):
        k[b, int(sl[b]):] = float("nan")
        v[b, int(sl[b]):] = float("nan")
    gen = torch.Generator().manual_seed(cfg.seed + 1)
    q = torch.randn(cfg.B, sq, cfg.Hq, 64, generator=gen).to(k.dtype)
    kz, vz = k.nan_to_num(0.0), v.nan_to_num(0.0)
    o_ref, l_ref = oracle.decode_append(q, kz, vz, sl, cfg.scale)
    absv = oracle.decode_append(q, kz, vz.abs(), sl, cfg.scale)[0] if dtype == "bf16" else None
    o, chk_o = guard_alloc((cfg.B, sq, cfg.Hq, 64), k.dtype, DEV)
    lse, chk_l = guard_alloc((cfg.B, cfg.Hq, sq), torch.float32, DEV)
    nbytes = fa.fa_decode_append_workspace_bytes(cfg.B, sq, cfg.Hq, cfg.Hkv, smax, 64)
    assert nbytes > 0
    ws, chk_w = guard_alloc((nbytes // 4,), torch.float32, DEV)
    table = None
    kd, vd = k, v
    if form.startswith("paged"):
        page = 16 if form == "paged16" else 256
        kd, vd, table = synth.paged_cache(k, v, sl, page, seed=9, spare_pages=2, poison=True)
        table = table.to(DEV)
    fa.fa_decode_ex(q.to(DEV), kd.to(DEV), vd.to(DEV), o, lse, sl.to(DEV), cfg.scale, ws, block_table=table)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o(); chk_l(); chk_w()
    assert_close_to_oracle(o, lse, o_ref, l_ref, stored_bf16=(dtype == "bf16"), p_absv=absv,
                           what=f"decode d=64 {form} {dtype}")
    assert float(o[1].float().abs().max()) == 0.0 and torch.isneginf(lse[1]).all()


def test_decode_head_dimension_64_large_batch_sampled(fa):
    # a batch that fills the GPU (2048-key chunks, 64 sequences of up to 16K keys, GQA): sampled rows
    cfg = synth.DecodeConfig("t", 64, 32, 8, 16384, 1024, 16384, d=64, dtype="fp16", seed=1450)
    q, k, v, sl = synth.decode_inputs(cfg, DEV, poison=True)
    o, chk_o = guard_alloc((cfg.B, 1, cfg.Hq, 64), torch.float16, DEV)
    lse, chk_l = guard_alloc((cfg.B, cfg.Hq), torch.float32, DEV)
    ws, chk_w = guard_alloc((fa.fa_decode_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Smax, 64) // 4,), torch.float32, DEV)
    fa.fa_decode(q, k, v, o, lse, sl.to(DEV), cfg.scale, ws)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o(); chk_l(); chk_w()
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    g = cfg.Hq // cfg.Hkv
    for b in (0, 17, cfg.B - 1, int(torch.argmax(sl)), int(torch.argmin(sl))):
        n = int(sl[b])
        for h in (0, g - 1, cfg.Hq - 1):
            hk = h // g
            o_ref, l_ref = oracle.decode(q[b:b + 1, :, h:h + 1].cpu(), k[b:b + 1, :n, hk:hk + 1].contiguous().cpu(),
                                         v[b:b + 1, :n, hk:hk + 1].contiguous().cpu(), [n], cfg.scale)
            assert_close_to_oracle(o[b, 0, h].view(1, 1, -1), lse[b, h].view(1, 1), o_ref, l_ref, what=f"decode d=64 b{b} h{h}")


# ------------------------------------------------------------------ decode over an FP8 cache
def run_decode_fp8(fa, q, k8, v8, seqlens_dev, scale, k_scale, v_scale):
    B, _, Hq, d = q.shape
    Smax, Hkv = k8.shape[1], k8.shape[2]
    o, chk_o = guard_alloc((B, 1, Hq, d), torch.float16, DEV)
    lse, chk_l = guard_alloc((B, Hq), torch.float32, DEV)
    nbytes = fa.fa_decode_workspace_bytes(B, Hq, Hkv, Smax, d)
    ws, chk_w = guard_alloc((max(nbytes // 4, 4),), torch.float32, DEV)
    fa.fa_decode_fp8(q, k8, v8, o, lse, seqlens_dev, scale, k_scale, v_scale, ws)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o(); chk_l(); chk_w()
    return o, lse


@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 2), (8, 1), (6, 2), (17, 1), (40, 2)])
def test_decode_fp8_small_full(fa, hq, hkv):
    # N(0,1) caches stored as e4m3 with factors 1/4 and 1/8 (so that the 8-bit grid is used over
    # its range), NaN patterns past every sequence's end; lengths: full, empty, one key, ragged
    cfg = synth.DecodeConfig("t", 5, hq, hkv, 1500, 1, 1500, seed=hq * 41 + hkv)
    q, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
    sl[0], sl[1], sl[2] = 1500, 0, 1
    k8, v8 = synth.fp8_cache(k, v, sl, 0.25, 0.125, poison=True)
    o_ref, l_ref = oracle.decode_fp8(q, k8, v8, sl, cfg.scale, 0.25, 0.125)
    o, lse = run_decode_fp8(fa, q.to(DEV), k8.to(DEV), v8.to(DEV), sl.to(DEV), cfg.scale, 0.25, 0.125)
    assert_close_to_oracle(o[:, 0], lse, o_ref, l_ref, what=f"fp8 decode {hq}/{hkv}")
    assert float(o[1].abs().max()) == 0.0 and torch.isneginf(lse[1]).all()


@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 1), (12, 1)])
def test_decode_fp8_with_a_single_chunk_per_sequence(fa, hq, hkv):
    # caches short enough for one chunk: the split kernel writes the result itself and no merge
    # kernel runs; an empty sequence must still get its zeros and -inf.  Also a large batch of
    # 4K-key caches, where the chunk is the whole cache
    for (B, smax, lens) in [(4, 200, [200, 0, 1, 129]), (130, 4096, None)]:
        cfg = synth.DecodeConfig("t", B, hq, hkv, smax, 1, smax, seed=1700 + B + hq)
        q, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
        if lens is not None:
            sl[:] = torch.tensor(lens, dtype=torch.int32)
        sl[0] = smax
        assert fa.fa_decode_workspace_bytes(B, hq, hkv, smax, 128) == B * hq * 129 * 4     # one chunk
        k8, v8 = synth.fp8_cache(k, v, sl, 0.25, 0.125, poison=True)
        o_ref, l_ref = oracle.decode_fp8(q, k8, v8, sl, cfg.scale, 0.25, 0.125)
        o, lse = run_decode_fp8(fa, q.to(DEV), k8.to(DEV), v8.to(DEV), sl.to(DEV), cfg.scale, 0.25, 0.125)
        assert_close_to_oracle(o[:, 0], lse, o_ref, l_ref, what=f"fp8 single-chunk decode B{B} {hq}/{hkv}")
        if lens is not None:
            assert float(o[1].abs().max()) == 0.0 and torch.isneginf(lse[1]).all()


def test_decode_fp8_every_bit_pattern_in_every_position(fa):
    # every finite e4m3 pattern in K and V (drawn uniformly over the bit patterns, so that
    # subnormals, both signs and the largest values occur), lengths around tile and chunk
    # boundaries; the factors keep the scores in a sane range
    cfg = synth.DecodeConfig("t", 6, 8, 4, 4096, 1, 4096, seed=555)
    q, _, _, _ = synth.decode_inputs(cfg, "cpu", poison=False)
    gen = torch.Generator().manual_seed(556)
    shape = (cfg.B, cfg.Smax, cfg.Hkv, cfg.d)
    mag = torch.randint(0, 0x7f, shape, generator=gen, dtype=torch.uint8)       # 0x00 .. 0x7e
    sgn = torch.randint(0, 2, shape, generator=gen, dtype=torch.uint8) << 7
    k8, v8 = mag | sgn, torch.randint(0, 0x7f, shape, generator=gen, dtype=torch.uint8) | sgn
    sl = torch.tensor([127, 128, 129, 2047, 2049, 4096], dtype=torch.int32)
    for b in range(cfg.B):
        k8[b, int(sl[b]):] = 0xff
        v8[b, int(sl[b]):] = 0x7f
    ks, vs = 1.0 / 256, 1.0 / 64
    o_ref, l_ref = oracle.decode_fp8(q, k8, v8, sl, cfg.scale, ks, vs)
    o, lse = run_decode_fp8(fa, q.to(DEV), k8.to(DEV), v8.to(DEV), sl.to(DEV), cfg.scale, ks, vs)
    assert_close_to_oracle(o[:, 0], lse, o_ref, l_ref, what="fp8 decode, all patterns")


@pytest.mark.parametrize("cfg", [synth.C5_MHA, synth.C5_GQA], ids=["mha", "gqa"])
def test_c5_decode_fp8_full_size_sampled(fa, cfg):
    q, k, v, sl = synth.decode_inputs(cfg, DEV, poison=False)
    k8, v8 = synth.fp8_cache(k, v, sl, 0.25, 0.125, poison=True)
    del k, v
    o, lse = run_decode_fp8(fa, q, k8, v8, sl.to(DEV), cfg.scale, 0.25, 0.125)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    g = cfg.Hq // cfg.Hkv
    gen = torch.Generator().manual_seed(cfg.seed + 6)
    order = torch.argsort(sl)
    seqs = {int(order[0]), int(order[-1]), 0, cfg.B - 1}
    seqs.update(int(x) for x in torch.randint(0, cfg.B, (4,), generator=gen))
    for b in sorted(seqs):
        n = int(sl[b])
        for h in sorted({0, g - 1, cfg.Hq - 1, int(torch.randint(0, cfg.Hq, (1,), generator=gen))}):
            hk = h // g
            o_ref, l_ref = oracle.decode_fp8(q[b:b + 1, :, h:h + 1].cpu(), k8[b:b + 1, :n, hk:hk + 1].contiguous().cpu(),
                                             v8[b:b + 1, :n, hk:hk + 1].contiguous().cpu(), [n], cfg.scale, 0.25, 0.125)
            assert_close_to_oracle(o[b, 0, h].view(1, 1, -1), lse[b, h].view(1, 1), o_ref, l_ref,
                                   what=f"{cfg.name} fp8 b{b} h{h} n{n}")


@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 2), (17, 1), (40, 2)])
def test_decode_fp8_bf16_queries(fa, hq, hkv):
    # the same 8-bit cache with q and o in bf16: q widens to fp16 exactly (N(0,1) values), the
    # probabilities are fp16 as in the fp16 form, so only the stored bf16 output adds a rounding
    # (2^-8 |O|, allowed with its exact bound); contiguous and paged forms agree bit for bit;
    # a sequence without keys and ragged lengths around the tile size are included
    cfg = synth.DecodeConfig("t", 6, hq, hkv, 2304, 1, 2304, seed=960 + hq)
    q, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
    q = q.to(torch.bfloat16)
    sl[0], sl[1], sl[2], sl[3] = 2304, 0, 1, 257
    k8, v8 = synth.fp8_cache(k, v, sl, 0.25, 0.125, poison=True)
    B, _, Hq, d = q.shape
    o, chk_o = guard_alloc((B, 1, Hq, d), torch.bfloat16, DEV)
    lse, chk_l = guard_alloc((B, Hq), torch.float32, DEV)
    ws, chk_w = guard_alloc((max(fa.fa_decode_workspace_bytes(B, Hq, cfg.Hkv, cfg.Smax, d) // 4, 4),), torch.float32, DEV)
    fa.fa_decode_fp8_bf16(q.to(DEV), k8.to(DEV), v8.to(DEV), o, lse, sl.to(DEV), cfg.scale, 0.25, 0.125, ws)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o(); chk_l(); chk_w()
    o_ref, l_ref = oracle.decode_fp8(q, k8, v8, sl, cfg.scale, 0.25, 0.125)
    assert_close_to_oracle(o[:, 0], lse, o_ref, l_ref, stored_bf16=True, what=f"fp8 decode, bf16 q/o, {hq}/{hkv}")
    page = 256
    kp, vp, table = synth.paged_cache(k8, v8, sl, page, seed=11, spare_pages=2, poison=False)
    o2 = torch.full((B, 1, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse2 = torch.full((B, Hq), float("nan"), device=DEV)
    ws2 = torch.empty(fa.fa_decode_workspace_bytes(B, Hq, cfg.Hkv, table.shape[1] * page, d), dtype=torch.uint8, device=DEV)
    fa.fa_decode_fp8_paged_bf16(q.to(DEV), kp.to(DEV), vp.to(DEV), table.to(DEV), o2, lse2, sl.to(DEV), cfg.scale, 0.25, 0.125, ws2)
    torch.cuda.synchronize()
    check_status(fa)
    assert torch.equal(o, o2) and torch.equal(lse, lse2)


def test_decode_fp8_bf16_single_chunk_writes_the_result_itself(fa):
    # short caches: one chunk per sequence, the split kernel stores the bf16 result without a merge launch
    cfg = synth.DecodeConfig("t", 5, 8, 2, 640, 1, 640, seed=977)
    q, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
    q = q.to(torch.bfloat16)
    sl[0], sl[1] = 640, 0
    k8, v8 = synth.fp8_cache(k, v, sl, 0.25, 0.125, poison=True)
    B, _, Hq, d = q.shape
    o = torch.full((B, 1, Hq, d), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), device=DEV)
    ws = torch.empty(max(16, fa.fa_decode_workspace_bytes(B, Hq, cfg.Hkv, cfg.Smax, d)), dtype=torch.uint8, device=DEV)
    fa.fa_decode_fp8_bf16(q.to(DEV), k8.to(DEV), v8.to(DEV), o, lse, sl.to(DEV), cfg.scale, 0.25, 0.125, ws)
    torch.cuda.synchronize()
    check_status(fa)
    o_ref, l_ref = oracle.decode_fp8(q, k8, v8, sl, cfg.scale, 0.25, 0.125)
    assert_close_to_oracle(o[:, 0], lse, o_ref, l_ref, stored_bf16=True, what="fp8 decode, bf16 q/o, one chunk")


@pytest.mark.parametrize("page", [256, 16, 64])
def test_decode_fp8_paged_equals_contiguous_fp8_decode(fa, page):
    # the 8-bit cache in pages: bit for bit what fa_decode_fp8 gives on the same keys stored
    # contiguously (which the tests above check against the oracle), pages in random order, NaN
    # patterns in every unused row and page
    cfg = synth.DecodeConfig("t", 6, 8, 2, 2048, 1, 2048, seed=931)
    q, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
    sl[0], sl[1], sl[2], sl[3] = 2048, 0, 1, 257
    k8, v8 = synth.fp8_cache(k, v, sl, 0.25, 0.125, poison=True)
    o1, lse1 = run_decode_fp8(fa, q.to(DEV), k8.to(DEV), v8.to(DEV), sl.to(DEV), cfg.scale, 0.25, 0.125)
    kp, vp, table = synth.paged_cache(k8, v8, sl, page, seed=7, spare_pages=3, poison=False)
    used = torch.zeros(kp.shape[0], page, dtype=torch.bool)
    for b in range(cfg.B):
        for j in range(int(sl[b])):
            used[int(table[b, j // page]), j % page] = True
    kp[~used] = 0x7f
    vp[~used] = 0xff
    B, _, Hq, d = q.shape
    o2 = torch.full((B, 1, Hq, d), float("nan"), dtype=torch.float16, device=DEV)
    lse2 = torch.full((B, Hq), float("nan"), device=DEV)
    ws = torch.empty(fa.fa_decode_workspace_bytes(B, Hq, cfg.Hkv, table.shape[1] * page, d), dtype=torch.uint8, device=DEV)
    fa.fa_decode_fp8_paged(q.to(DEV), kp.to(DEV), vp.to(DEV), table.to(DEV), o2, lse2, sl.to(DEV), cfg.scale, 0.25, 0.125, ws)
    torch.cuda.synchronize()
    check_status(fa)
    assert table.shape[1] * page == cfg.Smax
    assert torch.equal(o1, o2) and torch.equal(lse1, lse2)
    o_ref, l_ref = oracle.decode_fp8(q, k8, v8, sl, cfg.scale, 0.25, 0.125)
    assert_close_to_oracle(o2[:, 0], lse2, o_ref, l_ref, what="fp8 paged decode")


# ------------------------------------------------------------------ decode over a paged cache
def run_decode_paged(fa, q, kp, vp, table_dev, seqlens_dev, scale, max_pages=None):
    B, _, Hq, d = q.shape
    page_size, Hkv = kp.shape[1], kp.shape[2]
    mp = table_dev.shape[1] if max_pages is None else max_pages
    o, chk_o = guard_alloc((B, 1, Hq, d), torch.float16, DEV)
    lse, chk_l = guard_alloc((B, Hq), torch.float32, DEV)
    nbytes = fa.fa_decode_workspace_bytes(B, Hq, Hkv, mp * page_size, d)
    ws, chk_w = guard_alloc((max(nbytes // 4, 4),), torch.float32, DEV)
    fa.fa_decode_paged(q, kp, vp, table_dev, o, lse, seqlens_dev, scale, ws, max_pages=mp)
    torch.cuda.synchronize()
    check_status(fa)
    chk_o(); chk_l(); chk_w()
    return o, lse


@pytest.mark.parametrize("hq,hkv,page", [(4, 4, 128), (8, 2, 128), (8, 2, 256), (17, 1, 384), (40, 2, 512),
                                         (4, 4, 16), (8, 2, 32), (8, 1, 64), (17, 1, 16)])
def test_decode_paged_small_full(fa, hq, hkv, page):
    # pages handed out in random order from a pool with unused pages; NaN in every row no key
    # lives in; lengths: several pages, none, one key, exactly one page, one past a page
    cfg = synth.DecodeConfig("t", 6, hq, hkv, 1500, 1, 1500, seed=hq * 37 + hkv + page)
    q, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
    sl[0], sl[1], sl[2], sl[3], sl[4] = 1500, 0, 1, page, page + 1
    kp, vp, table = synth.paged_cache(k, v, sl, page, seed=cfg.seed + 1, spare_pages=3, poison=True)
    o_ref, l_ref = oracle.decode_paged(q, kp, vp, table, sl, cfg.scale)
    o, lse = run_decode_paged(fa, q.to(DEV), kp.to(DEV), vp.to(DEV), table.to(DEV), sl.to(DEV), cfg.scale)
    assert_close_to_oracle(o[:, 0], lse, o_ref, l_ref, what=f"paged decode {hq}/{hkv} page {page}")
    assert float(o[1].abs().max()) == 0.0 and torch.isneginf(lse[1]).all()


def test_decode_paged_table_with_a_wider_stride_and_clamped_length(fa):
    # the table is a view into a wider array (stride > max_pages); a length beyond
    # max_pages * page_size is clamped
    cfg = synth.DecodeConfig("t", 3, 8, 4, 1024, 1, 1024, seed=911)
    q, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=False)
    sl[0], sl[1], sl[2] = 1024, 300, 1024
    kp, vp, table = synth.paged_cache(k, v, sl, 256, seed=5, poison=True)
    o_ref, l_ref = oracle.decode_paged(q, kp, vp, table, sl, cfg.scale)
    wide = torch.full((3, 9), -1, dtype=torch.int32)
    wide[:, :4] = table
    sl_dev = sl.clone(); sl_dev[2] = 99999
    o, lse = run_decode_paged(fa, q.to(DEV), kp.to(DEV), vp.to(DEV), wide.to(DEV)[:, :4], sl_dev.to(DEV), cfg.scale)
    assert_close_to_oracle(o[:, 0], lse, o_ref, l_ref, what="paged decode, strided table")


@pytest.mark.parametrize("cfg", [synth.C5_MHA, synth.C5_GQA], ids=["mha", "gqa"])
def test_c5_decode_paged_full_size_equals_contiguous_decode(fa, cfg):
    # at full size: the paged call must give, bit for bit, what fa_decode gives on the same
    # keys stored contiguously (same chunks, same order of operations; fa_decode itself is
    # checked against the oracle above), with the pages in random order
    q, k, v, sl = synth.decode_inputs(cfg, DEV, poison=True)
    o1, lse1 = run_decode(fa, q, k, v, sl.to(DEV), cfg.scale)
    kp, vp, table = synth.paged_cache(k, v, sl, 256, seed=cfg.seed + 2, spare_pages=5, poison=True)
    del k, v
    assert table.shape[1] * 256 == cfg.Smax
    o2, lse2 = run_decode_paged(fa, q, kp, vp, table.to(DEV), sl.to(DEV), cfg.scale)
    assert torch.equal(o1, o2) and torch.equal(lse1, lse2)


# ------------------------------------------------------------------ stream capture
def test_calls_can_be_captured_in_a_cuda_graph_and_replayed(fa):
    # the entry points only launch kernels on the caller's stream (no allocation, no
    # synchronisation), so after one warm-up call each they can be recorded in a CUDA graph;
    # the replay on new inputs (same buffers) must give what a direct call gives
    pc = synth.PrefillConfig("t", 2, 4, 2, 300, 1300, dtype="fp16", causal=True, seed=950)
    dc = synth.DecodeConfig("t", 4, 8, 2, 3000, 1, 3000, seed=951)
    q, k, v = synth.prefill_inputs(pc, DEV)
    o = torch.empty_like(q); lse = torch.empty(pc.B, pc.Hq, pc.Sq, device=DEV)
    dq, dk, dv, sl = synth.decode_inputs(dc, DEV, poison=True)
    sld = sl.to(DEV)
    do = torch.empty_like(dq); dl = torch.empty(dc.B, dc.Hq, device=DEV)
    ws = torch.empty(fa.fa_decode_workspace_bytes(dc.B, dc.Hq, dc.Hkv, dc.Smax, dc.d), dtype=torch.uint8, device=DEV)

    def both():
        fa.fa_forward(q, k, v, o, lse, pc.causal, pc.scale)
        fa.fa_decode(dq, dk, dv, do, dl, sld, dc.scale, ws)

    both()                                  # first use of each kernel outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            both()
    torch.cuda.synchronize()
    q.copy_(torch.flip(q, dims=[1]))        # new inputs in the same buffers
    dq.mul_(-1.0)
    both()
    torch.cuda.synchronize()
    o_direct, lse_direct, do_direct, dl_direct = o.clone(), lse.clone(), do.clone(), dl.clone()
    o.fill_(float("nan")); lse.fill_(float("nan")); do.fill_(float("nan")); dl.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    check_status(fa)
    assert torch.equal(o, o_direct) and torch.equal(lse, lse_direct)
    assert torch.equal(do, do_direct) and torch.equal(dl, dl_direct)


# ------------------------------------------------------------------ host-buffer entry point
def test_forward_host_entry(fa):
    c = synth.C1
    q, k, v = (t.pin_memory() for t in synth.prefill_inputs(c, "cpu"))
    o = torch.empty_like(q).pin_memory()
    lse = torch.empty(c.B, c.Hq, c.Sq, dtype=torch.float32).pin_memory()
    n = fa.fa_forward_host_staging_bytes(c.B, c.Hq, c.Hkv, c.Sq, c.Skv, c.d)
    st = torch.empty(n + 1024, dtype=torch.uint8, device=DEV)
    off = (-st.data_ptr()) % 1024
    fa.fa_forward_host(q, k, v, o, lse, c.causal, c.scale, st[off:off + n])
    torch.cuda.synchronize()
    check_status(fa)
    o_ref, l_ref = oracle.attention_full(q, k, v, c.causal, c.scale)
    assert_close_to_oracle(o, lse, o_ref, l_ref, what="host entry")


@pytest.mark.parametrize("d", [64, 256])
def test_forward_host_entry_other_head_dimensions(fa, d):
    # the host entry takes the head dimensions fa_forward takes: the staging layout follows d
    cfg = synth.PrefillConfig("t", 3, 4, 2, 150, 300, d=d, dtype="fp16", causal=True, seed=90 + d)
    q, k, v = (t.pin_memory() for t in synth.prefill_inputs(cfg, "cpu"))
    o = torch.full_like(q, float("nan")).pin_memory()
    lse = torch.full((cfg.B, cfg.Hq, cfg.Sq), float("nan"), dtype=torch.float32).pin_memory()
    n = fa.fa_forward_host_staging_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Skv, cfg.d)
    st = torch.empty(n + 1024, dtype=torch.uint8, device=DEV)
    off = (-st.data_ptr()) % 1024
    fa.fa_forward_host(q, k, v, o, lse, True, cfg.scale, st[off:off + n])
    torch.cuda.synchronize()
    check_status(fa)
    o_ref, l_ref = oracle.attention_full(q, k, v, True, cfg.scale)
    assert_close_to_oracle(o, lse, o_ref, l_ref, what=f"host entry d={d}")


@pytest.mark.parametrize("B", [2, 5])
def test_forward_host_entry_batch_parts(fa, B):
    # the host entry cuts the batch into up to four parts that it copies and computes in a
    # pipeline over its own streams: even and uneven splits, bf16, twice in a row on one staging
    # buffer (the second call must wait for the first one's copies out), NaN-filled outputs
    cfg = synth.PrefillConfig("t", B, 4, 2, 200, 333, dtype="bf16", causal=True, seed=70 + B)
    q, k, v = (t.pin_memory() for t in synth.prefill_inputs(cfg, "cpu"))
    o_ref, l_ref = oracle.attention_full(q, k, v, True, cfg.scale)
    absv = oracle.attention_full(q, k, v.abs(), True, cfg.scale)[0]
    n = fa.fa_forward_host_staging_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Skv, cfg.d)
    st = torch.empty(n + 1024, dtype=torch.uint8, device=DEV)
    off = (-st.data_ptr()) % 1024
    outs = []
    for _ in range(2):
        o = torch.full_like(q, float("nan")).pin_memory()
        lse = torch.full((cfg.B, cfg.Hq, cfg.Sq), float("nan"), dtype=torch.float32).pin_memory()
        fa.fa_forward_host(q, k, v, o, lse, True, cfg.scale, st[off:off + n])
        outs.append((o, lse))
    torch.cuda.synchronize()
    check_status(fa)
    for o, lse in outs:
        assert_close_to_oracle(o, lse, o_ref, l_ref, stored_bf16=True, p_absv=absv, what=f"host entry B={B}")
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])



# ------------------------------------------------------------------ the give-up path of the bounded waits
def test_a_wait_that_cannot_be_satisfied_gives_up_and_is_reported(fa):
    # every device-side wait of the library is bounded; this runs the give-up path on purpose, in
    # a kernel made for it: 64 threads wait at most 2 ms on a barrier that stays one arrival short.
    # The wait expires by itself (nothing traps, faults or spins for ever), every thread returns,
    # the status word names the place once, and the device is as usable as before.
    check_status(fa)
    gave_up = torch.zeros(1, dtype=torch.int32, device=DEV)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    fa.fa_selftest_wait(2000, gave_up)
    t1.record()
    torch.cuda.synchronize()
    assert int(gave_up.item()) == 64
    assert 1.5 <= t0.elapsed_time(t1) <= 500.0           # it waited about the limit, not for ever
    rc, where, blk = fa.fa_device_status()
    assert rc == fa.FA_ERR_TIMEOUT and where == 990 and blk == 0
    assert fa.fa_device_status()[0] == fa.FA_OK          # reported once, then cleared
    # and an ordinary forward right after it is still correct
    c = synth.C1
    q, k, v = synth.prefill_inputs(c, "cpu")
    o_ref, l_ref = oracle.attention_full(q, k, v, c.causal, c.scale)
    o, lse = run_forward(fa, q.to(DEV), k.to(DEV), v.to(DEV), c.causal, c.scale)
    assert_close_to_oracle(o, lse, o_ref, l_ref, what="C1 after the self-test")
