"""Runs one attention case through the C ABI a few times and prints its device time.

Meant for profilers (ncu wraps this command) and quick timing:
  python -m paper_2410_16663_b200.run_case prefill --B 1 --H 32 --Hkv 32 --S 8192 --dtype bf16 --iters 3
  python -m paper_2410_16663_b200.run_case decode  --B 16 --H 32 --Hkv 8 --Smax 16384 --iters 3
  python -m paper_2410_16663_b200.run_case decode  --B 16 --H 32 --Hkv 8 --Smax 16384 --d 64    (head dimension 64)
  python -m paper_2410_16663_b200.run_case prefill --B 1 --H 32 --S 8192 --fp8           (8-bit operands)
  python -m paper_2410_16663_b200.run_case proj    --B 4 --H 32 --S 2048 --fused 1       (attention + projection)
"""
from __future__ import annotations

import argparse
import math

import torch

from . import binding as fa
from . import inputs as synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kind", choices=["prefill", "decode", "proj"])
    ap.add_argument("--B", type=int, default=1)
    ap.add_argument("--H", type=int, default=32)
    ap.add_argument("--Hkv", type=int, default=0)
    ap.add_argument("--S", type=int, default=8192)
    ap.add_argument("--Skv", type=int, default=0)
    ap.add_argument("--Smax", type=int, default=16384)
    ap.add_argument("--d", type=int, default=128, choices=[64, 128, 256], help="head dimension (prefill: 64, 128, 256; decode: 64, 128)")
    ap.add_argument("--dtype", default="fp16", choices=["fp16", "bf16"])
    ap.add_argument("--noncausal", action="store_true")
    ap.add_argument("--fp8", action="store_true", help="decode: the cache as FP8 e4m3 (factors 1/4 and 1/8); "
                                                       "prefill: q, k, v as FP8 e4m3 (fa_forward_fp8)")
    ap.add_argument("--fused", type=int, default=1, help="proj: one launch (1) or two (0)")
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    a = ap.parse_args()
    hkv = a.Hkv or a.H
    dev = "cuda"
    if a.kind == "prefill":
        cfg = synth.PrefillConfig("case", a.B, a.H, hkv, a.S, a.Skv or a.S, d=a.d, dtype=a.dtype,
                                  causal=not a.noncausal, seed=7)
        q, k, v = synth.prefill_inputs(cfg, dev)
        o = torch.empty_like(q)
        lse = torch.empty(cfg.B, cfg.Hq, cfg.Sq, dtype=torch.float32, device=dev)
        run = lambda: fa.fa_forward_ex(q, k, v, o, lse, cfg.causal, cfg.scale, variant=a.variant)
        if a.fp8:
            q8, k8, v8 = synth.fp8_operands(q, k, v, 0.125, 0.25, 0.0625)
            o = torch.empty(q.shape, dtype=torch.float16, device=dev)
            run = lambda: fa.fa_forward_fp8(q8, k8, v8, o, lse, cfg.causal, cfg.scale, 0.125, 0.25, 0.0625)
        work, unit = cfg.flops() / 1e12, "TFLOPS"
    elif a.kind == "proj":
        cfg = synth.PrefillConfig("case", a.B, a.H, hkv, a.S, a.Skv or a.S, d=128, dtype=a.dtype,
                                  causal=not a.noncausal, seed=7)
        q, k, v = synth.prefill_inputs(cfg, dev)
        K = a.H * 128
        w = (torch.randn(K, K, device=dev) / math.sqrt(K)).to(q.dtype)
        o = torch.empty_like(q)
        lse = torch.empty(cfg.B, cfg.Hq, cfg.Sq, dtype=torch.float32, device=dev)
        out = torch.empty(cfg.B, cfg.Sq, K, dtype=q.dtype, device=dev)
        ws = torch.empty(max(4, fa.fa_forward_proj_workspace_bytes(cfg.B, cfg.Sq)), dtype=torch.uint8, device=dev)
        run = lambda: fa.fa_forward_proj(q, k, v, w, o, lse, out, cfg.causal, cfg.scale, bool(a.fused), ws)
        work, unit = (cfg.flops() + 2.0 * cfg.B * cfg.Sq * K * K) / 1e12, "TFLOPS"
    else:
        if a.d == 256 or (a.fp8 and a.d != 128):
            raise SystemExit("decode takes d = 128 or 64 (the 8-bit cache form d = 128 only)")
        cfg = synth.DecodeConfig("case", a.B, a.H, hkv, a.Smax, max(1, a.Smax // 32), a.Smax, d=a.d, seed=8)
        q, k, v, sl = synth.decode_inputs(cfg, dev, poison=True)
        o = torch.empty_like(q)
        lse = torch.empty(cfg.B, cfg.Hq, dtype=torch.float32, device=dev)
        ws = torch.empty(max(16, fa.fa_decode_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Smax, cfg.d)),
                         dtype=torch.uint8, device=dev)
        sld = sl.to(dev)
        if a.fp8:
            k8, v8 = synth.fp8_cache(k, v, sl, 0.25, 0.125, poison=True)
            del k, v
            run = lambda: fa.fa_decode_fp8(q, k8, v8, o, lse, sld, cfg.scale, 0.25, 0.125, ws)
        else:
            run = lambda: fa.fa_decode(q, k, v, o, lse, sld, cfg.scale, ws)
        work, unit = float(sl.sum()) * cfg.Hkv * cfg.d * (2 if a.fp8 else 4) / 1e9, "GB/s"
    for _ in range(a.warmup):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    rc, where, blk = fa.fa_device_status()
    print(f"{a.kind} {vars(a)}: {ms:.4f} ms/iter, {work / (ms * 1e-3):.1f} {unit}, status {rc} {where} {blk}")


if __name__ == "__main__":
    main()
