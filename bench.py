#!/usr/bin/env python
"""Benchmark of the attention hot path on B200: one JSON line on stdout.

A step is one pass of the whole path over one batch of synthetic input:
  1. causal prefill, Llama-7B shape (B=4, Hq=Hkv=32, S=2048, d=128, fp16)  -> fa_forward
  2. split-KV decode, B=64, Hq=32, Hkv=32, Skv ~ U[1K,32K], fp16 cache     -> fa_decode
  3. the same decode with Hkv=8 (grouped-query variant)                   -> fa_decode
Each part is timed with CUDA events on the launching stream inside the step.  `value` is the
prefill throughput in TFLOPS (causal FLOPs credited as 2*B*Hq*Sq*Skv*d); the decode parts
report cache bytes per second.  Inputs are resident in HBM before the timed region; the `e2e`
object repeats the measurement through the host-buffer entry point with the copies timed.

`--impl reference` times the CPU oracle (oracle/) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2410_16663_b200 import inputs as synth

METRIC = "causal fp16 attention fwd TFLOPS + % of tensor peak; decode KV HBM GB/s"
NOMINAL_TENSOR_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_traffic():
    """DRAM bytes per launch of the two roofline kernels, from the ncu captures kept under
    profiles/ (the file records the commit each figure was captured at)."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            return json.load(f)
    except Exception:
        return {}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        pk["source"] = "measured"
        return pk
    pk = dict(FALLBACK_PEAKS)
    pk["source"] = "fallback"
    return pk


# --------------------------------------------------------------------------- clock sampling
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {}
        for n in dir(nv):
            if n.startswith("nvmlClocksThrottleReason") or n.startswith("nvmlClocksEventReason"):
                val = getattr(nv, n)
                if isinstance(val, int) and val not in (0,):
                    names[val] = n.replace("nvmlClocksThrottleReason", "").replace("nvmlClocksEventReason", "")
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit and bit & (bit - 1) == 0 and name not in ("GpuIdle", "All"):
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples), "sm_mhz_min": min(self.samples) if self.samples else None,
                "sm_mhz_max_seen": max(self.samples) if self.samples else None, "period_ms": self.period * 1e3}


# --------------------------------------------------------------------------- workload
def visible_device_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def decode_cache_bytes(cfg, seqlens) -> float:
    """Algorithmic HBM bytes of one decode pass: every valid K and V row once, plus q, o."""
    kv = float(seqlens.sum().item()) * cfg.Hkv * cfg.d * 2 * 2
    return kv + 2.0 * cfg.B * cfg.Hq * cfg.d * 2


def max_over_ranks(values, world, device):
    """Element-wise maximum of per-rank device timings over all ranks (the slowest rank sets the
    job's time); every rank gets the result.  No data-path collective exists in this workload:
    this reduction of a few timing scalars is the only communication."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.barrier()
    return [float(x) for x in t]


def whole_job_rate(units_per_rank: float, world: int, ms: float) -> float:
    """Aggregate rate of `world` ranks that each process `units_per_rank` in `ms` (weak scaling)."""
    return world * units_per_rank / (ms * 1e-3)


def run_product(args, rank, world, local_rank):
    from paper_2410_16663_b200 import binding as fa  # raises if the CUDA library is missing

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback exists)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    peaks = load_peaks()

    pc = synth.C2
    dcs = [synth.C5_MHA, synth.C5_GQA]
    if args.small:  # debugging aid: same path, small shapes (not a reportable number)
        pc = synth.PrefillConfig("C2-small", 1, 8, 8, 1024, 1024, seed=5)
        dcs = [synth.DecodeConfig("C5-small", 8, 8, 8, 4096, 512, 4096, seed=6),
               synth.DecodeConfig("C5-small-gqa", 8, 8, 2, 4096, 512, 4096, seed=7)]

    q, k, v = synth.prefill_inputs(pc, device=dev)
    o = torch.empty_like(q)
    lse = torch.empty(pc.B, pc.Hq, pc.Sq, dtype=torch.float32, device=dev)
    dec = []
    for dc in dcs:
        dq, dk, dv, sl = synth.decode_inputs(dc, device=dev, poison=True)
        do = torch.empty_like(dq)
        dl = torch.empty(dc.B, dc.Hq, dtype=torch.float32, device=dev)
        ws = torch.empty(max(16, fa.fa_decode_workspace_bytes(dc.B, dc.Hq, dc.Hkv, dc.Smax, dc.d)),
                         dtype=torch.uint8, device=dev)
        dec.append(dict(cfg=dc, q=dq, k=dk, v=dv, sl_host=sl, sl=sl.to(dev), o=do, lse=dl, ws=ws,
                        bytes=decode_cache_bytes(dc, sl)))

    def step(ev=None):
        if ev: ev[0].record()
        fa.fa_forward(q, k, v, o, lse, pc.causal, pc.scale)
        if ev: ev[1].record()
        for i, d in enumerate(dec):
            fa.fa_decode(d["q"], d["k"], d["v"], d["o"], d["lse"], d["sl"], d["cfg"].scale, d["ws"])
            if ev: ev[2 + i].record()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")

    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    sampler = ClockSampler(visible_device_index(local_rank))
    nparts = 1 + len(dec)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(nparts + 1)] for _ in range(args.steps)]
    torch.cuda.synchronize()
    sampler.start()
    t_all0 = torch.cuda.Event(enable_timing=True)
    t_all1 = torch.cuda.Event(enable_timing=True)
    t_all0.record()
    for s in range(args.steps):
        step(events[s])
    t_all1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    total_ms = t_all0.elapsed_time(t_all1)
    part_ms = [sum(ev[i].elapsed_time(ev[i + 1]) for ev in events) / args.steps for i in range(nparts)]
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")

    # ---- max over ranks (device-timed), whole-job aggregate
    ms_step = total_ms / args.steps
    times = max_over_ranks([ms_step] + part_ms, world, dev)
    ms_step, part_ms = times[0], times[1:]

    tflops = whole_job_rate(pc.flops(), world, part_ms[0]) / 1e12
    out = {
        "metric": METRIC, "value": round(tflops, 2), "unit": "TFLOPS", "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16",
        "data": "synthetic",
        "config": {"workload": f"{pc.name}: causal prefill B={pc.B} Hq=Hkv={pc.Hq} Sq=Skv={pc.Sq} d=128 fp16"
                               f" + decode {dcs[0].name} and {dcs[1].name} (B={dcs[0].B}, Hq={dcs[0].Hq},"
                               f" Hkv={dcs[0].Hkv}/{dcs[1].Hkv}, Skv~U[{dcs[0].len_lo},{dcs[0].len_hi}])",
                   "parallelism": f"replicas x{world} (batch/head sharding, no collective)",
                   "l2": "inputs larger than L2 (prefill 256 MiB per step; the decode passes between "
                         "prefill launches stream tens of GiB)",
                   "flop_convention": "causal 2*B*Hq*Sq*Skv*d"},
        "prefill": {"ms": round(part_ms[0], 4), "tflops": round(tflops, 2),
                    "frac_nominal_tensor": round(tflops / world / NOMINAL_TENSOR_TFLOPS, 4),
                    "frac_measured_tensor": round(tflops / world / peaks["bf16_tflops"], 4)},
        "gpu_launches": args.steps * (1 + 2 * len(dec)),
        "clocks": clocks,
    }
    if clocks.get("sm_mhz"):
        # prefill time in SM clocks (ms x median MHz over the timed region): lets runs on boxes whose
        # clocks settled differently be compared; approximate, since the samples cover whole steps
        out["prefill"]["kclocks_at_median_mhz"] = round(part_ms[0] * clocks["sm_mhz"], 1)
    for i, d in enumerate(dec):
        gbs = whole_job_rate(d["bytes"], world, part_ms[1 + i]) / 1e9
        out["decode_" + ("mha" if i == 0 else "gqa")] = {
            "ms": round(part_ms[1 + i], 4), "gbs": round(gbs, 1), "kv_bytes": d["bytes"],
            "frac_nominal_hbm": round(gbs / world / NOMINAL_HBM_GBS, 4),
            "frac_measured_hbm": round(gbs / world / peaks["hbm_gbs"], 4)}
    # roofline of the kernel behind `value` (prefill: a dense contraction -> tensor peak, burst
    # figure because one launch lasts a fraction of a millisecond) and of the decode scan (HBM)
    # `traffic`: DRAM bytes per launch from one ncu capture (profiles/): the C2 prefill launch
    # itself, and for decode a 4.3 GB case of the same kernel whose dram bytes were 1.007 x its
    # algorithmic bytes, scaled to this launch by the cache bytes it scans
    traffic = load_traffic()
    c2_rec = traffic.get("prefill_c2", {})
    c2_traffic = c2_rec.get("dram_bytes_per_launch") if (pc.B, pc.Hq, pc.Sq) == (4, 32, 2048) else None
    dec_ratio = traffic.get("decode_split", {}).get("dram_bytes_over_algorithmic")
    algo_prefill_bytes = (2.0 * pc.B * pc.Sq * pc.Hq + 2.0 * pc.B * pc.Skv * pc.Hkv) * pc.d * 2 + 4.0 * pc.B * pc.Hq * pc.Sq
    out["roofline"] = {"kernel": "fa_fwd_pingpong_kernel (prefill C2, the kernel behind `value`; the library picks it for Skv >= 1024)", "bound": "tensor",
                       "achieved": round(tflops / world, 2), "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                       "frac": round(tflops / world / peaks["bf16_tflops"], 4),
                       "peak_source": peaks["source"] + " bf16 GEMM burst (of measured; fp16 has the same nominal rate)",
                       "frac_nominal": round(tflops / world / NOMINAL_TENSOR_TFLOPS, 4),
                       "algorithmic_flops": pc.flops(), "algorithmic_bytes": algo_prefill_bytes,
                       "traffic": c2_traffic, "traffic_source": c2_rec.get("source")}
    g0 = out["decode_mha"]["gbs"] / world
    out["roofline_decode"] = {"kernel": "fa_decode_split_mma_kernel (decode Hkv=32, the dominant kernel by time)",
                              "bound": "hbm", "achieved": round(g0, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                              "frac": round(g0 / peaks["hbm_gbs"], 4),
                              "peak_source": peaks["source"] + " copy bandwidth (of measured; the scan only reads)",
                              "frac_nominal": round(g0 / NOMINAL_HBM_GBS, 4),
                              "algorithmic_bytes": dec[0]["bytes"],
                              "traffic": round(dec_ratio * dec[0]["bytes"]) if dec_ratio else None,
                              "traffic_source": traffic.get("decode_split", {}).get("source")}

    if rank == 0:
        # the same prefill launch back to back, without the decode passes in between: inside the
        # step it runs right after ~3 ms of HBM streaming at the board's power cap and is slower
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(100):   # long enough for the clocks to settle after the memory-bound decode passes
            fa.fa_forward(q, k, v, o, lse, pc.causal, pc.scale)
        e0.record()
        for _ in range(50):
            fa.fa_forward(q, k, v, o, lse, pc.causal, pc.scale)
        e1.record()
        torch.cuda.synchronize()
        ms_b2b = e0.elapsed_time(e1) / 50
        out["prefill"]["back_to_back"] = {"ms": round(ms_b2b, 4), "tflops": round(pc.flops() / (ms_b2b * 1e-3) / 1e12, 2),
                                          "note": "50 launches after 100 untimed ones, without the decode passes between them (inputs 256 MiB > L2); context, not `value`"}
        if not args.small:
            out["prefill_long_context"] = run_long_context(fa, dev, peaks)
        out["decode_paged"] = run_decode_paged(fa, dec[0], dev, peaks)
        out["decode_fp8"] = run_decode_fp8(fa, dec[0], dev, peaks)
        out["decode_append"] = run_decode_append(fa, dec[-1], dev, peaks)
        out["prefill_varlen"] = run_varlen(fa, dev, peaks, small=args.small)
        out["prefill_d64"] = run_d64(fa, dev, peaks, small=args.small)
        out["prefill_d256"] = run_d256(fa, dev, peaks, small=args.small)
        out["d64_long_and_decode"] = run_d64_long(fa, dev, peaks, small=args.small)
        out["prefill_fp8"] = run_prefill_fp8(fa, dev, peaks, small=args.small)
        out["prefill_proj"] = run_prefill_proj(fa, dev, peaks, small=args.small)
        out["e2e"] = run_e2e(args, fa, pc, dec, dev)
        out["cpu_baseline"] = run_cpu_baseline(pc, budget_s=args.cpu_seconds)
        print(json.dumps(out), flush=True)


def run_long_context(fa, dev, peaks):
    """Context for the headline number, outside the timed steps: the long-sequence and GQA prefill
    configurations (bf16, causal), which the library serves with its ping-pong kernel.  Inputs
    are larger than L2 (>= 192 MiB per launch); CUDA events around back-to-back launches."""
    res = {"kernel": "fa_fwd_pingpong_kernel (the same kernel as for C2)", "dtype": "bf16", "cases": {}}
    for cfg, iters in ((synth.C3[8192], 10), (synth.C3[32768], 3), (synth.C4, 5), (synth.C3[131072], 2), (synth.C3[262144], 1)):
        q, k, v = synth.prefill_inputs(cfg, device=dev)
        o = torch.empty_like(q)
        lse = torch.empty(cfg.B, cfg.Hq, cfg.Sq, dtype=torch.float32, device=dev)
        for _ in range(3 if cfg.Sq <= 32768 else 1):
            fa.fa_forward(q, k, v, o, lse, cfg.causal, cfg.scale)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fa.fa_forward(q, k, v, o, lse, cfg.causal, cfg.scale)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        tf = cfg.flops() / (ms * 1e-3) / 1e12
        res["cases"][cfg.name] = {"ms": round(ms, 4), "tflops": round(tf, 1),
                                  "frac_nominal_tensor": round(tf / NOMINAL_TENSOR_TFLOPS, 4),
                                  "frac_measured_tensor": round(tf / peaks["bf16_tflops"], 4)}
        del q, k, v, o, lse
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")
    return res


def _time_launches(fa, run, warm, iters):
    for _ in range(warm):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        run()
    e1.record()
    torch.cuda.synchronize()
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")
    return e0.elapsed_time(e1) / iters


def run_prefill_fp8(fa, dev, peaks, small=False):
    """The headline shape and the 8K long-context shape with 8-bit operands (fa_forward_fp8: Q, K, V
    and the probabilities as FP8 e4m3 on the tensor cores), next to the 16-bit kernel on the same
    numbers in the same process, outside the timed steps.  The fp8 tensor peak is twice the 16-bit
    one; the fractions below are against that."""
    res = {"kernel": "fa_fwd_pingpong_kernel, 8-bit operand instantiation (tcgen05 kind::f8f6f4)", "cases": {}}
    cfgs = [synth.PrefillConfig("C2-small", 1, 8, 8, 1024, 1024, seed=5)] if small else [synth.C2, synth.C3[8192]]
    for cfg in cfgs:
        c16 = synth.PrefillConfig(cfg.name, cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Skv, dtype="fp16", causal=True, seed=cfg.seed)
        q, k, v = synth.prefill_inputs(c16, device=dev)
        q8, k8, v8 = synth.fp8_operands(q, k, v, 0.125, 0.25, 0.0625)
        o = torch.empty_like(q)
        lse = torch.empty(cfg.B, cfg.Hq, cfg.Sq, dtype=torch.float32, device=dev)
        # alternately, twice each, and the faster of the two: the launches are long enough for the
        # board's power state to move between them
        run16 = lambda: fa.fa_forward(q, k, v, o, lse, True, c16.scale)
        run8 = lambda: fa.fa_forward_fp8(q8, k8, v8, o, lse, True, c16.scale, 0.125, 0.25, 0.0625)
        ms16 = _time_launches(fa, run16, 20, 20)
        ms8 = _time_launches(fa, run8, 20, 20)
        ms16 = min(ms16, _time_launches(fa, run16, 5, 20))
        ms8 = min(ms8, _time_launches(fa, run8, 5, 20))
        tf8 = c16.flops() / (ms8 * 1e-3) / 1e12
        res["cases"][cfg.name] = {"ms_fp8": round(ms8, 4), "tflops_fp8": round(tf8, 1), "ms_fp16": round(ms16, 4),
                                  "tflops_fp16": round(c16.flops() / (ms16 * 1e-3) / 1e12, 1),
                                  "speedup": round(ms16 / ms8, 3),
                                  "frac_nominal_fp8_tensor": round(tf8 / (2 * NOMINAL_TENSOR_TFLOPS), 4)}
        del q, k, v, q8, k8, v8, o, lse
    return res


def run_prefill_proj(fa, dev, peaks, small=False):
    """Attention followed by the output projection to d_model = Hq * 128 columns (fa_forward_proj) on
    the headline shape: one launch against the same two kernels as two launches, outside the timed
    steps; torch.matmul on the same operands for the size of the projection itself."""
    cfg = synth.PrefillConfig("C2-small", 1, 8, 8, 1024, 1024, seed=5) if small else synth.C2
    q, k, v = synth.prefill_inputs(cfg, device=dev)
    K = cfg.Hq * cfg.d
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed + 31)
    w = (torch.randn(K, K, generator=gen, device=dev) / math.sqrt(K)).to(q.dtype)
    o = torch.empty_like(q)
    lse = torch.empty(cfg.B, cfg.Hq, cfg.Sq, dtype=torch.float32, device=dev)
    out = torch.empty(cfg.B, cfg.Sq, K, dtype=q.dtype, device=dev)
    ws = torch.empty(max(4, fa.fa_forward_proj_workspace_bytes(cfg.B, cfg.Sq)), dtype=torch.uint8, device=dev)
    ms_att = _time_launches(fa, lambda: fa.fa_forward_ex(q, k, v, o, lse, True, cfg.scale, variant=3), 20, 20)
    ms_two = _time_launches(fa, lambda: fa.fa_forward_proj(q, k, v, w, o, lse, out, True, cfg.scale, False, ws), 20, 20)
    ms_one = _time_launches(fa, lambda: fa.fa_forward_proj(q, k, v, w, o, lse, out, True, cfg.scale, True, ws), 20, 20)
    ms_mm = _time_launches(fa, lambda: torch.matmul(o.view(cfg.B, cfg.Sq, K), w, out=out), 20, 20)
    fl = cfg.flops() + 2.0 * cfg.B * cfg.Sq * K * K
    return {"workload": f"{cfg.name} + projection [{K} x {K}], fp16", "ms_one_launch": round(ms_one, 4),
            "ms_two_launches": round(ms_two, 4), "ms_attention_alone": round(ms_att, 4),
            "ms_projection_by_difference": round(ms_two - ms_att, 4), "ms_torch_matmul_same_projection": round(ms_mm, 4),
            "tflops_one_launch": round(fl / (ms_one * 1e-3) / 1e12, 1), "tflops_two_launches": round(fl / (ms_two * 1e-3) / 1e12, 1)}


def run_d64(fa, dev, peaks, small=False, iters=10):
    """The short non-causal vision workload with head dimension 64 (197 tokens, 12 heads, batch
    1024; batch 64 for the small debugging run), outside the timed steps.  With 99 FLOPs per byte
    of q, k, v, o the shape sits under the HBM roof, so both rates are printed."""
    cfg = synth.DEIT_B if not small else synth.PrefillConfig("DeiT-B-small", 64, 12, 12, 197, 197, d=64,
                                                             dtype="fp16", causal=False, seed=1031)
    q, k, v = synth.prefill_inputs(cfg, device=dev)
    o = torch.empty_like(q)
    lse = torch.empty(cfg.B, cfg.Hq, cfg.Sq, dtype=torch.float32, device=dev)
    for _ in range(100):   # the legs before this one are memory-bound: let the clocks settle
        fa.fa_forward(q, k, v, o, lse, cfg.causal, cfg.scale)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fa.fa_forward(q, k, v, o, lse, cfg.causal, cfg.scale)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")
    tf = cfg.flops() / (ms * 1e-3) / 1e12
    nbytes = 4.0 * q.numel() * 2 + lse.numel() * 4
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"workload": f"{cfg.name}: non-causal B={cfg.B} H={cfg.Hq} S={cfg.Sq} d=64 fp16", "kernel": "fa_fwd_d64_stream_kernel",
            "ms": round(ms, 4), "tflops": round(tf, 1), "gbs": round(gbs, 1), "algorithmic_bytes": nbytes,
            "bound": "hbm", "frac_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4),
            "frac_measured_hbm": round(gbs / peaks["hbm_gbs"], 4)}


def run_d64_long(fa, dev, peaks, small=False, iters=5):
    """Head dimension 64 on long sequences and in the decode stage, outside the timed steps: causal
    fp16 self-attention, B = 8, 32 heads, 4096 tokens (the ping-pong kernel's d = 64 instantiation),
    and the GQA decode configuration's lengths with d = 64 caches (the split-KV kernel's)."""
    cfg = (synth.PrefillConfig("d64-4K", 8, 32, 32, 4096, 4096, d=64, dtype="fp16", causal=True, seed=1060)
           if not small else
           synth.PrefillConfig("d64-small", 1, 4, 4, 1024, 1024, d=64, dtype="fp16", causal=True, seed=1061))
    q, k, v = synth.prefill_inputs(cfg, device=dev)
    o = torch.empty_like(q)
    lse = torch.empty(cfg.B, cfg.Hq, cfg.Sq, dtype=torch.float32, device=dev)
    for _ in range(10):
        fa.fa_forward(q, k, v, o, lse, cfg.causal, cfg.scale)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fa.fa_forward(q, k, v, o, lse, cfg.causal, cfg.scale)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    tf = cfg.flops() / (ms * 1e-3) / 1e12
    del q, k, v, o
    dc = (synth.DecodeConfig("C5-gqa-d64", 64, 32, 8, 32768, 1024, 32768, d=64, dtype="fp16", seed=1021)
          if not small else synth.DecodeConfig("C5-small-d64", 8, 8, 2, 4096, 512, 4096, d=64, dtype="fp16", seed=1062))
    dq, dk, dv, sl = synth.decode_inputs(dc, dev, poison=True)
    do = torch.empty_like(dq)
    dl = torch.empty(dc.B, dc.Hq, dtype=torch.float32, device=dev)
    ws = torch.empty(max(16, fa.fa_decode_workspace_bytes(dc.B, dc.Hq, dc.Hkv, dc.Smax, dc.d)), dtype=torch.uint8, device=dev)
    sld = sl.to(dev)
    for _ in range(3):
        fa.fa_decode(dq, dk, dv, do, dl, sld, dc.scale, ws)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(iters):
        fa.fa_decode(dq, dk, dv, do, dl, sld, dc.scale, ws)
    e1.record()
    torch.cuda.synchronize()
    dms = e0.elapsed_time(e1) / iters
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")
    nbytes = float(sl.sum()) * dc.Hkv * dc.d * 2 * 2
    gbs = nbytes / (dms * 1e-3) / 1e9
    return {"prefill": {"workload": f"{cfg.name}: causal B={cfg.B} H={cfg.Hq} S={cfg.Sq} d=64 fp16",
                        "kernel": "fa_fwd_pingpong_kernel, d = 64 instantiation", "ms": round(ms, 4), "tflops": round(tf, 1),
                        "frac_nominal_tensor": round(tf / NOMINAL_TENSOR_TFLOPS, 4)},
            "decode": {"workload": f"{dc.name}: B={dc.B} Hq={dc.Hq} Hkv={dc.Hkv} Skv~U[{dc.len_lo},{dc.len_hi}] d=64 fp16",
                       "kernel": "fa_decode_split_mma_kernel, d = 64 instantiation", "ms": round(dms, 4), "gbs": round(gbs, 1),
                       "kv_bytes": nbytes, "frac_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4),
                       "frac_measured_hbm": round(gbs / peaks["hbm_gbs"], 4)}}


def run_d256(fa, dev, peaks, small=False, iters=5):
    """Head dimension 256 (its own kernel), outside the timed steps: causal fp16
    self-attention, B = 2, 16 heads, 8192 tokens (512 MiB of q, k, v, o: larger than L2); one head
    of 1024 tokens for the small debugging run."""
    cfg = (synth.PrefillConfig("d256-8K", 2, 16, 16, 8192, 8192, d=256, dtype="fp16", causal=True, seed=1040)
           if not small else
           synth.PrefillConfig("d256-small", 1, 4, 4, 1024, 1024, d=256, dtype="fp16", causal=True, seed=1041))
    q, k, v = synth.prefill_inputs(cfg, device=dev)
    o = torch.empty_like(q)
    lse = torch.empty(cfg.B, cfg.Hq, cfg.Sq, dtype=torch.float32, device=dev)
    for _ in range(30):   # let the clocks settle after the memory-bound legs
        fa.fa_forward(q, k, v, o, lse, cfg.causal, cfg.scale)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fa.fa_forward(q, k, v, o, lse, cfg.causal, cfg.scale)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")
    tf = cfg.flops() / (ms * 1e-3) / 1e12
    return {"workload": f"{cfg.name}: causal B={cfg.B} H={cfg.Hq} S={cfg.Sq} d=256 fp16", "kernel": "fa_fwd_d256_kernel",
            "ms": round(ms, 4), "tflops": round(tf, 1), "bound": "tensor",
            "frac_nominal_tensor": round(tf / NOMINAL_TENSOR_TFLOPS, 4),
            "frac_measured_tensor": round(tf / peaks["bf16_tflops"], 4)}


def run_varlen(fa, dev, peaks, small=False, iters=10):
    """A packed batch of causal self-attention requests of different lengths (fa_forward_varlen),
    outside the timed steps: 32 requests with lengths uniform in [256, 8192] (8 in [64, 1024] for
    the small debugging run), Hq = Hkv = 32, bf16."""
    cfg = synth.serving_batch("serving-8x", 8, 64, 1024, seed=31, Hq=8, Hkv=8) if small else \
        synth.serving_batch("serving-32x", 32, 256, 8192, seed=31)
    q, k, v, cu_q, cu_k = synth.varlen_inputs(cfg, dev)
    cu_q, cu_k = cu_q.to(dev), cu_k.to(dev)
    o = torch.empty_like(q)
    lse = torch.empty(cfg.Hq, q.shape[0], dtype=torch.float32, device=dev)
    mq, mk = max(cfg.seqlens_q), max(cfg.seqlens_k)
    # the same keys and values behind a block table (256-key pages in a seeded random order), for
    # the packed-batch prefill over a paged cache: the two forms are timed in alternation, because
    # the box's power state moves either one by more than they differ
    page = 128 if small else 256
    kp, vp, table = synth.paged_from_packed(k, v, cfg.seqlens_k, page, seed=cfg.seed + 5)
    table = table.to(dev)
    sk = torch.tensor(cfg.seqlens_k, dtype=torch.int32, device=dev)
    o2 = torch.empty_like(q)
    lse2 = torch.empty_like(lse)
    packed = lambda: fa.fa_forward_varlen(q, k, v, o, lse, cu_q, cu_k, mq, mk, cfg.causal, cfg.scale)
    paged = lambda: fa.fa_forward_varlen_paged(q, kp, vp, table, o2, lse2, cu_q, sk, mq, mk, cfg.causal, cfg.scale)
    times = {"packed": [], "paged": []}
    for _ in range(3):
        for name, run in (("packed", packed), ("paged", paged)):
            for _ in range(3):
                run()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(iters):
                run()
            e1.record()
            torch.cuda.synchronize()
            times[name].append(e0.elapsed_time(e1) / iters)
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")
    same = bool(torch.equal(o, o2) and torch.equal(lse, lse2))
    ms = sorted(times["packed"])[1]
    ms_paged = sorted(times["paged"])[1]
    tf = cfg.flops() / (ms * 1e-3) / 1e12
    return {"workload": f"{len(cfg.seqlens_q)} causal requests, lengths {min(cfg.seqlens_q)}..{mq} "
                        f"(sum {int(q.shape[0])}), Hq=Hkv={cfg.Hq}, bf16, packed", "ms": round(ms, 4),
            "tflops": round(tf, 1), "frac_nominal_tensor": round(tf / NOMINAL_TENSOR_TFLOPS, 4),
            "frac_measured_tensor": round(tf / peaks["bf16_tflops"], 4),
            "ms_all": [round(x, 4) for x in times["packed"]],
            "paged": {"workload": f"the same requests with K and V in {page}-key pages in random order "
                                  "(fa_forward_varlen_paged)", "ms": round(ms_paged, 4),
                      "tflops": round(cfg.flops() / (ms_paged * 1e-3) / 1e12, 1),
                      "ms_all": [round(x, 4) for x in times["paged"]],
                      "paged_over_packed": round(ms_paged / ms, 4), "bit_identical_to_packed": same},
            "note": "medians of three alternating measurements of each form"}


def run_decode_append(fa, d, dev, peaks, Sq=4, iters=5):
    """The GQA decode configuration with four new tokens per sequence instead of one
    (fa_decode_append: the queries of the last four cache positions, causal among themselves),
    outside the timed steps.  The cache is read once, as in plain decode."""
    cfg = d["cfg"]
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed + 21)
    q = torch.randn(cfg.B, Sq, cfg.Hq, cfg.d, generator=gen, device=dev).to(torch.float16)
    o = torch.empty_like(q)
    lse = torch.empty(cfg.B, cfg.Hq, Sq, dtype=torch.float32, device=dev)
    ws = torch.empty(max(16, fa.fa_decode_append_workspace_bytes(cfg.B, Sq, cfg.Hq, cfg.Hkv, cfg.Smax, cfg.d)),
                     dtype=torch.uint8, device=dev)
    for _ in range(3):
        fa.fa_decode_append(q, d["k"], d["v"], o, lse, d["sl"], cfg.scale, ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fa.fa_decode_append(q, d["k"], d["v"], o, lse, d["sl"], cfg.scale, ws)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")
    gbs = d["bytes"] / (ms * 1e-3) / 1e9
    return {"workload": f"{cfg.name} with {Sq} new tokens per sequence", "ms": round(ms, 4), "gbs": round(gbs, 1),
            "kv_bytes": d["bytes"], "frac_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4),
            "frac_measured_hbm": round(gbs / peaks["hbm_gbs"], 4)}


def run_decode_fp8(fa, d, dev, peaks, iters=5):
    """The first decode configuration once more with its cache stored as FP8 e4m3 (fa_decode_fp8),
    outside the timed steps: the same keys in half the bytes.  `gbs` counts the 8-bit cache
    bytes actually read; `fp16_equivalent_gbs` is the rate the fp16 cache would need for the same time."""
    cfg = d["cfg"]
    k8, v8 = synth.fp8_cache(d["k"], d["v"], d["sl_host"], 0.25, 0.125, poison=True)
    for _ in range(3):
        fa.fa_decode_fp8(d["q"], k8, v8, d["o"], d["lse"], d["sl"], cfg.scale, 0.25, 0.125, d["ws"])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fa.fa_decode_fp8(d["q"], k8, v8, d["o"], d["lse"], d["sl"], cfg.scale, 0.25, 0.125, d["ws"])
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")
    nbytes = d["bytes"] / 2
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"workload": f"{cfg.name} with the cache as FP8 e4m3 (one factor per tensor)", "ms": round(ms, 4),
            "gbs": round(gbs, 1), "kv_bytes": nbytes, "fp16_equivalent_gbs": round(2 * gbs, 1),
            "frac_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4), "frac_measured_hbm": round(gbs / peaks["hbm_gbs"], 4)}


def run_decode_paged(fa, d, dev, peaks, page_size=256, iters=5):
    """The first decode configuration once more with its cache in pages of 256 keys handed out in
    a seeded random order (fa_decode_paged), outside the timed steps: the same cache bytes
    through a block table."""
    cfg = d["cfg"]
    kp, vp, table = synth.paged_cache(d["k"], d["v"], d["sl_host"], page_size, seed=cfg.seed + 11, spare_pages=4)
    table = table.to(dev)
    for _ in range(3):
        fa.fa_decode_paged(d["q"], kp, vp, table, d["o"], d["lse"], d["sl"], cfg.scale, d["ws"])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fa.fa_decode_paged(d["q"], kp, vp, table, d["o"], d["lse"], d["sl"], cfg.scale, d["ws"])
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    rc, where, blk = fa.fa_device_status()
    if rc != 0:
        raise SystemExit(f"device status {rc} at {where} block {blk}")
    gbs = d["bytes"] / (ms * 1e-3) / 1e9
    return {"workload": f"{cfg.name} with the cache in {page_size}-key pages in random order", "ms": round(ms, 4),
            "gbs": round(gbs, 1), "kv_bytes": d["bytes"], "pages": int(kp.shape[0]),
            "frac_nominal_hbm": round(gbs / NOMINAL_HBM_GBS, 4), "frac_measured_hbm": round(gbs / peaks["hbm_gbs"], 4)}


def run_e2e(args, fa, pc, dec, dev):
    """Same metric through the host-buffer entry point: inputs start in pinned host memory, the
    result is read back to the host, copies inside the timed region."""
    qh, kh, vh = [t.pin_memory() for t in synth.prefill_inputs(pc, device="cpu")]
    oh = torch.empty_like(qh).pin_memory()
    lh = torch.empty(pc.B, pc.Hq, pc.Sq, dtype=torch.float32).pin_memory()
    nbytes = fa.fa_forward_host_staging_bytes(pc.B, pc.Hq, pc.Hkv, pc.Sq, pc.Skv, pc.d)
    staging = torch.empty(nbytes + 1024, dtype=torch.uint8, device=dev)
    off = (-staging.data_ptr()) % 1024
    staging = staging[off:off + nbytes]
    steps = max(3, min(args.steps, 20))
    for _ in range(3):
        fa.fa_forward_host(qh, kh, vh, oh, lh, pc.causal, pc.scale, staging)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fa.fa_forward_host(qh, kh, vh, oh, lh, pc.causal, pc.scale, staging)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    h2d = qh.numel() * 2 + kh.numel() * 2 + vh.numel() * 2
    d2h = oh.numel() * 2 + lh.numel() * 4
    res = {"value": round(pc.flops() / (ms * 1e-3) / 1e12, 3), "unit": "TFLOPS", "ms": round(ms, 4),
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps,
           "entry": "fa_forward_host (pinned host q,k,v -> device, forward, o,lse -> host)"}
    # decode end to end: the KV cache is device-resident state by definition; the step's inputs
    # are the new queries and lengths, its result the attention rows
    d = dec[0]
    qh2 = d["q"].cpu().pin_memory()
    slh = d["sl_host"].pin_memory()
    oh2 = torch.empty_like(qh2).pin_memory()
    for it in range(steps + 3):
        if it == 3:
            torch.cuda.synchronize()
            e0.record()
        d["q"].copy_(qh2, non_blocking=True)
        d["sl"].copy_(slh, non_blocking=True)
        fa.fa_decode(d["q"], d["k"], d["v"], d["o"], d["lse"], d["sl"], d["cfg"].scale, d["ws"])
        oh2.copy_(d["o"], non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    ms2 = e0.elapsed_time(e1) / steps
    res["decode_mha"] = {"gbs": round(d["bytes"] / (ms2 * 1e-3) / 1e9, 1), "ms": round(ms2, 4),
                         "h2d_bytes_per_step": qh2.numel() * 2 + slh.numel() * 4,
                         "d2h_bytes_per_step": oh2.numel() * 2,
                         "note": "KV cache resident on the device (it is the decode stage's state)"}
    return res


# --------------------------------------------------------------------------- CPU oracle legs
def oracle_sample_rows(pc, n_rows, seed):
    g = torch.Generator().manual_seed(seed)
    b = torch.randint(0, pc.B, (n_rows,), generator=g)
    h = torch.randint(0, pc.Hq, (n_rows,), generator=g)
    i = torch.randint(0, pc.Sq, (n_rows,), generator=g)
    return torch.stack([b, h, i], dim=1).to(torch.int32).numpy()


def rows_flops(pc, rows) -> float:
    """Credited FLOPs of the sampled rows: 4*d per visible key (QK^T and PV)."""
    off = pc.Skv - pc.Sq
    vis = [(min(pc.Skv, int(r[2]) + off + 1) if pc.causal else pc.Skv) for r in rows]
    return 4.0 * pc.d * float(sum(vis))


def time_oracle(pc, q, k, v, n_rows, seed):
    import oracle
    rows = oracle_sample_rows(pc, n_rows, seed)
    t0 = time.perf_counter()
    oracle.attention_rows(q, k, v, pc.causal, pc.scale, rows)
    dt = time.perf_counter() - t0
    return dt, rows_flops(pc, rows)


def run_cpu_baseline(pc, budget_s=12.0):
    import oracle
    q, k, v = synth.prefill_inputs(pc, device="cpu")
    dt, fl = time_oracle(pc, q, k, v, 256, 11)           # calibration
    n = int(max(256, min(2_000_000, 256 * budget_s / max(dt, 1e-3))))
    dt, fl = time_oracle(pc, q, k, v, n, 12)
    return {"value": round(fl / dt / 1e12, 6), "unit": "TFLOPS", "cores": oracle.num_threads(),
            "kind": "oracle", "seconds": round(dt, 2),
            "sample": f"{n} uniformly sampled (b,h,i) rows of {pc.name} (row-sampled fp64 oracle, "
                      f"credited 4*d FLOPs per visible key)"}


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle as it stands, on the host cores, rank 0 only."""
    if rank != 0:
        return
    import oracle
    pc = synth.C2
    q, k, v = synth.prefill_inputs(pc, device="cpu")
    dt, _ = time_oracle(pc, q, k, v, 128, 21)
    per_step_s = min(8.0, 120.0 / max(1, args.steps + args.warmup))
    n = int(max(64, 128 * per_step_s / max(dt, 1e-3)))
    for s in range(args.warmup):
        time_oracle(pc, q, k, v, n, 100 + s)
    tot_t, tot_f = 0.0, 0.0
    for s in range(args.steps):
        dt, fl = time_oracle(pc, q, k, v, n, 200 + s)
        tot_t += dt
        tot_f += fl
    val = tot_f / tot_t / 1e12
    sample = f"{n} sampled rows of {pc.name} per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(val, 6), "unit": "TFLOPS", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(tot_t / max(1, args.steps) * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{pc.name}: causal prefill B={pc.B} Hq=Hkv={pc.Hq} Sq=Skv={pc.Sq} d=128 fp16 "
                               f"(bounded row sample per step)"},
        "cpu_baseline": {"value": round(val, 6), "unit": "TFLOPS", "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": round(val, 6), "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


def _free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn_entry(rank, world, port, fn, fn_args):
    os.environ.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world),
                       "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    fn(*fn_args)


def spawn_ranks(world: int, fn, fn_args=()):
    """Runs fn(*fn_args) in `world` processes with the environment torchrun would give them
    (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1, MASTER_PORT); returns when all have
    exited and raises if one failed."""
    import torch.multiprocessing as mp
    mp.spawn(_spawn_entry, args=(world, _free_port(), fn, fn_args), nprocs=world, join=True)


def _rank_main(argv):
    sys.argv = [sys.argv[0]] + list(argv)
    main()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="product", choices=["product", "reference"])
    ap.add_argument("--small", action="store_true", help="small shapes, for debugging only")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    args = ap.parse_args()

    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and args.impl == "product":
        # plain `python bench.py --gpus N`: start the N ranks here (under torchrun they exist already)
        spawn_ranks(args.gpus, _rank_main, (sys.argv[1:],))
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_product(args, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
