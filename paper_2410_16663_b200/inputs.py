"""Seeded synthetic inputs for the attention workloads.

This module only draws random numbers and shapes them; it contains none of the
attention arithmetic, so both the CUDA tests and the CPU oracle can be fed from
it.  Values are N(0,1) rounded to the storage type, the distribution the
benchmark configurations name; sequence lengths for decode are uniform integers
in a closed range.  Small problems are drawn on the host (identical bits on any
machine); problems too large for that are drawn on the device with torch's
seeded generator and the rows the oracle needs are copied back by the caller.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

FP16_NAN_BITS = 0x7E00  # quiet NaN in binary16, used to poison cache padding
BF16_NAN_BITS = 0x7FC0


@dataclass(frozen=True)
class PrefillConfig:
    name: str
    B: int
    Hq: int
    Hkv: int
    Sq: int
    Skv: int
    d: int = 128
    dtype: str = "fp16"
    causal: bool = True
    seed: int = 0

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    @property
    def torch_dtype(self):
        return torch.float16 if self.dtype == "fp16" else torch.bfloat16

    def flops(self) -> float:
        """Credited FLOPs: 4*B*Hq*Sq*Skv*d, halved when causal (the masked half is not credited)."""
        f = 4.0 * self.B * self.Hq * self.Sq * self.Skv * self.d
        return f / 2 if self.causal else f


@dataclass(frozen=True)
class VarlenConfig:
    """A packed batch of sequences of different lengths (query and key lengths per sequence)."""
    name: str
    Hq: int
    Hkv: int
    seqlens_q: tuple
    seqlens_k: tuple
    d: int = 128
    dtype: str = "fp16"
    causal: bool = True
    seed: int = 0

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)

    @property
    def torch_dtype(self):
        return torch.float16 if self.dtype == "fp16" else torch.bfloat16

    def flops(self) -> float:
        """Credited FLOPs: 4*Hq*d per visible (query, key) pair of every sequence."""
        pairs = 0
        for nq, nk in zip(self.seqlens_q, self.seqlens_k):
            if self.causal:
                lo = max(0, nq - nk)                 # rows that see no key
                rows = nq - lo
                pairs += rows * (nk - rows) + rows * (rows + 1) // 2
            else:
                pairs += nq * nk
        return 4.0 * self.Hq * self.d * pairs


def serving_batch(name: str, n_seqs: int, len_lo: int, len_hi: int, seed: int, Hq: int = 32, Hkv: int = 32,
                  dtype: str = "bf16") -> VarlenConfig:
    """Self-attention prefill of ``n_seqs`` requests whose lengths are uniform in [len_lo, len_hi]."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(int(seed) + 13)
    lens = tuple(int(x) for x in torch.randint(len_lo, len_hi + 1, (n_seqs,), generator=gen))
    return VarlenConfig(name, Hq, Hkv, lens, lens, dtype=dtype, causal=True, seed=seed)


@dataclass(frozen=True)
class DecodeConfig:
    name: str
    B: int
    Hq: int
    Hkv: int
    Smax: int
    len_lo: int
    len_hi: int
    d: int = 128
    dtype: str = "fp16"
    seed: int = 0

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.d)


# The five benchmark configurations (C1..C5) with fixed seeds.
C1 = PrefillConfig("C1", 1, 2, 2, 512, 512, dtype="fp16", causal=True, seed=1001)
C2 = PrefillConfig("C2", 4, 32, 32, 2048, 2048, dtype="fp16", causal=True, seed=1002)
C3 = {s: PrefillConfig(f"C3-{s // 1024}K", 1, 32, 32, s, s, dtype="bf16", causal=True,
                       seed=1003 + i)
      for i, s in enumerate((8192, 32768, 131072, 262144))}
C4 = PrefillConfig("C4", 2, 64, 8, 8192, 8192, dtype="bf16", causal=True, seed=1010)
C4_NC = PrefillConfig("C4-noncausal", 2, 64, 8, 1024, 8192, dtype="bf16", causal=False, seed=1011)
# the short non-causal vision workload (DeiT-B dimensions: 197 tokens, 12 heads of 64), batch 1024
DEIT_B = PrefillConfig("DeiT-B", 1024, 12, 12, 197, 197, d=64, dtype="fp16", causal=False, seed=1030)
C5_MHA = DecodeConfig("C5-mha", 64, 32, 32, 32768, 1024, 32768, seed=1020)
C5_GQA = DecodeConfig("C5-gqa", 64, 32, 8, 32768, 1024, 32768, seed=1021)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn(shape, dtype, gen, device) -> torch.Tensor:
    """N(0,1) in fp32 rounded to ``dtype``, drawn in slabs along dim 0/1 to bound temporaries."""
    out = torch.empty(shape, dtype=dtype, device=device)
    flat = out.view(-1)
    n = flat.numel()
    step = 1 << 26
    for s in range(0, n, step):
        e = min(n, s + step)
        flat[s:e] = torch.randn(e - s, dtype=torch.float32, device=device, generator=gen).to(dtype)
    return out


def prefill_inputs(cfg: PrefillConfig, device="cpu"):
    """q [B,Sq,Hq,d], k and v [B,Skv,Hkv,d] for a prefill configuration."""
    device = torch.device(device)
    gen = _gen(cfg.seed, device)
    dt = cfg.torch_dtype
    q = _randn((cfg.B, cfg.Sq, cfg.Hq, cfg.d), dt, gen, device)
    k = _randn((cfg.B, cfg.Skv, cfg.Hkv, cfg.d), dt, gen, device)
    v = _randn((cfg.B, cfg.Skv, cfg.Hkv, cfg.d), dt, gen, device)
    return q, k, v


def varlen_inputs(cfg: VarlenConfig, device="cpu"):
    """q [total_q,Hq,d], k and v [total_k,Hkv,d], cu_seqlens_q, cu_seqlens_k (int32 [B+1], host)."""
    device = torch.device(device)
    gen = _gen(cfg.seed, device)
    dt = cfg.torch_dtype
    cu_q = torch.zeros(len(cfg.seqlens_q) + 1, dtype=torch.int32)
    cu_k = torch.zeros(len(cfg.seqlens_k) + 1, dtype=torch.int32)
    cu_q[1:] = torch.cumsum(torch.tensor(cfg.seqlens_q, dtype=torch.int64), 0).to(torch.int32)
    cu_k[1:] = torch.cumsum(torch.tensor(cfg.seqlens_k, dtype=torch.int64), 0).to(torch.int32)
    q = _randn((int(cu_q[-1]), cfg.Hq, cfg.d), dt, gen, device)
    k = _randn((int(cu_k[-1]), cfg.Hkv, cfg.d), dt, gen, device)
    v = _randn((int(cu_k[-1]), cfg.Hkv, cfg.d), dt, gen, device)
    return q, k, v, cu_q, cu_k


def decode_seqlens(cfg: DecodeConfig) -> torch.Tensor:
    """Per-sequence cache lengths, uniform integers in [len_lo, len_hi], drawn on the host."""
    gen = _gen(cfg.seed + 7, "cpu")
    return torch.randint(cfg.len_lo, cfg.len_hi + 1, (cfg.B,), generator=gen, dtype=torch.int32)


def decode_inputs(cfg: DecodeConfig, device="cpu", poison: bool = True):
    """q [B,1,Hq,d], k_cache and v_cache [B,Smax,Hkv,d], seqlens [B] (int32, host).

    Cache rows at or beyond ``seqlens[b]`` hold NaN bit patterns when ``poison`` is set, so a
    kernel that lets padding reach its result is caught.
    """
    device = torch.device(device)
    gen = _gen(cfg.seed, device)
    dt = torch.float16 if cfg.dtype == "fp16" else torch.bfloat16
    seqlens = decode_seqlens(cfg)
    q = _randn((cfg.B, 1, cfg.Hq, cfg.d), dt, gen, device)
    k = _randn((cfg.B, cfg.Smax, cfg.Hkv, cfg.d), dt, gen, device)
    v = _randn((cfg.B, cfg.Smax, cfg.Hkv, cfg.d), dt, gen, device)
    if poison:
        bits = FP16_NAN_BITS if dt == torch.float16 else BF16_NAN_BITS
        for b in range(cfg.B):
            n = int(seqlens[b])
            if n < cfg.Smax:
                k[b, n:].view(torch.int16).fill_(bits)
                v[b, n:].view(torch.int16).fill_(bits)
    return q, k, v, seqlens


def fp8_cache(k, v, seqlens, k_scale: float, v_scale: float, poison: bool = True):
    """The caches of ``decode_inputs`` as FP8 e4m3 bit patterns (uint8) for given factors: each
    value divided by its factor and rounded to e4m3 by torch's conversion.  Rows at or beyond a
    sequence's length hold the NaN pattern 0x7f when ``poison`` is set.  (An input generator: the
    8-bit cache is what the decode stage is handed.)"""
    k8 = (k.float() / k_scale).to(torch.float8_e4m3fn).view(torch.uint8)
    v8 = (v.float() / v_scale).to(torch.float8_e4m3fn).view(torch.uint8)
    for b in range(k.shape[0]):
        n = int(seqlens[b])
        if n < k.shape[1]:
            k8[b, n:] = 0x7f if poison else 0
            v8[b, n:] = 0x7f if poison else 0
    return k8, v8


def fp8_operands(q, k, v, q_scale: float, k_scale: float, v_scale: float):
    """The tensors of ``prefill_inputs`` as FP8 e4m3 bit patterns (uint8) for given factors: each
    value divided by its tensor's factor and rounded to e4m3 by torch's conversion (an input
    generator: 8-bit operands are what ``fa_forward_fp8`` is handed)."""
    return tuple((t.float() / s).to(torch.float8_e4m3fn).view(torch.uint8) for t, s in ((q, q_scale), (k, k_scale), (v, v_scale)))


def paged_cache(k, v, seqlens, page_size: int, seed: int, spare_pages: int = 3, poison: bool = True):
    """The caches of ``decode_inputs`` laid out in pages: returns ``(k_pages, v_pages, block_table)``.

    ``k_pages``/``v_pages`` are ``[num_pages, page_size, Hkv, d]``; sequence b's keys
    ``[p*page_size, (p+1)*page_size)`` live in page ``block_table[b, p]``.  Pages are handed out in
    a seeded random order from a pool with ``spare_pages`` pages nobody uses; table entries past a
    sequence's last page are -1, and unused pages and the rows of a last page past the end of
    its sequence hold NaN bit patterns when ``poison`` is set.  Layout only: no arithmetic.
    """
    B, Smax, Hkv, d = k.shape
    max_pages = (Smax + page_size - 1) // page_size
    need = [(int(n) + page_size - 1) // page_size for n in seqlens]
    num_pages = sum(need) + spare_pages
    gen = _gen(seed, "cpu")
    order = torch.randperm(num_pages, generator=gen).tolist()
    bits = FP16_NAN_BITS if k.dtype == torch.float16 else BF16_NAN_BITS
    k_pages = torch.empty(num_pages, page_size, Hkv, d, dtype=k.dtype, device=k.device)
    v_pages = torch.empty_like(k_pages)
    if poison:
        k_pages.view(torch.int16).fill_(bits)
        v_pages.view(torch.int16).fill_(bits)
    else:
        k_pages.zero_()
        v_pages.zero_()
    table = torch.full((B, max(1, max_pages)), -1, dtype=torch.int32)
    nxt = 0
    for b in range(B):
        n = int(seqlens[b])
        for p in range(need[b]):
            page = order[nxt]
            nxt += 1
            table[b, p] = page
            lo = p * page_size
            rows = min(page_size, n - lo)
            k_pages[page, :rows] = k[b, lo:lo + rows]
            v_pages[page, :rows] = v[b, lo:lo + rows]
    return k_pages, v_pages, table


def paged_from_packed(k, v, seqlens, page_size: int, seed: int, spare_pages: int = 3, poison: bool = True):
    """The packed keys and values of ``varlen_inputs`` (``[total_k, Hkv, d]``, sequences back to back)
    laid out in pages: returns ``(k_pages, v_pages, block_table)`` as ``paged_cache`` does, pages
    handed out in a seeded random order, unused rows and pages holding NaN bit patterns when
    ``poison`` is set.  Layout only: no arithmetic."""
    need = [(int(n) + page_size - 1) // page_size for n in seqlens]
    num_pages = sum(need) + spare_pages
    order = torch.randperm(num_pages, generator=_gen(seed, "cpu")).tolist()
    bits = FP16_NAN_BITS if k.dtype == torch.float16 else BF16_NAN_BITS
    k_pages = torch.empty(num_pages, page_size, k.shape[1], k.shape[2], dtype=k.dtype, device=k.device)
    v_pages = torch.empty_like(k_pages)
    if poison:
        k_pages.view(torch.int16).fill_(bits)
        v_pages.view(torch.int16).fill_(bits)
    else:
        k_pages.zero_()
        v_pages.zero_()
    table = torch.full((len(need), max(1, max(need))), -1, dtype=torch.int32)
    nxt, base = 0, 0
    for b, n in enumerate(int(x) for x in seqlens):
        for pg in range(need[b]):
            page = order[nxt]
            nxt += 1
            table[b, pg] = page
            lo = pg * page_size
            rows = min(page_size, n - lo)
            k_pages[page, :rows] = k[base + lo:base + lo + rows]
            v_pages[page, :rows] = v[base + lo:base + lo + rows]
        base += n
    return k_pages, v_pages, table


def sample_rows(cfg: PrefillConfig, n_random: int, seed: int, pairs=None, tile: int = 128):
    """Rows (b, h, i) for row-sampled checks: the first four and the last row, both sides of
    tile boundaries near the start, middle and end, and uniformly random rows, over a few
    (b, h) pairs that include both ends of a GQA group."""
    gen = _gen(seed, "cpu")
    if pairs is None:
        g = cfg.Hq // cfg.Hkv
        pairs = {(0, 0), (0, g - 1), (cfg.B - 1, cfg.Hq - 1), (cfg.B - 1, cfg.Hq - g),
                 (0, cfg.Hq // 2)}
        pairs = sorted(pairs)
    fixed = {0, 1, 2, 3, cfg.Sq - 1}
    ntile = (cfg.Sq + tile - 1) // tile
    for t in {1, 2, ntile // 2, ntile - 1}:
        for dlt in (-1, 0):
            i = t * tile + dlt
            if 0 <= i < cfg.Sq:
                fixed.add(i)
    rows = []
    for (b, h) in pairs:
        mine = set(fixed)
        if n_random > 0:
            mine.update(int(x) for x in torch.randint(0, cfg.Sq, (n_random,), generator=gen))
        rows.extend((b, h, i) for i in sorted(mine))
    return rows
