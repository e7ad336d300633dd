"""Pins for the CPU oracle: each test fixes the oracle to something other than its own
formulas -- closed forms, a brute-force evaluation in another arithmetic, invariants of
softmax attention, or a library routine on a special case.  A dropped term, a wrong mask
inequality, a transposed operand or a wrong head mapping fails at least one of them."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2410_16663_b200 import inputs as synth

F64 = torch.float64


def rnd(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=F64) * scale


# ---------------------------------------------------------------- worked example by hand
def test_hand_example_two_keys():
    # scores (0, ln 3) -> probabilities (1/4, 3/4); V = I2 -> O = P; LSE = ln 4
    q = torch.tensor([[[[1.0, 0.0]]]], dtype=F64)                       # [1,1,1,2]
    k = torch.tensor([[[[0.0, 5.0]], [[math.log(3.0), -2.0]]]], dtype=F64)  # [1,2,1,2]
    v = torch.tensor([[[[1.0, 0.0]], [[0.0, 1.0]]]], dtype=F64)
    O, LSE = oracle.attention_full(q, k, v, causal=False, scale=1.0)
    assert torch.allclose(O[0, 0, 0], torch.tensor([0.25, 0.75], dtype=F64), atol=1e-15)
    assert abs(float(LSE[0, 0, 0]) - math.log(4.0)) < 1e-15
    # the scale multiplies the scores: scale 2 -> scores (0, ln 9) -> (0.1, 0.9)
    O, LSE = oracle.attention_full(q, k, v, causal=False, scale=2.0)
    assert torch.allclose(O[0, 0, 0], torch.tensor([0.1, 0.9], dtype=F64), atol=1e-15)
    assert abs(float(LSE[0, 0, 0]) - math.log(10.0)) < 1e-14


# ---------------------------------------------------------------- brute force, tiny inputs
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("shape", [(1, 1, 1, 1, 1, 1), (2, 4, 2, 5, 8, 3), (1, 6, 3, 8, 8, 4),
                                   (2, 2, 2, 3, 7, 2), (1, 4, 1, 1, 6, 4)])
def test_bruteforce_agrees(shape, causal):
    B, Hq, Hkv, Sq, Skv, d = shape
    q, k, v = rnd((B, Sq, Hq, d), 1), rnd((B, Skv, Hkv, d), 2), rnd((B, Skv, Hkv, d), 3)
    O, LSE = oracle.attention_full(q, k, v, causal, 0.7)
    Ob, LSEb = oracle.bruteforce(q, k, v, causal, 0.7)
    assert torch.allclose(O, Ob, atol=1e-12, rtol=0)
    assert torch.allclose(LSE, LSEb, atol=1e-12, rtol=0)


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("causal", [False, True])
def test_identical_keys_give_prefix_mean(causal):
    B, H, Sq, Skv, d = 1, 2, 6, 9, 4
    q, v = rnd((B, Sq, H, d), 4), rnd((B, Skv, H, d), 5)
    krow = rnd((1, 1, H, d), 6)
    k = krow.expand(B, Skv, H, d).contiguous()
    scale = 0.37
    O, LSE = oracle.attention_full(q, k, v, causal, scale)
    off = Skv - Sq
    for h in range(H):
        for i in range(Sq):
            n = i + off + 1 if causal else Skv
            want = v[0, :n, h].mean(dim=0)
            assert torch.allclose(O[0, i, h], want, atol=1e-14)
            s = scale * float(torch.dot(q[0, i, h], krow[0, 0, h]))
            assert abs(float(LSE[0, h, i]) - (s + math.log(n))) < 1e-13


def test_scale_zero_is_uniform_attention():
    B, H, S, d = 2, 3, 7, 5
    q, k, v = rnd((B, S, H, d), 7), rnd((B, S, H, d), 8), rnd((B, S, H, d), 9)
    O, LSE = oracle.attention_full(q, k, v, True, 0.0)
    for i in range(S):
        assert torch.allclose(O[:, i], v[:, : i + 1].mean(dim=1), atol=1e-14)
        assert torch.allclose(LSE[:, :, i], torch.full((B, H), math.log(i + 1), dtype=F64),
                              atol=1e-14)


def test_one_hot_dominant_score_returns_that_value_row():
    S, d, jstar, gap = 12, 4, 5, 40.0
    q = torch.zeros(1, 1, 1, d, dtype=F64)
    q[..., 0] = 1.0
    k = torch.zeros(1, S, 1, d, dtype=F64)
    k[0, jstar, 0, 0] = gap
    v = rnd((1, S, 1, d), 10)
    O, LSE = oracle.attention_full(q, k, v, False, 1.0)
    bound = (S - 1) * math.exp(-gap) * 2 * float(v.abs().max())
    assert float((O[0, 0, 0] - v[0, jstar, 0]).abs().max()) <= bound
    assert abs(float(LSE[0, 0, 0]) - gap) < 1e-12


def test_rows_sum_to_one_and_identity_values_read_out_probabilities():
    # V = all ones -> O = 1.  V = identity (Skv <= d) -> O_i[j] = P_ij, exactly 0 where masked.
    B, H, Sq, Skv, d = 1, 2, 5, 8, 8
    q, k = rnd((B, Sq, H, d), 11), rnd((B, Skv, H, d), 12)
    ones = torch.ones(B, Skv, H, d, dtype=F64)
    O, _ = oracle.attention_full(q, k, ones, True, 0.5)
    assert float((O - 1.0).abs().max()) < 1e-15
    eye = torch.eye(Skv, d, dtype=F64).view(1, Skv, 1, d).expand(B, Skv, H, d).contiguous()
    P, LSE = oracle.attention_full(q, k, eye, True, 0.5)
    off = Skv - Sq
    for h in range(H):
        s = 0.5 * q[0, :, h] @ k[0, :, h].T                      # [Sq, Skv]
        for i in range(Sq):
            vis = i + off + 1
            assert float(P[0, i, h, vis:].abs().max() if vis < Skv else 0.0) == 0.0
            assert float(P[0, i, h, :vis].min()) > 0.0
            e = torch.exp(s[i, :vis])
            assert torch.allclose(P[0, i, h, :vis], e / e.sum(), atol=1e-14)
            assert abs(float(LSE[0, h, i]) - math.log(float(e.sum()))) < 1e-13
    assert float((P.sum(dim=-1) - 1.0).abs().max()) < 1e-15


def test_causal_alignment_is_bottom_right_when_lengths_differ():
    # Sq < Skv: the LAST query row sees every key, the first sees Skv-Sq+1 keys.
    Sq, Skv, d = 3, 7, 7
    q, k = rnd((1, Sq, 1, d), 13), rnd((1, Skv, 1, d), 14)
    eye = torch.eye(Skv, d, dtype=F64).view(1, Skv, 1, d).contiguous()
    P, _ = oracle.attention_full(q, k, eye, True, 1.0)
    nz = (P[0, :, 0] > 0).sum(dim=-1).tolist()
    assert nz == [5, 6, 7]


def test_rows_without_visible_keys():
    # Sq > Skv under the bottom-right rule leaves the first Sq-Skv rows with nothing to see.
    Sq, Skv, d = 5, 3, 2
    q, k, v = rnd((1, Sq, 1, d), 15), rnd((1, Skv, 1, d), 16), rnd((1, Skv, 1, d), 17)
    O, LSE = oracle.attention_full(q, k, v, True, 1.0)
    assert float(O[0, :2].abs().max()) == 0.0
    assert torch.isneginf(LSE[0, 0, :2]).all()
    assert torch.isfinite(LSE[0, 0, 2:]).all()
    assert torch.allclose(O[0, 2, 0], v[0, 0, 0], atol=1e-15)


# ---------------------------------------------------------------- invariants
def test_causal_row_equals_noncausal_over_truncated_keys():
    B, H, Sq, Skv, d = 1, 2, 6, 10, 4
    q, k, v = rnd((B, Sq, H, d), 18), rnd((B, Skv, H, d), 19), rnd((B, Skv, H, d), 20)
    O, LSE = oracle.attention_full(q, k, v, True, 0.9)
    for i in range(Sq):
        n = i + (Skv - Sq) + 1
        Oi, Li = oracle.attention_full(q[:, i:i + 1].contiguous(), k[:, :n].contiguous(),
                                       v[:, :n].contiguous(), False, 0.9)
        assert torch.allclose(O[:, i], Oi[:, 0], atol=1e-14)
        assert torch.allclose(LSE[:, :, i], Li[:, :, 0], atol=1e-14)


def test_joint_key_value_permutation_changes_nothing():
    B, H, Sq, Skv, d = 1, 2, 4, 9, 3
    q, k, v = rnd((B, Sq, H, d), 21), rnd((B, Skv, H, d), 22), rnd((B, Skv, H, d), 23)
    perm = torch.randperm(Skv, generator=torch.Generator().manual_seed(5))
    O1, L1 = oracle.attention_full(q, k, v, False, 1.1)
    O2, L2 = oracle.attention_full(q, k[:, perm].contiguous(), v[:, perm].contiguous(), False, 1.1)
    assert torch.allclose(O1, O2, atol=1e-13)
    assert torch.allclose(L1, L2, atol=1e-13)


def test_gqa_equals_mha_with_repeated_kv_heads():
    B, Hq, Hkv, Sq, Skv, d = 2, 6, 2, 5, 5, 4
    q, k, v = rnd((B, Sq, Hq, d), 24), rnd((B, Skv, Hkv, d), 25), rnd((B, Skv, Hkv, d), 26)
    O1, L1 = oracle.attention_full(q, k, v, True, 0.6)
    g = Hq // Hkv
    kr, vr = k.repeat_interleave(g, dim=2), v.repeat_interleave(g, dim=2)
    O2, L2 = oracle.attention_full(q, kr, vr, True, 0.6)
    assert torch.equal(O1, O2) and torch.equal(L1, L2)
    # and the head mapping is consecutive grouping: query head 3 (g = 3) reads kv head 1
    Oh, _ = oracle.attention_full(q[:, :, 3:4].contiguous(), k[:, :, 1:2].contiguous(),
                                  v[:, :, 1:2].contiguous(), True, 0.6)
    assert torch.equal(O1[:, :, 3], Oh[:, :, 0])


def test_split_merge_identity():
    # attention over KV equals the LSE-weighted merge of attention over any partition of KV
    B, H, Skv, d = 1, 2, 23, 4
    q, k, v = rnd((B, 1, H, d), 27), rnd((B, Skv, H, d), 28), rnd((B, Skv, H, d), 29)
    O, LSE = oracle.attention_full(q, k, v, False, 0.8)
    cuts = [0, 5, 6, 17, 23]
    parts = [oracle.attention_full(q, k[:, a:b].contiguous(), v[:, a:b].contiguous(), False, 0.8)
             for a, b in zip(cuts[:-1], cuts[1:])]
    Ls = torch.stack([p[1][:, :, 0] for p in parts])            # [c,B,H]
    Os = torch.stack([p[0][:, 0] for p in parts])               # [c,B,H,d]
    M = Ls.max(dim=0).values
    w = torch.exp(Ls - M)
    merged = (w.unsqueeze(-1) * Os).sum(0) / w.sum(0).unsqueeze(-1)
    assert torch.allclose(merged, O[:, 0], atol=1e-14)
    assert torch.allclose(M + torch.log(w.sum(0)), LSE[:, :, 0], atol=1e-14)


def test_large_scores_are_stable_and_shift_consistent():
    B, H, S, d = 1, 1, 6, 3
    q, k, v = rnd((B, S, H, d), 30), rnd((B, S, H, d), 31), rnd((B, S, H, d), 32)
    # append a constant coordinate: scores shift by c for every key
    for c in (600.0, -600.0):
        q2 = torch.cat([q, torch.ones(B, S, H, 1, dtype=F64)], dim=-1)
        k2 = torch.cat([k, torch.full((B, S, H, 1), c, dtype=F64)], dim=-1)
        v2 = torch.cat([v, torch.zeros(B, S, H, 1, dtype=F64)], dim=-1)
        O1, L1 = oracle.attention_full(q, k, v, True, 1.0)
        O2, L2 = oracle.attention_full(q2, k2, v2, True, 1.0)
        assert torch.isfinite(O2).all() and torch.isfinite(L2).all()
        assert torch.allclose(O2[..., :d], O1, atol=1e-12)
        assert torch.allclose(L2, L1 + c, atol=1e-10)


# ---------------------------------------------------------------- library special case
@pytest.mark.parametrize("causal", [False, True])
def test_against_torch_softmax_matmul(causal):
    B, H, Sq, Skv, d = 2, 3, 9, 13, 16
    q, k, v = rnd((B, Sq, H, d), 33), rnd((B, Skv, H, d), 34), rnd((B, Skv, H, d), 35)
    scale = 1 / math.sqrt(d)
    s = torch.einsum("bihd,bjhd->bhij", q, k) * scale
    if causal:
        i = torch.arange(Sq).view(-1, 1)
        j = torch.arange(Skv).view(1, -1)
        s = s.masked_fill(j > i + (Skv - Sq), float("-inf"))
    want_o = torch.einsum("bhij,bjhd->bihd", torch.softmax(s, dim=-1), v)
    want_l = torch.logsumexp(s, dim=-1)
    O, LSE = oracle.attention_full(q, k, v, causal, scale)
    assert torch.allclose(O, want_o, atol=1e-13)
    assert torch.allclose(LSE, want_l, atol=1e-13)


# ---------------------------------------------------------------- storage types
@pytest.mark.parametrize("dt", [torch.float16, torch.bfloat16])
def test_sixteen_bit_inputs_are_widened_exactly(dt):
    # one key: O is that key's value row exactly, so every finite bit pattern can be read back
    bits = torch.arange(0, 65536, dtype=torch.int32).to(torch.int16)
    vals = bits.view(dt)
    finite = torch.isfinite(vals.float())
    vals = vals[finite]
    n = vals.numel()
    d = 8
    pad = (-n) % d
    vals = torch.cat([vals, torch.zeros(pad, dtype=dt)])
    v = vals.view(-1, 1, 1, d)                                   # batch of single-key problems
    Bn = v.shape[0]
    q = torch.zeros(Bn, 1, 1, d, dtype=dt)
    k = torch.zeros(Bn, 1, 1, d, dtype=dt)
    O, LSE = oracle.attention_full(q, k, v, False, 1.0)
    assert torch.equal(O.view(-1), v.view(-1).to(F64))
    assert float(LSE.abs().max()) == 0.0


def test_sixteen_bit_inputs_match_widened_copy():
    g = torch.Generator().manual_seed(36)
    for dt in (torch.float16, torch.bfloat16):
        q = torch.randn(1, 5, 2, 8, generator=g).to(dt)
        k = torch.randn(1, 7, 2, 8, generator=g).to(dt)
        v = torch.randn(1, 7, 2, 8, generator=g).to(dt)
        O1, L1 = oracle.attention_full(q, k, v, True, 0.3)
        O2, L2 = oracle.attention_full(q.double(), k.double(), v.double(), True, 0.3)
        assert torch.equal(O1, O2) and torch.equal(L1, L2)


# ---------------------------------------------------------------- the oracle's other entry points
def test_row_mode_equals_full_mode_and_handles_strides():
    B, Hq, Hkv, Sq, Skv, d = 2, 4, 2, 6, 9, 4
    q, k, v = rnd((B, Sq, Hq, d), 37), rnd((B, Skv, Hkv, d), 38), rnd((B, Skv, Hkv, d), 39)
    O, LSE = oracle.attention_full(q, k, v, True, 0.5)
    rows = [(b, h, i) for b in range(B) for h in range(Hq) for i in range(Sq)]
    Or, Lr = oracle.attention_rows(q, k, v, True, 0.5, rows)
    for n, (b, h, i) in enumerate(rows):
        assert torch.equal(Or[n], O[b, i, h]) and Lr[n] == LSE[b, h, i]
    # [B,H,S,d] storage viewed as [B,S,H,d] (non-contiguous) gives the same answer
    qt = q.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    kt = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vt = v.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    O2, L2 = oracle.attention_full(qt, kt, vt, True, 0.5)
    assert torch.equal(O, O2) and torch.equal(LSE, L2)


def test_decode_equals_attention_over_the_valid_prefix_and_ignores_padding():
    B, Hq, Hkv, Smax, d = 3, 4, 2, 11, 4
    q, k, v = rnd((B, 1, Hq, d), 40), rnd((B, Smax, Hkv, d), 41), rnd((B, Smax, Hkv, d), 42)
    seqlens = [11, 4, 0]
    kp, vp = k.clone(), v.clone()
    for b, n in enumerate(seqlens):
        kp[b, n:] = float("nan")
        vp[b, n:] = float("nan")
    O, LSE = oracle.decode(q, kp, vp, seqlens, 0.4)
    for b, n in enumerate(seqlens):
        if n == 0:
            assert float(O[b].abs().max()) == 0.0 and torch.isneginf(LSE[b]).all()
            continue
        Ob, Lb = oracle.attention_full(q[b:b + 1], k[b:b + 1, :n].contiguous(),
                                       v[b:b + 1, :n].contiguous(), False, 0.4)
        assert torch.equal(O[b], Ob[0, 0]) and torch.equal(LSE[b], Lb[0, :, 0])


def test_varlen_attention_is_attention_of_each_sequence_alone():
    # a packed batch with equal lengths is the batched problem; with unequal lengths every
    # sequence must come out as if it were alone (checked against the extended-precision brute
    # force on its own slice), whatever its neighbours hold
    B, S, Hq, Hkv, d = 3, 7, 4, 2, 8
    q, k, v = rnd((B, S, Hq, d), 60), rnd((B, S, Hkv, d), 61), rnd((B, S, Hkv, d), 62)
    cu = [0, 7, 14, 21]
    for causal in (False, True):
        O_ref, L_ref = oracle.attention_full(q, k, v, causal, 0.3)
        O, LSE = oracle.attention_varlen(q.reshape(B * S, Hq, d), k.reshape(B * S, Hkv, d), v.reshape(B * S, Hkv, d),
                                         cu, cu, causal, 0.3)
        assert torch.equal(O.reshape(B, S, Hq, d), O_ref)
        assert torch.equal(LSE.reshape(Hq, B, S).permute(1, 0, 2), L_ref)
    lens_q, lens_k = [5, 0, 3, 2, 6], [9, 4, 3, 0, 2]        # chunked, no queries, square, no keys, more queries than keys
    cq, ck = np.concatenate([[0], np.cumsum(lens_q)]), np.concatenate([[0], np.cumsum(lens_k)])
    qp, kp, vp = rnd((int(cq[-1]), Hq, d), 63), rnd((int(ck[-1]), Hkv, d), 64), rnd((int(ck[-1]), Hkv, d), 65)
    for causal in (False, True):
        O, LSE = oracle.attention_varlen(qp, kp, vp, cq, ck, causal, 0.3)
        for b, (nq, nk) in enumerate(zip(lens_q, lens_k)):
            rows = slice(int(cq[b]), int(cq[b + 1]))
            if nq == 0:
                continue
            if nk == 0:
                assert float(O[rows].abs().max()) == 0.0 and torch.isneginf(LSE[:, rows]).all()
                continue
            hidden = max(0, nq - nk) if causal else 0      # rows above the bottom-right diagonal's first column
            if hidden:
                top = slice(int(cq[b]), int(cq[b]) + hidden)
                assert float(O[top].abs().max()) == 0.0 and torch.isneginf(LSE[:, top]).all()
            vis = slice(int(cq[b]) + hidden, int(cq[b + 1]))
            Ob, Lb = oracle.bruteforce(qp[vis].unsqueeze(0), kp[int(ck[b]):int(ck[b + 1])].unsqueeze(0),
                                       vp[int(ck[b]):int(ck[b + 1])].unsqueeze(0), causal, 0.3)
            assert float((O[vis] - Ob[0]).abs().max()) < 1e-12
            assert float((LSE[:, vis] - Lb[0]).abs().max()) < 1e-12
    with pytest.raises(ValueError):
        oracle.attention_varlen(qp, kp, vp, cq[:-1], ck[:-1], False, 0.3)   # sums do not reach the end


def test_decode_append_is_one_decode_per_new_token_on_the_cache_as_it_stood_then():
    # query t of the last Sq positions must come out as plain decode over the cache truncated
    # to what existed when that token was appended; with Sq = 1 it is decode itself; a sequence
    # shorter than Sq leaves its first queries without keys
    B, Sq, Hq, Hkv, Smax, d = 3, 4, 4, 2, 12, 4
    q, k, v = rnd((B, Sq, Hq, d), 80), rnd((B, Smax, Hkv, d), 81), rnd((B, Smax, Hkv, d), 82)
    seqlens = [12, 5, 2]
    kp, vp = k.clone(), v.clone()
    for b, n in enumerate(seqlens):
        kp[b, n:] = float("nan")
        vp[b, n:] = float("nan")
    O, LSE = oracle.decode_append(q, kp, vp, seqlens, 0.4)
    for t in range(Sq):
        then = [max(0, n - (Sq - 1 - t)) for n in seqlens]
        Ot, Lt = oracle.decode(q[:, t:t + 1].contiguous(), k, v, then, 0.4)
        assert torch.equal(O[:, t], Ot) and torch.equal(LSE[:, :, t], Lt)
    assert float(O[2, :2].abs().max()) == 0.0 and torch.isneginf(LSE[2, :, :2]).all()   # 2 keys, 4 queries
    O1, L1 = oracle.decode_append(q[:, 3:4].contiguous(), kp, vp, seqlens, 0.4)
    Od, Ld = oracle.decode(q[:, 3:4].contiguous(), kp, vp, seqlens, 0.4)
    assert torch.equal(O1[:, 0], Od) and torch.equal(L1[:, :, 0], Ld)


def test_e4m3_values_and_fp8_decode():
    # the format's landmarks: 0x38 = 1, 0x40 = 2, 0x01 = 2^-9 (smallest subnormal), 0x08 = 2^-6
    # (smallest normal), 0x7e = 448 (largest), 0x7f / 0xff = NaN, sign bit; and all 256 patterns
    # against torch's own conversion (a library routine the decoder does not use)
    val = oracle.e4m3_to_float64(torch.tensor([0x38, 0x40, 0x01, 0x08, 0x7e, 0xb8, 0x00, 0x80, 0x3c], dtype=torch.uint8))
    assert val.tolist() == [1.0, 2.0, 2.0 ** -9, 2.0 ** -6, 448.0, -1.0, 0.0, 0.0, 1.5]
    assert torch.isnan(oracle.e4m3_to_float64(torch.tensor([0x7f, 0xff], dtype=torch.uint8))).all()
    bits = torch.arange(256, dtype=torch.uint8)
    mine, ref = oracle.e4m3_to_float64(bits), bits.view(torch.float8_e4m3fn).to(torch.float64)
    assert ((mine == ref) | (torch.isnan(mine) & torch.isnan(ref))).all()
    # fp8 decode = decode on the widened, scaled cache; NaN patterns past a sequence's end are ignored;
    # doubling v_scale doubles O and leaves LSE, and k_scale is interchangeable with the softmax scale
    B, Hq, Hkv, Smax, d = 2, 4, 2, 9, 8
    q = rnd((B, 1, Hq, d), 70)
    gen = torch.Generator().manual_seed(71)
    k8 = torch.randint(0, 0x78, (B, Smax, Hkv, d), generator=gen, dtype=torch.uint8) | (torch.randint(0, 2, (B, Smax, Hkv, d), generator=gen, dtype=torch.uint8) << 7)
    v8 = torch.randint(0, 0x78, (B, Smax, Hkv, d), generator=gen, dtype=torch.uint8)
    seqlens = [9, 4]
    k8[1, 4:] = 0x7f
    v8[1, 4:] = 0xff
    O, LSE = oracle.decode_fp8(q, k8, v8, seqlens, 0.3, 0.5, 0.25)
    kf = k8.view(torch.float8_e4m3fn).to(torch.float64) * 0.5
    vf = v8.view(torch.float8_e4m3fn).to(torch.float64) * 0.25
    for b, n in enumerate(seqlens):
        Ob, Lb = oracle.attention_full(q[b:b + 1], kf[b:b + 1, :n].contiguous(), vf[b:b + 1, :n].contiguous(), False, 0.3)
        assert torch.equal(O[b], Ob[0, 0]) and torch.equal(LSE[b], Lb[0, :, 0])
    O2, L2 = oracle.decode_fp8(q, k8, v8, seqlens, 0.3, 0.5, 0.5)
    assert torch.allclose(O2, 2 * O, rtol=1e-14, atol=0) and torch.equal(L2, LSE)
    O3, L3 = oracle.decode_fp8(q, k8, v8, seqlens, 0.15, 1.0, 0.25)
    assert torch.allclose(O3, O, rtol=1e-12, atol=1e-14) and torch.allclose(L3, LSE, rtol=1e-12, atol=1e-14)


def test_projection_after_attention():
    # hand example: scores 0 and ln 3 give P = (1/4, 3/4); V = 4 I gives O = (1, 3); W = [[1, 2], [3, 4]]
    # gives out = (1*1 + 3*3, 1*2 + 3*4) = (10, 14)
    q = torch.tensor([[[[1.0, 0.0]]]], dtype=torch.float64)
    k = torch.tensor([[[[0.0, 0.0]], [[math.log(3.0), 0.0]]]], dtype=torch.float64)
    v = torch.tensor([[[[4.0, 0.0]], [[0.0, 4.0]]]], dtype=torch.float64)
    w = torch.tensor([[1.0, 2.0], [3.0, 4.0]], dtype=torch.float64)
    O, LSE, out = oracle.attention_proj(q, k, v, w, False, 1.0)
    assert torch.allclose(O[0, 0, 0], torch.tensor([1.0, 3.0], dtype=torch.float64), atol=1e-14)
    assert torch.allclose(out[0, 0], torch.tensor([10.0, 14.0], dtype=torch.float64), atol=1e-13)
    # W = I returns O (rounded to the operands' type: the projection reads the 16-bit output), in the
    # order (head, d) of a row; a permutation matrix picks columns; linear in W
    B, Sq, Skv, Hq, Hkv, d = 2, 5, 9, 4, 2, 8
    qh, kh, vh = rnd((B, Sq, Hq, d), 81).half(), rnd((B, Skv, Hkv, d), 82).half(), rnd((B, Skv, Hkv, d), 83).half()
    K = Hq * d
    O, LSE, out = oracle.attention_proj(qh, kh, vh, torch.eye(K, dtype=torch.float64), True, 0.3)
    O2, L2 = oracle.attention_full(qh, kh, vh, True, 0.3)
    assert torch.equal(O, O2) and torch.equal(LSE, L2)
    assert torch.equal(out, O.half().double().reshape(B, Sq, K))
    perm = torch.randperm(K, generator=torch.Generator().manual_seed(5))
    P = torch.zeros(K, K, dtype=torch.float64); P[perm, torch.arange(K)] = 1.0       # out[:, n] = O[:, perm[n]]
    assert torch.equal(oracle.attention_proj(qh, kh, vh, P, True, 0.3)[2], O.half().double().reshape(B, Sq, K)[..., perm])
    w1, w2 = rnd((K, 6), 84).double(), rnd((K, 6), 85).double()
    o1 = oracle.attention_proj(qh, kh, vh, w1, False, 0.3)[2]
    o2 = oracle.attention_proj(qh, kh, vh, w2, False, 0.3)[2]
    o12 = oracle.attention_proj(qh, kh, vh, w1 + 2 * w2, False, 0.3)[2]
    assert torch.allclose(o12, o1 + 2 * o2, rtol=1e-12, atol=1e-12)
    # float64 operands are not rounded in between
    O64, _, out64 = oracle.attention_proj(qh.double(), kh.double(), vh.double(), w1, False, 0.3)
    assert torch.allclose(out64, O64.reshape(B, Sq, K) @ w1, rtol=1e-13, atol=1e-13)


def test_fp8_attention_is_attention_on_the_widened_operands():
    # 8-bit operands: the definition on Q = q_scale * value(bits) etc.  Pins: torch's own widening and
    # softmax.matmul in float64 (library routines the oracle does not use); the factors of q and k
    # are interchangeable with the softmax scale; v's factor scales O and leaves LSE; a value
    # tensor whose bit patterns all read 1.0 (0x38) gives O = v_scale exactly; rows mode = full mode
    B, Sq, Skv, Hq, Hkv, d = 2, 5, 7, 4, 2, 8
    gen = torch.Generator().manual_seed(91)
    def bits(shape):
        return torch.randint(0, 0x78, shape, generator=gen, dtype=torch.uint8) | (torch.randint(0, 2, shape, generator=gen, dtype=torch.uint8) << 7)
    q8, k8, v8 = bits((B, Sq, Hq, d)), bits((B, Skv, Hkv, d)), bits((B, Skv, Hkv, d))
    for causal in (False, True):
        O, LSE = oracle.attention_fp8(q8, k8, v8, causal, 0.02, 0.5, 0.25, 0.125)
        qf = q8.view(torch.float8_e4m3fn).to(torch.float64) * 0.5
        kf = (k8.view(torch.float8_e4m3fn).to(torch.float64) * 0.25).repeat_interleave(Hq // Hkv, dim=2)
        vf = (v8.view(torch.float8_e4m3fn).to(torch.float64) * 0.125).repeat_interleave(Hq // Hkv, dim=2)
        s = torch.einsum("bihd,bjhd->bhij", qf, kf) * 0.02
        if causal:
            vis = torch.ones(Sq, Skv, dtype=torch.bool).tril(Skv - Sq)
            s = s.masked_fill(~vis, float("-inf"))
        want = torch.einsum("bhij,bjhd->bihd", torch.softmax(s, -1), vf)
        assert torch.allclose(O, want, rtol=1e-12, atol=1e-13)
        assert torch.allclose(LSE, torch.logsumexp(s, -1), rtol=1e-12, atol=1e-13)
        O2, L2 = oracle.attention_fp8(q8, k8, v8, causal, 0.02 * 0.5 * 0.25, 1.0, 1.0, 0.25)
        assert torch.allclose(O2, 2 * O, rtol=1e-12, atol=1e-13) and torch.allclose(L2, LSE, rtol=1e-12, atol=1e-13)
        ones = torch.full_like(v8, 0x38)
        O3, _ = oracle.attention_fp8(q8, k8, ones, causal, 0.02, 0.5, 0.25, 0.125)
        assert torch.allclose(O3, torch.full_like(O3, 0.125), rtol=1e-14, atol=0)
        rows = [(0, 0, 0), (1, 3, 4), (0, 2, 2)]
        Or, Lr = oracle.attention_fp8(q8, k8, v8, causal, 0.02, 0.5, 0.25, 0.125, rows=rows)
        for n, (b, h, i) in enumerate(rows):
            assert torch.equal(Or[n], O[b, i, h]) and Lr[n] == LSE[b, h, i]
        Oa, _ = oracle.attention_fp8(q8, k8, v8, causal, 0.02, 0.5, 0.25, 0.125, abs_v=True)
        assert torch.allclose(Oa, torch.einsum("bhij,bjhd->bihd", torch.softmax(s, -1), vf.abs()), rtol=1e-12, atol=1e-13)


def test_paged_packed_batch_equals_the_packed_batch_on_the_same_keys():
    # pools filled by hand, page by page in a scrambled order; NaN wherever no key lives
    Hq, Hkv, d, ps = 4, 2, 4, 4
    lens_q, lens_k = [3, 2, 5], [9, 2, 5]
    cq, ck = np.concatenate([[0], np.cumsum(lens_q)]), np.concatenate([[0], np.cumsum(lens_k)])
    q, k, v = rnd((int(cq[-1]), Hq, d), 90), rnd((int(ck[-1]), Hkv, d), 91), rnd((int(ck[-1]), Hkv, d), 92)
    order = [4, 0, 6, 2, 5, 1, 3]
    kp = torch.full((7, ps, Hkv, d), float("nan"), dtype=k.dtype)
    vp = torch.full((7, ps, Hkv, d), float("nan"), dtype=v.dtype)
    table = -np.ones((3, 3), dtype=np.int32)
    nxt = 0
    for b, n in enumerate(lens_k):
        for p_ in range((n + ps - 1) // ps):
            slot = order[nxt]; nxt += 1
            table[b, p_] = slot
            for r in range(min(ps, n - p_ * ps)):
                kp[slot, r] = k[int(ck[b]) + p_ * ps + r]
                vp[slot, r] = v[int(ck[b]) + p_ * ps + r]
    for causal in (False, True):
        O1, L1 = oracle.attention_varlen(q, k, v, cq, ck, causal, 0.3)
        O2, L2 = oracle.attention_varlen_paged(q, kp, vp, table, cq, lens_k, causal, 0.3)
        assert torch.equal(O1, O2) and torch.equal(L1, L2)


def test_paged_decode_equals_decode_on_the_same_keys_wherever_the_pages_lie():
    # the paged form only changes where a key is stored: build the pools by hand (page p of
    # sequence b at a chosen pool slot), compare with decode on the contiguous caches, then move
    # the pages around (with the table) and check that nothing changes; tiny page size so that
    # several pages and a ragged last page occur
    B, Hq, Hkv, Smax, d, ps = 3, 4, 2, 11, 4, 4
    q, k, v = rnd((B, 1, Hq, d), 50), rnd((B, Smax, Hkv, d), 51), rnd((B, Smax, Hkv, d), 52)
    seqlens = [11, 4, 0]
    O_ref, L_ref = oracle.decode(q, k, v, seqlens, 0.4)
    for order in ([5, 2, 7, 0, 3, 1, 6, 4], [0, 1, 2, 3, 4, 5, 6, 7]):
        kp = torch.full((8, ps, Hkv, d), float("nan"), dtype=k.dtype)
        vp = torch.full((8, ps, Hkv, d), float("nan"), dtype=v.dtype)
        table = -np.ones((B, 3), dtype=np.int32)
        nxt = 0
        for b, n in enumerate(seqlens):
            for p in range((n + ps - 1) // ps):
                slot = order[nxt]; nxt += 1
                table[b, p] = slot
                for r in range(min(ps, n - p * ps)):
                    kp[slot, r] = k[b, p * ps + r]
                    vp[slot, r] = v[b, p * ps + r]
        O, LSE = oracle.decode_paged(q, kp, vp, table, seqlens, 0.4)
        assert torch.equal(O, O_ref) and torch.equal(LSE, L_ref)
    # a table entry outside the pool is an error, not a silent read
    table[0, 1] = 8
    with pytest.raises(ValueError):
        oracle.decode_paged(q, kp, vp, table, seqlens, 0.4)


def test_paged_cache_layout_of_the_input_generator_round_trips():
    # the seeded generator's page layout, read back position by position, is the contiguous cache
    cfg = synth.DecodeConfig("t", 4, 4, 2, 700, 1, 700, seed=77)
    q, k, v, sl = synth.decode_inputs(cfg, "cpu", poison=True)
    sl[1] = 0
    sl[2] = 512            # ends exactly on a page boundary
    kp, vp, table = synth.paged_cache(k, v, sl, 256, seed=3, spare_pages=2)
    assert kp.shape[0] == sum((int(n) + 255) // 256 for n in sl) + 2
    used = table[table >= 0]
    assert len(set(used.tolist())) == used.numel()          # no page handed out twice
    for b in range(cfg.B):
        for j in (0, 1, 255, 256, 257, int(sl[b]) - 1):
            if 0 <= j < int(sl[b]):
                page = int(table[b, j // 256])
                assert torch.equal(kp[page, j % 256], k[b, j]) and torch.equal(vp[page, j % 256], v[b, j])
    O1, L1 = oracle.decode(q, k, v, sl, cfg.scale)
    O2, L2 = oracle.decode_paged(q, kp, vp, table, sl, cfg.scale)
    assert torch.equal(O1, O2) and torch.equal(L1, L2)


def test_argument_errors_are_reported():
    q, k, v = rnd((1, 2, 3, 4), 43), rnd((1, 2, 2, 4), 44), rnd((1, 2, 2, 4), 45)
    with pytest.raises(RuntimeError):
        oracle.attention_full(q, k, v, False, 1.0)              # Hq % Hkv != 0
    with pytest.raises(RuntimeError):
        oracle.attention_rows(q[:, :, :2].contiguous(), k, v, False, 1.0, [(0, 0, 9)])
