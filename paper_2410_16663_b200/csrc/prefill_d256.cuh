// Attention forward for head dimension 256.  One CTA of six warps per (batch, head, 128-row query
// tile): four softmax warps (one thread per query row), a warp whose first lane loads K and
// issues the score MMAs, and a warp whose first lane loads V and issues the P V MMAs.  Tiles are
// 128 rows x 256 elements = four 64-column swizzled boxes (64 KiB).  Shared memory: Q, three
// slots of half a K tile along d (128 keys x 128, two boxes, 32 KiB) and two slots of half a V
// tile along the keys (64 keys x 256, 32 KiB): 224 KiB in all, one CTA per SM.  Tensor memory:
// two score buffers, columns [0,128) and [384,512), and O in [128,384).
//
// S = Q K^T of kv tile t goes into score buffer t & 1 as soon as P V of tile t - 2 has left it,
// i.e. while the softmax of tile t - 1 is at work, in two runs of eight k-steps, one per half of
// d; the K half-slot a run has read is refilled (with the half three further on) as soon as the
// run has completed, so every K load has about a step to arrive.  P goes back packed over the
// first 64 columns of its score buffer; O += P V is an N = 256 MMA per 16 keys with V as the
// N-major operand (its four boxes one leading-dimension stride apart), issued in two groups of
// four, one per half of V, and a V half-slot is refilled as soon as its group has completed.
// Online softmax as in Appendix A (rowmax / rowsum), with a reference max that moves only when
// the row max outgrew it by 2^8, and O rescaled only on steps where some row of the warp moved it.
#pragma once

#include "prefill_simple.cuh"

namespace fa {

constexpr int kD256TileBytes = 4 * kHalfBytes;              // 128 rows x 256 16-bit elements
constexpr int kD256VHalfBytes = kD256TileBytes / 2;         // 64 keys x 256: four boxes of 64 x 64
constexpr int kD256VBoxBytes = kD256VHalfBytes / 4;         // one of them (the MMA's LBO)
constexpr int kD256KHalfBytes = kD256TileBytes / 2;         // 128 keys x 128 of d: two boxes of 128 x 64
constexpr int kD256Smem = 1024 + kD256TileBytes + 3 * kD256KHalfBytes + 2 * kD256VHalfBytes;
constexpr int kD256Threads = 192;   // four softmax warps, the score-MMA warp, the P V warp

__device__ __forceinline__ void d256_load_tile(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int h, int s0,
                                               int b) {
#pragma unroll
    for (int c = 0; c < 4; ++c) tma_load_4d(dst + c * kHalfBytes, tm, bar, 64 * c, h, s0, b);
}

// Half of a K tile along d (two of its four boxes) into a half-slot: half 0 = head dimensions 0..127
__device__ __forceinline__ void d256_load_k_half(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int half, int h,
                                                 int s0, int b) {
    mbar_expect_tx(bar, kD256KHalfBytes);
#pragma unroll
    for (int c = 0; c < 2; ++c) tma_load_4d(dst + c * kHalfBytes, tm, bar, 64 * (2 * half + c), h, s0, b);
}

// tm_vh: the map over V with boxes of 64 keys
__device__ __forceinline__ void d256_load_v_half(uint32_t dst, const CUtensorMap* tm_vh, uint32_t bar, int h, int s0,
                                                 int b) {
    mbar_expect_tx(bar, kD256VHalfBytes);
#pragma unroll
    for (int c = 0; c < 4; ++c) tma_load_4d(dst + c * kD256VBoxBytes, tm_vh, bar, 64 * c, h, s0, b);
}

template <typename T>
__global__ void __launch_bounds__(kD256Threads, 1)
fa_fwd_d256_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_vh, const FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + kD256TileBytes;       // three half-tile slots (128 keys x 128 of d each)
    const uint32_t sV = sK + 3 * kD256KHalfBytes;   // two half-tile slots (64 keys x 256 each)
    __shared__ __align__(8) uint64_t bars[14];
    __shared__ uint32_t tmem_holder;
    __shared__ volatile uint32_t abort_flag;

    const uint32_t bar_q = smem_u32(&bars[0]);
    const uint32_t bar_kh = smem_u32(&bars[1]);    // +8 per K half-slot (3): half a K tile along d landed
    const uint32_t bar_vh = smem_u32(&bars[4]);    // +8 per V half-slot (2): half a V tile along the keys landed
    const uint32_t bar_s = smem_u32(&bars[6]);     // +8 per score buffer (2): S landed
    const uint32_t bar_p = smem_u32(&bars[8]);     // +8 per score buffer (2): P written, O rescaled (128 arrivals)
    const uint32_t bar_g = smem_u32(&bars[10]);    // first group of a tile's P V completed
    const uint32_t bar_o = smem_u32(&bars[11]);    // a tile's P V completed
    const uint32_t bar_sa = smem_u32(&bars[12]);   // the score MMAs over the first half of d completed

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int qt = p.n_qtiles - 1 - blockIdx.x;  // long (late) tiles first
    const int h = blockIdx.y;
    const int b = blockIdx.z;
    const int hk = h / (p.Hq / p.Hkv);
    const int q0 = qt * kTile;
    const int off = p.Skv - p.Sq;
    const int n_tiles = kv_tiles_for(q0, kTile, p.Sq, p.Skv, p.causal);

    if (tid == 128) {
        for (int i = 0; i < 13; ++i) mbar_init(smem_u32(&bars[i]), (i == 8 || i == 9) ? 128 : 1);
        abort_flag = 0;
        fence_mbar_init();
        if (n_tiles > 0) {
            mbar_expect_tx(bar_q, kD256TileBytes);
            d256_load_tile(sQ, &tm_q, bar_q, h, q0, b);
            for (int kh = 0; kh < 3 && kh < 2 * n_tiles; ++kh)
                d256_load_k_half(sK + kh * kD256KHalfBytes, &tm_k, bar_kh + 8 * kh, kh & 1, hk, (kh >> 1) * kTile, b);
            for (int hh = 0; hh < 2; ++hh)
                d256_load_v_half(sV + hh * kD256VHalfBytes, &tm_vh, bar_vh + 8 * hh, hk, hh * 64, b);
        }
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(smem_u32(&tmem_holder), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;

    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
    constexpr uint32_t idesc_qk = instr_desc_f16(kBf16, 128, 128, false, false);
    constexpr uint32_t idesc_pv = instr_desc_f16(kBf16, 128, 256, false, true);

    if (warp == 4) {
        // =========================== K loads and score MMAs: one thread
        if (tid == 128 && n_tiles > 0) {
            bool ok = mbar_wait(bar_q, 0, &abort_flag, 61);
            for (int t = 0; t < n_tiles && ok; ++t) {
                const int buf = t & 1;
                // S(t) overwrites the buffer P(t - 2) sat in: P V of that tile must have completed
                if (t >= 2) {
                    ok = mbar_wait(bar_o, t & 1, &abort_flag, 67);
                    if (!ok) break;
                }
                // S(t) = Q K_t^T in two runs of eight k-steps, one per half of d; K's halves go round
                // three half-slots, and the slot a run has read is refilled (with the half three
                // further on) as soon as that run has completed
                const uint32_t d_tmem = tmem_base + (buf ? 384u : 0u);
#pragma unroll
                for (int run = 0; run < 2; ++run) {
                    const int kh = 2 * t + run;
                    const uint32_t sKh = sK + (kh % 3) * kD256KHalfBytes;
                    ok = mbar_wait(bar_kh + 8 * (kh % 3), (kh / 3) & 1, &abort_flag, 62);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t koff = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                        mma_ss(d_tmem, smem_desc_sw128(sQ + run * 2 * kHalfBytes + koff, 16, 1024),
                               smem_desc_sw128(sKh + koff, 16, 1024), idesc_qk, run > 0 || ks > 0);
                    }
                    mma_commit(run ? bar_s + 8 * buf : bar_sa);
                }
                if (!ok) break;
                if (2 * t + 3 < 2 * n_tiles) {
                    ok = mbar_wait(bar_sa, t & 1, &abort_flag, 63);
                    if (!ok) break;
                    const int kh = 2 * t + 3;
                    d256_load_k_half(sK + (kh % 3) * kD256KHalfBytes, &tm_k, bar_kh + 8 * (kh % 3), kh & 1, hk,
                                     (kh >> 1) * kTile, b);
                }
                if (2 * t + 4 < 2 * n_tiles) {
                    ok = mbar_wait(bar_s + 8 * buf, (t >> 1) & 1, &abort_flag, 63);
                    if (!ok) break;
                    const int kh = 2 * t + 4;
                    d256_load_k_half(sK + (kh % 3) * kD256KHalfBytes, &tm_k, bar_kh + 8 * (kh % 3), kh & 1, hk,
                                     (kh >> 1) * kTile, b);
                }
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // =========================== V loads and P V MMAs: one thread
        if (tid == 160 && n_tiles > 0) {
            bool ok = true;
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int buf = j & 1;
                // ---- O += P(j) V_j, one group of four k-steps per half of V
                ok = mbar_wait(bar_p + 8 * buf, (j >> 1) & 1, &abort_flag, 64);
                if (!ok) break;
                const uint32_t p_tmem = tmem_base + (buf ? 384u : 0u);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int slot = half;   // half 2 j + half of V sits in slot `half`, its j-th use
                    ok = mbar_wait(bar_vh + 8 * slot, j & 1, &abort_flag, 65);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)   // 16 keys per step: 2048 bytes down each box of the half
                        mma_ts(tmem_base + 128, p_tmem + (half * 4 + ks) * 8,
                               smem_desc_sw128(sV + slot * kD256VHalfBytes + ks * 2048, kD256VBoxBytes, 1024), idesc_pv,
                               (j > 0) || (half > 0) || (ks > 0));
                    mma_commit(half == 0 ? bar_g : bar_o);
                }
                if (!ok) break;
                // ---- refill the half-slots as their groups complete
                ok = mbar_wait(bar_g, j & 1, &abort_flag, 66);
                if (!ok) break;
                if (j + 1 < n_tiles) d256_load_v_half(sV, &tm_vh, bar_vh, hk, (2 * j + 2) * 64, b);
                ok = mbar_wait(bar_o, j & 1, &abort_flag, 67);
                if (!ok) break;
                if (j + 1 < n_tiles)
                    d256_load_v_half(sV + kD256VHalfBytes, &tm_vh, bar_vh + 8, hk, (2 * j + 3) * 64, b);
            }
        }
        __syncwarp();
    } else {
        // =========================== softmax: one thread per query row
        const uint32_t lane_sel = static_cast<uint32_t>(warp * 32) << 16;
        const uint32_t tO = tmem_base + lane_sel + 128;
        const int row = q0 + tid;
        float m_run = -INFINITY;           // reference max of the row, in raw score units
        float l_run = 0.f;                 // running row sum, relative to it
        bool ok = true;

        for (int j = 0; j < n_tiles; ++j) {
            const int buf = j & 1;
            const uint32_t tS = tmem_base + lane_sel + (buf ? 384u : 0u);
            if (!mbar_wait(bar_s + 8 * buf, (j >> 1) & 1, &abort_flag, 68)) { ok = false; break; }
            tc_fence_after();
            // ---- this row of S (four loads in flight, one wait)
            uint32_t sr[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_x32(tS + c * 32, sr[c]);
            tmem_wait_ld();
            float s[128];
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int i = 0; i < 32; ++i) s[c * 32 + i] = __uint_as_float(sr[c][i]);
            // ---- mask: only tiles the diagonal or the end of the keys cross
            const int kv0 = j * kTile;
            const bool need_mask = (p.causal && kv0 + kTile - 1 > q0 + off) || (kv0 + kTile > p.Skv);
            int lim = kTile;
            if (need_mask) {
                lim = p.Skv - kv0;                                    // columns >= lim are past the keys
                if (p.causal) lim = min(lim, row + off - kv0 + 1);    // columns >= lim are above the diagonal
#pragma unroll
                for (int i = 0; i < 128; ++i)
                    if (i >= lim) s[i] = -INFINITY;
            }
            // ---- online softmax update (Appendix A: rowmax / rowsum).  m_run is the reference the
            // exponentials are taken against; it follows the row max only when that outgrew it by
            // more than 2^8 (P then stays <= 256, O and l carry the same reference, so O / l and
            // LSE are unchanged) -- the 256 columns of O are rarely rescaled after the first tiles.
            float m0 = s[0], m1 = s[1], m2 = s[2], m3 = s[3];
#pragma unroll
            for (int i = 4; i < 128; i += 4) {
                m0 = fmaxf(m0, s[i]);
                m1 = fmaxf(m1, s[i + 1]);
                m2 = fmaxf(m2, s[i + 2]);
                m3 = fmaxf(m3, s[i + 3]);
            }
            const float m_tile = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
            const bool moved = (m_tile > m_run) && (m_run == -INFINITY || (m_tile - m_run) * p.scale_log2 > 8.f);
            const float m_new = moved ? m_tile : m_run;
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;   // a row that sees nothing stays finite
            const float alpha =
                moved ? ((m_run == -INFINITY) ? 0.f : fast_exp2((m_run - m_use) * p.scale_log2)) : 1.f;
            const float neg_ms = -m_use * p.scale_log2;
            float l0 = 0.f, l1 = 0.f;
            if (need_mask) {
                // masked entries become exact zeros whatever the scale
#pragma unroll
                for (int i = 0; i < 128; i += 2) {
                    s[i] = (i < lim) ? fast_exp2(fmaf(s[i], p.scale_log2, neg_ms)) : 0.f;
                    s[i + 1] = (i + 1 < lim) ? fast_exp2(fmaf(s[i + 1], p.scale_log2, neg_ms)) : 0.f;
                    l0 += s[i];
                    l1 += s[i + 1];
                }
            } else {
#pragma unroll
                for (int i = 0; i < 128; i += 2) {
                    s[i] = fast_exp2(fmaf(s[i], p.scale_log2, neg_ms));
                    s[i + 1] = fast_exp2(fmaf(s[i + 1], p.scale_log2, neg_ms));
                    l0 += s[i];
                    l1 += s[i + 1];
                }
            }
            l_run = l_run * alpha + (l0 + l1);
            m_run = m_new;

            // ---- O <- alpha * O once the previous P V has landed
            if (j > 0) {
                if (!mbar_wait(bar_o, (j - 1) & 1, &abort_flag, 69)) { ok = false; break; }
                tc_fence_after();
                if (__any_sync(0xffffffffu, moved)) {   // alpha is exactly 1 for a row whose reference stayed
#pragma unroll 2
                    for (int c = 0; c < 8; ++c) {
                        uint32_t r[32];
                        tmem_ld_x32(tO + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                        tmem_st_x32(tO + c * 32, r);
                    }
                }
            }
            // ---- hand P to the second MMA through tensor memory
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t r[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = pack2<T>(s[c * 64 + 2 * i], s[c * 64 + 2 * i + 1]);
                tmem_st_x32(tS + c * 32, r);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar_p + 8 * buf);
        }

        // ---- epilogue: O / l, LSE = m * scale + ln l
        if (ok && n_tiles > 0) ok = mbar_wait(bar_o, (n_tiles - 1) & 1, &abort_flag, 70);
        if (ok && n_tiles > 0) {
            tc_fence_after();
            const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
            const bool live = row < p.Sq;
            const long long obase = (long long)b * p.o_sb + (long long)row * p.o_ss + (long long)h * p.o_sh;
#pragma unroll 2
            for (int c = 0; c < 8; ++c) {
                uint32_t r[32];
                tmem_ld_x32(tO + c * 32, r);
                tmem_wait_ld();
                if (live) {
                    if (p.o_fp32) {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.o) + obase + c * 32);
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            dst[i] = make_float4(__uint_as_float(r[4 * i]) * inv_l, __uint_as_float(r[4 * i + 1]) * inv_l,
                                                 __uint_as_float(r[4 * i + 2]) * inv_l, __uint_as_float(r[4 * i + 3]) * inv_l);
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(static_cast<T*>(p.o) + obase + c * 32);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint4 w;
                            w.x = pack2<T>(__uint_as_float(r[8 * i]) * inv_l, __uint_as_float(r[8 * i + 1]) * inv_l);
                            w.y = pack2<T>(__uint_as_float(r[8 * i + 2]) * inv_l, __uint_as_float(r[8 * i + 3]) * inv_l);
                            w.z = pack2<T>(__uint_as_float(r[8 * i + 4]) * inv_l, __uint_as_float(r[8 * i + 5]) * inv_l);
                            w.w = pack2<T>(__uint_as_float(r[8 * i + 6]) * inv_l, __uint_as_float(r[8 * i + 7]) * inv_l);
                            dst[i] = w;
                        }
                    }
                }
            }
            if (live && p.lse != nullptr) {
                const float lse =
                    (l_run > 0.f) ? (m_run * p.scale_log2 + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
                p.lse[((long long)b * p.Hq + h) * p.Sq + row] = lse;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace fa
