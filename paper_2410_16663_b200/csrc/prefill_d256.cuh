// Attention forward for head dimension 256: a first, straightforward kernel.  One CTA of 128
// threads per (batch, head, 128-row query tile), every stage sequential, one thread per query
// row.  Tiles are 128 rows x 256 elements = four 64-column swizzled TMA boxes (64 KiB); shared
// memory holds Q and one slot each for K and V (193 KiB, one CTA per SM).  S = Q K^T takes sixteen
// k-steps into tensor-memory columns [0,128); P goes back packed over [0,64); O += P V is an
// N = 256 MMA with V as the N-major operand (its four boxes one LBO apart) into columns
// [128,384).  K of the next kv tile is loaded as soon as the score MMA has finished with the
// slot, V as soon as P V has.  Online softmax as in Appendix A (rowmax / rowsum), with O rescaled
// only on steps where some row of the warp moved its max.
#pragma once

#include "prefill_simple.cuh"

namespace fa {

constexpr int kD256TileBytes = 4 * kHalfBytes;              // 128 rows x 256 16-bit elements
constexpr int kD256Smem = 1024 + 3 * kD256TileBytes;

__device__ __forceinline__ void d256_load_tile(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int h, int s0,
                                               int b) {
#pragma unroll
    for (int c = 0; c < 4; ++c) tma_load_4d(dst + c * kHalfBytes, tm, bar, 64 * c, h, s0, b);
}

template <typename T>
__global__ void __launch_bounds__(128, 1)
fa_fwd_d256_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + kD256TileBytes;
    const uint32_t sV = sK + kD256TileBytes;
    __shared__ __align__(8) uint64_t bars[6];
    __shared__ uint32_t tmem_holder;
    __shared__ volatile uint32_t abort_flag;

    const uint32_t bar_q = smem_u32(&bars[0]);
    const uint32_t bar_k = smem_u32(&bars[1]);
    const uint32_t bar_v = smem_u32(&bars[2]);
    const uint32_t bar_s = smem_u32(&bars[3]);
    const uint32_t bar_o = smem_u32(&bars[4]);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int qt = p.n_qtiles - 1 - blockIdx.x;  // long (late) tiles first
    const int h = blockIdx.y;
    const int b = blockIdx.z;
    const int hk = h / (p.Hq / p.Hkv);
    const int q0 = qt * kTile;
    const int off = p.Skv - p.Sq;
    const int n_tiles = kv_tiles_for(q0, kTile, p.Sq, p.Skv, p.causal);

    if (tid == 0) {
        for (int i = 0; i < 5; ++i) mbar_init(smem_u32(&bars[i]), 1);
        abort_flag = 0;
        fence_mbar_init();
        if (n_tiles > 0) {
            mbar_expect_tx(bar_q, kD256TileBytes);
            d256_load_tile(sQ, &tm_q, bar_q, h, q0, b);
            mbar_expect_tx(bar_k, kD256TileBytes);
            d256_load_tile(sK, &tm_k, bar_k, hk, 0, b);
            mbar_expect_tx(bar_v, kD256TileBytes);
            d256_load_tile(sV, &tm_v, bar_v, hk, 0, b);
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
    const uint32_t lane_sel = static_cast<uint32_t>(warp * 32) << 16;
    const uint32_t tS = tmem_base + lane_sel;        // columns [0,128): S, then P packed in [0,64)
    const uint32_t tO = tmem_base + lane_sel + 128;  // columns [128,384): O

    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
    constexpr uint32_t idesc_qk = instr_desc_f16(kBf16, 128, 128, false, false);
    constexpr uint32_t idesc_pv = instr_desc_f16(kBf16, 128, 256, false, true);

    const int row = q0 + tid;          // this thread's query row
    float m_run = -INFINITY;           // running row max, in raw score units
    float l_run = 0.f;                 // running row sum
    bool ok = true;

    for (int j = 0; j < n_tiles && ok; ++j) {
        // ---- S = Q K_j^T
        if (tid == 0) {
            if (j == 0) ok = mbar_wait(bar_q, 0, &abort_flag, 61);
            ok = ok && mbar_wait(bar_k, j & 1, &abort_flag, 62);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 16; ++ks) {
                    const uint32_t koff = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                    mma_ss(tmem_base, smem_desc_sw128(sQ + koff, 16, 1024), smem_desc_sw128(sK + koff, 16, 1024),
                           idesc_qk, ks > 0);
                }
                mma_commit(bar_s);
            }
        }
        __syncwarp();
        if (!mbar_wait(bar_s, j & 1, &abort_flag, 63)) { ok = false; break; }
        tc_fence_after();
        // the score MMA has finished with the K slot: fetch the next tile's keys
        if (tid == 0 && j + 1 < n_tiles) {
            mbar_expect_tx(bar_k, kD256TileBytes);
            d256_load_tile(sK, &tm_k, bar_k, hk, (j + 1) * kTile, b);
        }
        __syncwarp();

        // ---- this row of S
        float s[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld_x32(tS + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) s[c * 32 + i] = __uint_as_float(r[i]);
        }
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
        // ---- online softmax update (Appendix A: rowmax / rowsum)
        float m_tile = s[0];
#pragma unroll
        for (int i = 1; i < 128; ++i) m_tile = fmaxf(m_tile, s[i]);
        const float m_new = fmaxf(m_run, m_tile);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;   // a row that sees nothing stays finite
        const float alpha = (m_run == -INFINITY) ? 0.f : fast_exp2((m_run - m_use) * p.scale_log2);
        const float neg_ms = -m_use * p.scale_log2;
        float l_tile = 0.f;
        if (need_mask) {
            // masked entries become exact zeros whatever the scale
#pragma unroll
            for (int i = 0; i < 128; ++i) {
                s[i] = (i < lim) ? fast_exp2(fmaf(s[i], p.scale_log2, neg_ms)) : 0.f;
                l_tile += s[i];
            }
        } else {
#pragma unroll
            for (int i = 0; i < 128; ++i) {
                s[i] = fast_exp2(fmaf(s[i], p.scale_log2, neg_ms));
                l_tile += s[i];
            }
        }
        l_run = l_run * alpha + l_tile;
        const bool moved = (m_new != m_run);
        m_run = m_new;

        // ---- O <- alpha * O once the previous P V has landed; refill the V slot it freed
        if (j > 0) {
            if (!mbar_wait(bar_o, (j - 1) & 1, &abort_flag, 64)) { ok = false; break; }
            tc_fence_after();
            if (tid == 0) {
                mbar_expect_tx(bar_v, kD256TileBytes);
                d256_load_tile(sV, &tm_v, bar_v, hk, j * kTile, b);
            }
            __syncwarp();
            if (__any_sync(0xffffffffu, moved)) {   // alpha is exactly 1 for a row whose max stayed
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
        __syncthreads();
        // ---- O += P V_j
        if (tid == 0) {
            ok = mbar_wait(bar_v, j & 1, &abort_flag, 65);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)   // 16 kv rows per step: 2048 bytes down each box of V
                    mma_ts(tmem_base + 128, tmem_base + ks * 8, smem_desc_sw128(sV + ks * 2048, kHalfBytes, 1024),
                           idesc_pv, (j > 0) || (ks > 0));
                mma_commit(bar_o);
            }
        }
        __syncwarp();
    }

    // ---- epilogue: O / l, LSE = m * scale + ln l
    if (ok && n_tiles > 0) ok = mbar_wait(bar_o, (n_tiles - 1) & 1, &abort_flag, 66);
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
            const float lse = (l_run > 0.f) ? (m_run * p.scale_log2 + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
            p.lse[((long long)b * p.Hq + h) * p.Sq + row] = lse;
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
