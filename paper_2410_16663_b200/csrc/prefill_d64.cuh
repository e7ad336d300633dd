// Attention forward for head dimension 64 (the short, non-causal vision workload of the
// evaluation section: DeiT-like, 197 tokens, 12 heads, large batches; causal and longer
// sequences work too).  One CTA per (batch, head, 128-row query tile), 128 threads, two CTAs
// per SM.  Per kv tile: S = Q K^T (four tcgen05.mma k-steps of 16 over d = 64) into tensor
// memory, one thread per row does the online softmax (Appendix A: rowmax / rowsum) with the
// whole S row in registers, P goes back packed into S's columns, O += P V with V as the
// N-major B operand (N = 64).  K and V tiles (128 x 64, one swizzled TMA box each) run through
// a two-slot ring.  Tensor memory: S/P columns [0,128), O columns [128,192).
#pragma once

#include "prefill_simple.cuh"

namespace fa {

constexpr int kD64TileBytes = 16384;   // 128 rows x 64 16-bit elements: one TMA box
constexpr int kD64Smem = 1024 + 5 * kD64TileBytes;

template <typename T>
__global__ void __launch_bounds__(128, 2)
fa_fwd_d64_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;  // the 128-byte swizzle wants 1024
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + kD64TileBytes;        // 2 slots
    const uint32_t sV = sK + 2 * kD64TileBytes;    // 2 slots
    __shared__ __align__(8) uint64_t bars[8];
    __shared__ uint32_t tmem_holder;
    __shared__ volatile uint32_t abort_flag;

    const uint32_t bar_q = smem_u32(&bars[0]);
    const uint32_t bar_k0 = smem_u32(&bars[1]);  // +8 for slot 1
    const uint32_t bar_v0 = smem_u32(&bars[3]);
    const uint32_t bar_s = smem_u32(&bars[5]);
    const uint32_t bar_o = smem_u32(&bars[6]);

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
        for (int i = 0; i < 7; ++i) mbar_init(smem_u32(&bars[i]), 1);
        abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(smem_u32(&tmem_holder), 256);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;
    const uint32_t lane_sel = static_cast<uint32_t>(warp * 32) << 16;
    const uint32_t tS = tmem_base + lane_sel;        // columns [0,128): S, then P packed in [0,64)
    const uint32_t tO = tmem_base + lane_sel + 128;  // columns [128,192): O

    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
    constexpr uint32_t idesc_qk = instr_desc_f16(kBf16, 128, 128, false, false);
    constexpr uint32_t idesc_pv = instr_desc_f16(kBf16, 128, 64, false, true);

    if (tid == 0) {
        mbar_expect_tx(bar_q, kD64TileBytes);
        tma_load_4d(sQ, &tm_q, bar_q, 0, h, q0, b);
        for (int j = 0; j < 2 && j < n_tiles; ++j) {
            mbar_expect_tx(bar_k0 + 8 * j, kD64TileBytes);
            tma_load_4d(sK + j * kD64TileBytes, &tm_k, bar_k0 + 8 * j, 0, hk, j * kTile, b);
            mbar_expect_tx(bar_v0 + 8 * j, kD64TileBytes);
            tma_load_4d(sV + j * kD64TileBytes, &tm_v, bar_v0 + 8 * j, 0, hk, j * kTile, b);
        }
    }
    __syncwarp();

    const int row = q0 + tid;          // this thread's query row
    float m_run = -INFINITY;           // running row max, in raw score units
    float l_run = 0.f;                 // running row sum
    bool ok = true;

    for (int j = 0; j < n_tiles && ok; ++j) {
        const int slot = j & 1;
        const uint32_t ring_parity = (j >> 1) & 1;
        // ---- S = Q K_j^T
        if (tid == 0) {
            if (j == 0) ok = mbar_wait(bar_q, 0, &abort_flag, 41);
            ok = ok && mbar_wait(bar_k0 + 8 * slot, ring_parity, &abort_flag, 42);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    mma_ss(tmem_base, smem_desc_sw128(sQ + ks * 32, 16, 1024),
                           smem_desc_sw128(sK + slot * kD64TileBytes + ks * 32, 16, 1024), idesc_qk, ks > 0);
                mma_commit(bar_s);
            }
        }
        __syncwarp();
        if (!mbar_wait(bar_s, j & 1, &abort_flag, 43)) { ok = false; break; }
        tc_fence_after();

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
        int lim = 128;
        if (need_mask) {
            lim = p.Skv - kv0;                                    // columns >= lim are past the keys
            if (p.causal) lim = min(lim, row + off - kv0 + 1);    // columns >= lim are above the diagonal
#pragma unroll
            for (int i = 0; i < 128; ++i)
                if (i >= lim) s[i] = -INFINITY;
        }
        // ---- online softmax update
        float m_tile = s[0];
#pragma unroll
        for (int i = 1; i < 128; ++i) m_tile = fmaxf(m_tile, s[i]);
        const float m_new = fmaxf(m_run, m_tile);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;   // rows that see nothing stay finite
        const float alpha = (m_run == -INFINITY) ? 0.f : fast_exp2((m_run - m_use) * p.scale_log2);
        const float neg_ms = -m_use * p.scale_log2;
        float l_tile = 0.f;
#pragma unroll
        for (int i = 0; i < 128; ++i) {
            // masked entries become exact zeros whatever the scale
            s[i] = (i < lim) ? fast_exp2(fmaf(s[i], p.scale_log2, neg_ms)) : 0.f;
            l_tile += s[i];
        }
        l_run = l_run * alpha + l_tile;
        m_run = m_new;

        // ---- O <- alpha * O once the previous P V has landed; refill the slot it freed
        if (j > 0) {
            if (!mbar_wait(bar_o, (j - 1) & 1, &abort_flag, 44)) { ok = false; break; }
            tc_fence_after();
            if (tid == 0 && j + 1 < n_tiles) {
                const int ns = (j + 1) & 1;
                mbar_expect_tx(bar_k0 + 8 * ns, kD64TileBytes);
                tma_load_4d(sK + ns * kD64TileBytes, &tm_k, bar_k0 + 8 * ns, 0, hk, (j + 1) * kTile, b);
                mbar_expect_tx(bar_v0 + 8 * ns, kD64TileBytes);
                tma_load_4d(sV + ns * kD64TileBytes, &tm_v, bar_v0 + 8 * ns, 0, hk, (j + 1) * kTile, b);
            }
            __syncwarp();
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t r[32];
                tmem_ld_x32(tO + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                tmem_st_x32(tO + c * 32, r);
            }
        }
        // ---- P, packed two per column, over S's first 64 columns
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
            ok = mbar_wait(bar_v0 + 8 * slot, ring_parity, &abort_flag, 45);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)  // 16 kv rows per step: 2048 bytes down the swizzled V tile
                    mma_ts(tmem_base + 128, tmem_base + ks * 8,
                           smem_desc_sw128(sV + slot * kD64TileBytes + ks * 2048, 16, 1024), idesc_pv,
                           (j > 0) || (ks > 0));
                mma_commit(bar_o);
            }
        }
        __syncwarp();
    }

    // ---- epilogue: O / l, LSE = m * scale + ln l
    if (ok && n_tiles > 0) ok = mbar_wait(bar_o, (n_tiles - 1) & 1, &abort_flag, 46);
    if (ok && n_tiles > 0) {
        tc_fence_after();
        const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
        const bool live = row < p.Sq;
        const long long obase = (long long)b * p.o_sb + (long long)row * p.o_ss + (long long)h * p.o_sh;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
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
        tmem_dealloc(tmem_base, 256);
    }
}

}  // namespace fa
