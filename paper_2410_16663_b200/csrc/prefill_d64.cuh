// Attention forward for head dimension 64 (the short, non-causal vision workload of the
// evaluation section: DeiT-like, 197 tokens, 12 heads, large batches; causal and longer
// sequences work too).  The tcgen05 tile shapes of d = 64: Q, K and V tiles are single 128 x 64
// swizzled TMA boxes; S = Q K^T takes four k-steps of 16; O += P V is an N = 64 MMA with V as the
// N-major operand.  Three kernels:
//   fa_fwd_d64_stream_kernel (prefill_d64_stream.cuh)  128 < Skv <= 256: all keys as one tile,
//                            single-pass softmax, a persistent pipeline over (batch, head, two query tiles)
//   fa_fwd_pingpong_kernel   (prefill_pingpong.cuh, D = 64)  longer sequences and packed batches
//   fa_fwd_d64_slim_kernel   (here) any Skv, used up to 128 keys: online softmax over 128-key
//                            tiles, one thread per query row, O kept in registers
#pragma once

#include "prefill_simple.cuh"

namespace fa {

constexpr int kD64TileBytes = 16384;   // 128 rows x 64 16-bit elements: one TMA box

// ---------------------------------------------------------------------------------------
// The general d = 64 kernel, small enough for four CTAs per SM.  One CTA per (batch, head,
// query tile), 128 threads, 49 KiB of shared memory (Q and one slot each for K and V) and 128
// columns of tensor memory: S in [0,128), P packed over [0,64), and the product P V of ONE kv
// tile in [64,128) (columns of S the thread has read by then).  The running output lives in
// registers: after every kv tile the thread reads its row of P V and adds it to alpha * O.
// K of the next tile is loaded as soon as the score MMA has finished with the slot, V as soon
// as P V has.
constexpr int kD64SlimSmem = 1024 + 3 * kD64TileBytes;

template <typename T>
__global__ void __launch_bounds__(128, 4)
fa_fwd_d64_slim_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + kD64TileBytes;
    const uint32_t sV = sK + kD64TileBytes;
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
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(smem_u32(&tmem_holder), 128);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;
    const uint32_t tS = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);

    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
    constexpr uint32_t idesc_qk = instr_desc_f16(kBf16, 128, 128, false, false);
    constexpr uint32_t idesc_pv = instr_desc_f16(kBf16, 128, 64, false, true);

    if (tid == 0 && n_tiles > 0) {
        mbar_expect_tx(bar_q, kD64TileBytes);
        tma_load_4d(sQ, &tm_q, bar_q, 0, h, q0, b);
        mbar_expect_tx(bar_k, kD64TileBytes);
        tma_load_4d(sK, &tm_k, bar_k, 0, hk, 0, b);
        mbar_expect_tx(bar_v, kD64TileBytes);
        tma_load_4d(sV, &tm_v, bar_v, 0, hk, 0, b);
    }
    __syncwarp();

    const int row = q0 + tid;
    float m_run = -INFINITY, l_run = 0.f;
    float acc[64];   // this thread's row of O, relative to m_run
    bool ok = true;

    for (int j = 0; j < n_tiles && ok; ++j) {
        // ---- S = Q K_j^T
        if (tid == 0) {
            if (j == 0) ok = mbar_wait(bar_q, 0, &abort_flag, 71);
            ok = ok && mbar_wait(bar_k, j & 1, &abort_flag, 72);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    mma_ss(tmem_base, smem_desc_sw128(sQ + ks * 32, 16, 1024), smem_desc_sw128(sK + ks * 32, 16, 1024),
                           idesc_qk, ks > 0);
                mma_commit(bar_s);
            }
        }
        __syncwarp();
        if (!mbar_wait(bar_s, j & 1, &abort_flag, 73)) { ok = false; break; }
        tc_fence_after();
        if (tid == 0 && j + 1 < n_tiles) {   // the K slot is free: the next tile's keys
            mbar_expect_tx(bar_k, kD64TileBytes);
            tma_load_4d(sK, &tm_k, bar_k, 0, hk, (j + 1) * kTile, b);
        }
        // ---- mask limit: columns >= lim are past the keys or above the diagonal
        const int kv0 = j * kTile;
        int lim = p.Skv - kv0;
        if (p.causal) lim = min(lim, row + off - kv0 + 1);
        if (row >= p.Sq) lim = 0;
        const bool full = __all_sync(0xffffffffu, lim >= 128);
        // ---- pass 1: max of this tile's scores
        float m_tile = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld_x32(tS + c * 32, r);
            tmem_wait_ld();
            if (full) {
                float m0 = m_tile, m1 = -INFINITY;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    m0 = max3(m0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
                    m1 = max3(m1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                }
                m_tile = fmaxf(m0, m1);
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (c * 32 + i < lim) m_tile = fmaxf(m_tile, __uint_as_float(r[i]));
            }
        }
        const float m_new = fmaxf(m_run, m_tile);
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;   // rows that see nothing stay finite
        const float alpha = (m_run == -INFINITY) ? 0.f : fast_exp2((m_run - m_use) * p.scale_log2);
        const float neg_ms = -m_use * p.scale_log2;
        m_run = m_new;
        // ---- pass 2: P over S's first 64 columns, row sum
        float l_tile = 0.f;
        const uint64_t sc2 = f2_pack(p.scale_log2, p.scale_log2), nm2 = f2_pack(neg_ms, neg_ms);
        uint64_t l2 = f2_pack(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t pk[16];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {   // 16 columns at a time: the row of O keeps 64 registers busy
                uint32_t r[16];
                tmem_ld_x16(tS + c * 32 + hf * 16, r);
                tmem_wait_ld();
                const int col0 = c * 32 + hf * 16;
                if (full) {
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        float x0, x1;
                        f2_unpack(f2_fma(f2_pack(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), sc2, nm2), x0, x1);
                        const float e0 = fast_exp2(x0), e1 = fast_exp2(x1);
                        l2 = f2_add(l2, f2_pack(e0, e1));
                        pk[hf * 8 + (i >> 1)] = pack2<T>(e0, e1);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        const float e0 = (col0 + i < lim) ? fast_exp2(fmaf(__uint_as_float(r[i]), p.scale_log2, neg_ms)) : 0.f;
                        const float e1 = (col0 + i + 1 < lim) ? fast_exp2(fmaf(__uint_as_float(r[i + 1]), p.scale_log2, neg_ms)) : 0.f;
                        l_tile += e0 + e1;
                        pk[hf * 8 + (i >> 1)] = pack2<T>(e0, e1);
                    }
                }
            }
            tmem_st_x16(tS + c * 16, pk);
        }
        {
            float la, lb;
            f2_unpack(l2, la, lb);
            l_tile += la + lb;
        }
        l_run = l_run * alpha + l_tile;
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();
        // ---- P V_j into columns [64,128), not accumulated
        if (tid == 0) {
            ok = mbar_wait(bar_v, j & 1, &abort_flag, 74);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ts(tmem_base + 64, tmem_base + ks * 8, smem_desc_sw128(sV + ks * 2048, 16, 1024), idesc_pv, ks > 0);
                mma_commit(bar_o);
            }
        }
        __syncwarp();
        if (!mbar_wait(bar_o, j & 1, &abort_flag, 75)) { ok = false; break; }
        tc_fence_after();
        if (tid == 0 && j + 1 < n_tiles) {   // the V slot is free
            mbar_expect_tx(bar_v, kD64TileBytes);
            tma_load_4d(sV, &tm_v, bar_v, 0, hk, (j + 1) * kTile, b);
        }
        // ---- O = alpha * O + P V_j, in registers
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t r[32];
            tmem_ld_x32(tS + 64 + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i)
                acc[c * 32 + i] = (j == 0) ? __uint_as_float(r[i]) : fmaf(acc[c * 32 + i], alpha, __uint_as_float(r[i]));
        }
        // the next tile's scores overwrite the columns that were just read
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }

    if (ok && n_tiles > 0 && row < p.Sq) {
        const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
        const long long obase = (long long)b * p.o_sb + (long long)row * p.o_ss + (long long)h * p.o_sh;
        if (p.o_fp32) {
            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.o) + obase);
#pragma unroll
            for (int i = 0; i < 16; ++i)
                dst[i] = make_float4(acc[4 * i] * inv_l, acc[4 * i + 1] * inv_l, acc[4 * i + 2] * inv_l, acc[4 * i + 3] * inv_l);
        } else {
            uint4* dst = reinterpret_cast<uint4*>(static_cast<T*>(p.o) + obase);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                uint4 w;
                w.x = pack2<T>(acc[8 * i] * inv_l, acc[8 * i + 1] * inv_l);
                w.y = pack2<T>(acc[8 * i + 2] * inv_l, acc[8 * i + 3] * inv_l);
                w.z = pack2<T>(acc[8 * i + 4] * inv_l, acc[8 * i + 5] * inv_l);
                w.w = pack2<T>(acc[8 * i + 6] * inv_l, acc[8 * i + 7] * inv_l);
                dst[i] = w;
            }
        }
        if (p.lse != nullptr)
            p.lse[((long long)b * p.Hq + h) * p.Sq + row] =
                (l_run > 0.f) ? (m_run * p.scale_log2 + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, 128);
    }
}

}  // namespace fa
