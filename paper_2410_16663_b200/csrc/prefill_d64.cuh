// Attention forward for head dimension 64 (the short, non-causal vision workload of the
// evaluation section: DeiT-like, 197 tokens, 12 heads, large batches; causal and longer
// sequences work too).  Two kernels, both with one thread per query row and the tcgen05 tile
// shapes of d = 64 (Q, K and V tiles are single 128 x 64 swizzled TMA boxes; S = Q K^T takes four
// k-steps of 16; O += P V is an N = 64 MMA with V as the N-major operand):
//   fa_fwd_d64_short_kernel  128 < Skv <= 256: all keys as one 256-wide tile, single-pass softmax
//   fa_fwd_d64_slim_kernel   any Skv: online softmax over 128-key tiles, O kept in registers
#pragma once

#include "prefill_simple.cuh"

namespace fa {

constexpr int kD64TileBytes = 16384;   // 128 rows x 64 16-bit elements: one TMA box

// ---------------------------------------------------------------------------------------
// Short sequences (128 < Skv <= 256, d = 64): the whole key range is one 256-wide tile, so the
// softmax needs no running state.  One CTA of two warpgroups per (batch, head, pair of query
// tiles): K and V are loaded once for both query tiles; per query tile one N = 256 score MMA
// into tensor-memory columns [0,256).  Warpgroup w then owns keys [128 w, 128 w + 128) of every
// row: a first pass over its 128 columns for the row max of that half, a second pass that writes
// P = exp(S - max) packed over the half's first 64 columns (a chunk's P lands in columns the
// thread has already read), then the half's product P V into the half's last 64 columns, which
// the scores no longer need.  The epilogue brings the two products to a common reference max
// (their row max and row sum cross through shared memory) and each thread writes 32 of its
// row's 64 output columns.  Chunks of 32 columns that lie entirely past the keys are skipped
// (their P is written as 0).  Two CTAs per SM (97 KiB of shared memory, 256 tensor-memory
// columns each).
constexpr int kD64ShortSmem = 1024 + 6 * kD64TileBytes;

// One query row against up to 32 * kChunks keys whose raw scores sit in tensor-memory columns
// [0, 32 kChunks) at tS (this thread's lane): row max m (raw units), row sum l of
// P = exp2((S - m) * scale_log2), and P written packed over columns [0, 16 kChunks).  Columns
// >= lim are hidden (lim may be negative); n_chunks = chunks of 32 columns that hold keys.
// Warp-collective (tensor-memory loads and stores).
template <typename T, int kChunks>
__device__ __forceinline__ void d64_row_softmax(uint32_t tS, int lim, int n_chunks, float scale_log2, float& m,
                                                float& l) {
    // ---- pass 1: row max
    m = -INFINITY;
    // (a warp stops at the last chunk any of its rows can see)
    const int my_chunks = min(n_chunks, (__reduce_max_sync(0xffffffffu, max(lim, 0)) + 31) / 32);
    for (int c = 0; c < my_chunks; ++c) {
        uint32_t r[32];
        tmem_ld_x32(tS + c * 32, r);
        tmem_wait_ld();
        const int live = lim - c * 32;
        if (__all_sync(0xffffffffu, live >= 32)) {
            // every row of the warp sees the whole chunk: no selects
            float m0 = m, m1 = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
                m0 = max3(m0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
                m1 = max3(m1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
            }
            m = fmaxf(m0, m1);
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < live) m = fmaxf(m, __uint_as_float(r[i]));
        }
    }
    const float m_use = (m == -INFINITY) ? 0.f : m;   // a row that sees nothing stays finite
    const float neg_ms = -m_use * scale_log2;
    // ---- pass 2: P = exp2(S * scale_log2 - max * scale_log2), row sum
    l = 0.f;
    const uint64_t sc2 = f2_pack(scale_log2, scale_log2), nm2 = f2_pack(neg_ms, neg_ms);
    uint64_t l2 = f2_pack(0.f, 0.f);
    for (int c = 0; c < kChunks; ++c) {
        uint32_t pk[16];
        if (c < my_chunks) {
            uint32_t r[32];
            tmem_ld_x32(tS + c * 32, r);
            tmem_wait_ld();
            const int live = lim - c * 32;
            if (__all_sync(0xffffffffu, live >= 32)) {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float x0, x1;
                    f2_unpack(f2_fma(f2_pack(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), sc2, nm2), x0, x1);
                    const float e0 = fast_exp2(x0), e1 = fast_exp2(x1);
                    l2 = f2_add(l2, f2_pack(e0, e1));
                    pk[i >> 1] = pack2<T>(e0, e1);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float e0 = (i < live) ? fast_exp2(fmaf(__uint_as_float(r[i]), scale_log2, neg_ms)) : 0.f;
                    const float e1 = (i + 1 < live) ? fast_exp2(fmaf(__uint_as_float(r[i + 1]), scale_log2, neg_ms)) : 0.f;
                    l += e0 + e1;
                    pk[i >> 1] = pack2<T>(e0, e1);
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = 0u;
        }
        tmem_st_x16(tS + c * 16, pk);
    }
    {
        float la, lb;
        f2_unpack(l2, la, lb);
        l += la + lb;
    }
}

// This thread's row of O (64 fp32 columns in r0, r1) scaled by inv_l and stored.
template <typename T>
__device__ __forceinline__ void d64_store_row(const FwdParams& p, long long obase, const uint32_t (&r0)[32],
                                              const uint32_t (&r1)[32], float inv_l) {
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const uint32_t(&r)[32] = c ? r1 : r0;
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


constexpr int kD64ShortThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kD64ShortThreads, 2)
fa_fwd_d64_short_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, const FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;                  // 2 query tiles
    const uint32_t sK = sQ + 2 * kD64TileBytes;     // keys 0..255: two boxes back to back
    const uint32_t sV = sK + 2 * kD64TileBytes;
    __shared__ __align__(8) uint64_t bars[8];
    __shared__ uint32_t tmem_holder;
    __shared__ volatile uint32_t abort_flag;
    __shared__ float ex_m[2][kTile], ex_l[2][kTile];   // row max and row sum of each half of the keys

    const uint32_t bar_q0 = smem_u32(&bars[0]);  // +8 for the second query tile
    const uint32_t bar_k = smem_u32(&bars[2]);
    const uint32_t bar_v = smem_u32(&bars[3]);
    const uint32_t bar_s = smem_u32(&bars[4]);
    const uint32_t bar_o = smem_u32(&bars[5]);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int wg = tid >> 7;          // 0: keys 0..127, 1: keys 128..255
    const int r_in = tid & 127;       // row of the query tile (both warpgroups cover all rows)
    const int h = blockIdx.y;
    const int b = blockIdx.z;
    const int hk = h / (p.Hq / p.Hkv);
    const int qt0 = blockIdx.x * 2;                       // first query tile of this CTA
    const int nq = min(2, p.n_qtiles - qt0);              // its query tiles
    const int off = p.Skv - p.Sq;

    if (tid == 32) {
        // barriers and all loads of the CTA at once, while warp 0 allocates tensor memory
        for (int i = 0; i < 6; ++i) mbar_init(smem_u32(&bars[i]), i == 5 ? 2 : 1);   // two threads issue P V
        abort_flag = 0;
        fence_mbar_init();
        mbar_expect_tx(bar_q0, kD64TileBytes);
        tma_load_4d(sQ, &tm_q, bar_q0, 0, h, qt0 * kTile, b);
        mbar_expect_tx(bar_k, 2 * kD64TileBytes);   // rows past the keys arrive as zeros
        tma_load_4d(sK, &tm_k, bar_k, 0, hk, 0, b);
        tma_load_4d(sK + kD64TileBytes, &tm_k, bar_k, 0, hk, kTile, b);
        if (nq > 1) {
            mbar_expect_tx(bar_q0 + 8, kD64TileBytes);
            tma_load_4d(sQ + kD64TileBytes, &tm_q, bar_q0 + 8, 0, h, (qt0 + 1) * kTile, b);
        }
        mbar_expect_tx(bar_v, 2 * kD64TileBytes);
        tma_load_4d(sV, &tm_v, bar_v, 0, hk, 0, b);
        tma_load_4d(sV + kD64TileBytes, &tm_v, bar_v, 0, hk, kTile, b);
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
    // warps w and w + 4 reach the same 32 lanes (rows) of tensor memory
    const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
    // Columns: [0,128) scores of keys 0..127, P of those keys packed over [0,64), their product
    // P V in [64,128); the same for keys 128..255 in [128,256).  Each half belongs to one
    // warpgroup until the epilogue, so the two never wait for each other before it.
    const uint32_t tS = tmem_base + lane_sel + 128 * wg;
    const uint32_t tOa = tmem_base + lane_sel + 64 + 32 * wg;    // this thread's 32 output columns, keys 0..127
    const uint32_t tOb = tmem_base + lane_sel + 192 + 32 * wg;   // the same of keys 128..255

    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
    constexpr uint32_t idesc_qk = instr_desc_f16(kBf16, 128, 256, false, false);
    constexpr uint32_t idesc_pv = instr_desc_f16(kBf16, 128, 64, false, true);

    const int n_chunks = min(4, (p.Skv + 31) / 32 - 4 * wg);   // chunks of 32 columns of this half that hold keys
    bool ok = true;
    for (int t = 0; t < nq && ok; ++t) {
        const int q0 = (qt0 + t) * kTile;
        const int row = q0 + r_in;
        // ---- S = Q K^T over all keys
        if (tid == 0) {
            ok = mbar_wait(bar_q0 + 8 * t, 0, &abort_flag, 51);
            if (t == 0) ok = ok && mbar_wait(bar_k, 0, &abort_flag, 52);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    mma_ss(tmem_base, smem_desc_sw128(sQ + t * kD64TileBytes + ks * 32, 16, 1024),
                           smem_desc_sw128(sK + ks * 32, 16, 1024), idesc_qk, ks > 0);
                mma_commit(bar_s);
            }
        }
        __syncwarp();
        if (!mbar_wait(bar_s, t & 1, &abort_flag, 53)) { ok = false; break; }
        tc_fence_after();

        // columns >= lim are past the keys or above the diagonal; a row past the end of the
        // queries (the ragged last tile) keeps nothing, which spares its exponentials
        int lim = p.Skv;
        if (p.causal) lim = min(lim, row + off + 1);
        if (row >= p.Sq) lim = 0;
        // softmax of this half of the keys relative to the half's own row max; the epilogue
        // brings the two halves to a common reference
        float m, l;
        d64_row_softmax<T, 4>(tS, lim - 128 * wg, n_chunks, p.scale_log2, m, l);
        ex_m[wg][r_in] = m;
        ex_l[wg][r_in] = l;
        tmem_wait_st();
        tc_fence_before();
        if (wg == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
        else asm volatile("bar.sync 2, 128;" ::: "memory");
        // ---- O = P V, one half of the keys per warpgroup (each issued by the warpgroup's first thread)
        if (r_in == 0) {
            if (t == 0) ok = mbar_wait(bar_v, 0, &abort_flag, 54);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)  // 16 keys per step: 2048 bytes down the V boxes
                    mma_ts(tmem_base + 64 + 128 * wg, tmem_base + 128 * wg + ks * 8,
                           smem_desc_sw128(sV + (wg * 8 + ks) * 2048, 16, 1024), idesc_pv, ks > 0);
                mma_commit(bar_o);
            }
        }
        __syncwarp();
        if (!mbar_wait(bar_o, t & 1, &abort_flag, 55)) { ok = false; break; }
        tc_fence_after();
        __syncthreads();   // the other half's row max and row sum are in shared memory
        // ---- epilogue: both halves on a common reference, O / l, LSE = max * scale + ln l;
        // a thread writes 32 of its row's 64 columns
        const float m_o = ex_m[wg ^ 1][r_in], l_o = ex_l[wg ^ 1][r_in];
        const float mm = fmaxf(m, m_o);
        const float w_me = (m == -INFINITY) ? 0.f : fast_exp2((m - mm) * p.scale_log2);
        const float w_ot = (m_o == -INFINITY) ? 0.f : fast_exp2((m_o - mm) * p.scale_log2);
        const float lt = l * w_me + l_o * w_ot;
        const float inv_l = (lt > 0.f) ? 1.f / lt : 0.f;
        const float fa_ = (wg == 0 ? w_me : w_ot) * inv_l;   // weight of the product over keys 0..127
        const float fb_ = (wg == 0 ? w_ot : w_me) * inv_l;
        const bool live_row = row < p.Sq;
        const long long obase =
            (long long)b * p.o_sb + (long long)row * p.o_ss + (long long)h * p.o_sh + 32 * wg;
        {
            uint32_t r[32], r2[32];
            tmem_ld_x32(tOa, r);
            tmem_ld_x32(tOb, r2);
            tmem_wait_ld();
            float o[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __uint_as_float(r[i]) * fa_ + __uint_as_float(r2[i]) * fb_;
            if (live_row) {
                if (p.o_fp32) {
                    float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.o) + obase);
#pragma unroll
                    for (int i = 0; i < 8; ++i) dst[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                } else {
                    uint4* dst = reinterpret_cast<uint4*>(static_cast<T*>(p.o) + obase);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 w;
                        w.x = pack2<T>(o[8 * i], o[8 * i + 1]);
                        w.y = pack2<T>(o[8 * i + 2], o[8 * i + 3]);
                        w.z = pack2<T>(o[8 * i + 4], o[8 * i + 5]);
                        w.w = pack2<T>(o[8 * i + 6], o[8 * i + 7]);
                        dst[i] = w;
                    }
                }
            }
        }
        if (wg == 0 && live_row && p.lse != nullptr) {
            const float lse = (lt > 0.f) ? (mm * p.scale_log2 + log2f(lt)) * 0.6931471805599453f : -INFINITY;
            p.lse[((long long)b * p.Hq + h) * p.Sq + row] = lse;
        }
        // the next query tile's scores overwrite the columns O was read from
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, 256);
    }
}

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
