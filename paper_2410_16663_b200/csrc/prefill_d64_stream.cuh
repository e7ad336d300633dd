// Attention forward for head dimension 64 and 128 < Skv <= 256 (the short, non-causal vision
// workload of the evaluation section: 197 tokens, 12 heads, batches in the hundreds), as a
// persistent pipeline: one CTA per SM walks a static list of items (batch, head, pair of query
// tiles) and keeps several of them in flight at different stages.
//
//   loaders   two threads; Q (two tiles) + K, and V, of an item go into one of two shared-memory
//             stages of 96 KiB, one item ahead of the math
//   S thread  S = Q K^T of one query tile against ALL keys into one of two 256-column buffers of
//             tensor memory, as two chains of four k-steps: the first half of the keys (rounded
//             to 16) into the buffer's first columns, the second half into its last
//   softmax   four warpgroups in two pairs; pair p owns buffer p, i.e. every other query tile.
//             Inside a pair warpgroup h takes half h of the keys of every row (a row has two
//             threads, in different warps): row max of the half, the halves' maxima cross through
//             shared memory, then P = exp(S - max) written packed over columns the thread has
//             already read, and the row sum
//   PV thread O = P V for the tile (N = 64, V as the N-major operand) into columns [64,128) of
//             the same buffer -- columns of half 0's scores, read by then, that half 1 never
//             touches -- starting on half 0's keys as soon as its warpgroup is through
//   epilogue  by the same pair: each thread scales and stores 32 of its row's 64 columns; the
//             buffer goes back to the S thread as soon as O is in registers
//
// While pair 0 is in the exponentials of one query tile, pair 1 is in its row-max pass or its
// epilogue, the S thread fills the other buffer as soon as it is handed back, and the loads of
// the next item are under way; every scheduler has four softmax warps to pick from.  All keys
// are one tile, so the softmax needs no running state (Appendix A's recurrence with one block).
#pragma once

#include "prefill_d64.cuh"
#include "prefill_pipelined.cuh"

namespace fa {

constexpr int kD64StThreads = 640;     // 16 softmax warps + S thread, Q/K loader, PV thread, V loader
constexpr int kD64StStageBytes = 6 * kD64TileBytes;          // Q0 Q1 K0 K1 V0 V1
constexpr int kD64StSmem = 1024 + 2 * kD64StStageBytes;

namespace d64b {   // barrier indices
constexpr int qk_full = 0;    // [2] by stage: TMA -> S thread
constexpr int qk_empty = 2;   // [2] S thread (commit) -> Q/K loader
constexpr int v_full = 4;     // [2] TMA -> PV thread
constexpr int v_empty = 6;    // [2] PV thread (commit) -> V loader
constexpr int s_full = 8;     // [2][2] by buffer and half of the keys: S thread (commit) -> that warpgroup
constexpr int o_full = 12;    // [2] PV thread (commit) -> pair
// every thread of a warpgroup arrives (count 128)
constexpr int p_full = 14;    // [2][2] by buffer and half: warpgroup -> PV thread
// every thread of a pair arrives (count 256)
constexpr int s_free = 18;    // [2] pair -> S thread: O has been read, the buffer may take new scores
constexpr int row_max = 20;   // [2] the two halves of a pair -> each other
constexpr int count = 22;
}  // namespace d64b

struct D64StItem {
    int b, h, hk, q0, nq, first;   // q0: first query row of the pair of tiles; first: tile taken first
};
// Item `ord` of this CTA (items are dealt round-robin); false past the end.
__device__ __forceinline__ bool d64st_item(const FwdParams& p, int n_qpairs, int total_items, int ord, D64StItem& it) {
    // (32-bit arithmetic: the launcher keeps total_items below 2^31, and every role pays for this
    // between two items)
    const unsigned int idx = blockIdx.x + (unsigned int)ord * gridDim.x;
    if (idx >= (unsigned int)total_items) return false;
    unsigned int bh = idx, qp = 0;
    if (n_qpairs > 1) {
        bh = idx / (unsigned int)n_qpairs;
        qp = idx - bh * (unsigned int)n_qpairs;
    }
    const unsigned int b = bh / (unsigned int)p.Hq;
    it.b = (int)b;
    it.h = (int)(bh - b * (unsigned int)p.Hq);
    it.hk = (p.Hq == p.Hkv) ? it.h : it.h / (p.Hq / p.Hkv);
    it.q0 = (int)qp * 2 * kTile;
    it.nq = min(2, p.n_qtiles - 2 * (int)qp);
    // the pairs alternate over an item's tiles, and the second tile of a ragged pair has fewer
    // live rows: taking it first in every other item evens the pairs out
    it.first = (it.nq == 2) ? (ord & 1) : 0;
    return true;
}
__device__ __forceinline__ uint32_t d64_bar(uint32_t bar0, int i) { return bar0 + 8 * i; }
__device__ __forceinline__ bool d64_warp_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, unsigned int where) {
    const bool ok = mbar_wait(bar, parity, abort_flag, where);
    return __all_sync(0xffffffffu, ok);
}

template <typename T>
__global__ void __launch_bounds__(kD64StThreads, 1)
fa_fwd_d64_stream_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                         const __grid_constant__ CUtensorMap tm_v, const FwdParams p, const int n_qpairs,
                         const int total_items) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bars[d64b::count];
    __shared__ uint32_t tmem_holder;
    __shared__ uint32_t abort_word;
    __shared__ float half_max[2][2][kTile];   // [pair][half][row]
    __shared__ float half_sum[2][2][kTile];
    volatile uint32_t* abort_flag = &abort_word;
    const uint32_t bar0 = smem_u32(&bars[0]);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < d64b::count; ++i) mbar_init(d64_bar(bar0, i), i >= d64b::s_free ? 256u : (i >= d64b::p_full ? 128u : 1u));
        abort_word = 0;
        fence_mbar_init();
    }
    if (warp == 16) {
        tmem_alloc(smem_u32(&tmem_holder), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;
    const int off = p.Skv - p.Sq;
    // chunks of 16 keys: half 0 takes the first c0 of them, half 1 the rest
    const int nch = (p.Skv + 15) >> 4;
    const int c0 = (nch + 1) >> 1;
    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;

    if (warp < 16) {
        // ================================================================ softmax + epilogue
        const int pr = warp >> 3;            // pair: owns buffer pr, takes the units with u & 1 == pr
        const int hf = (warp >> 2) & 1;      // half of the keys
        const int r = tid & 127;             // row of the tile
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tBuf = tmem_base + lane_sel + 256 * pr;
        const int cs = hf ? c0 : 0, ce = hf ? nch : c0;           // this half's chunks
        // Columns of a buffer: the scores of half 0 from column 0 up, those of half 1 up to column
        // 256 (chunk c of either half at col0 + 16 c); P of a half packed from the half's first
        // column on; O in [64,128), which half 0's scores leave free once they have been read and
        // which half 1 never touches -- so O += P V may start on half 0's keys while half 1 is
        // still at its exponentials.
        const uint32_t tS = tBuf + (hf ? 256 - 16 * nch : 0);
        const uint32_t tP = tBuf + (hf ? 256 - 16 * (nch - c0) : 0);
        const uint32_t tO = tBuf + 64 + 32 * hf;                  // this thread's 32 output columns
        const float scale_log2 = p.scale_log2;
        float* const hm_mine = &half_max[pr][hf][r];
        const float* const hm_partner = &half_max[pr][1 - hf][r];
        float* const hl_mine = &half_sum[pr][hf][r];
        const float* const hl_partner = &half_sum[pr][1 - hf][r];
        uint32_t u = 0;
        bool ok = true;
        D64StItem it;
        for (int ord = 0; ok && d64st_item(p, n_qpairs, total_items, ord, it); ++ord) {
            for (int t = 0; t < it.nq && ok; ++t, ++u) {
                if ((u & 1u) != (uint32_t)pr) continue;
                const uint32_t ph = (u >> 1) & 1;     // the pair's barriers change phase once per unit of its own
                const int row = it.q0 + (t ^ it.first) * kTile + r;
                // columns >= lim are past the keys or above the diagonal; a row past the end of the
                // queries keeps nothing
                int lim = p.Skv;
                if (p.causal) lim = min(lim, row + off + 1);
                if (row >= p.Sq) lim = 0;
                const int warp_lim = __reduce_max_sync(0xffffffffu, max(lim, 0));
                // a warp without any live row (the ragged tile's last warps) only keeps step with the barriers
                const int cend = min(ce, (warp_lim + 15) >> 4);   // chunks some row of the warp sees
                if (!d64_warp_wait(d64_bar(bar0, d64b::s_full + 2 * pr + hf), ph, abort_flag, 310 + pr)) { ok = false; break; }
                tc_fence_after();
                // ---- pass 1: row max over this half
                float m = -INFINITY;
                for (int c = cs; c < cend; ++c) {
                    uint32_t s[16];
                    tmem_ld_x16(tS + 16 * c, s);
                    tmem_wait_ld();
                    const int live = lim - 16 * c;
                    if (__all_sync(0xffffffffu, live >= 16)) {
                        float m0 = m, m1 = -INFINITY;
#pragma unroll
                        for (int i = 0; i < 16; i += 4) {
                            m0 = max3(m0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
                            m1 = max3(m1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
                        }
                        m = fmaxf(m0, m1);
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (i < live) m = fmaxf(m, __uint_as_float(s[i]));
                    }
                }
                *hm_mine = m;
                mbar_arrive(d64_bar(bar0, d64b::row_max + pr));
                if (!d64_warp_wait(d64_bar(bar0, d64b::row_max + pr), ph, abort_flag, 312 + pr)) { ok = false; break; }
                m = fmaxf(m, *hm_partner);
                const float m_use = (m == -INFINITY) ? 0.f : m;   // a row that sees nothing stays finite
                const float neg_ms = -m_use * scale_log2;
                // ---- pass 2: P = exp2(S * scale - max * scale), row sum of the half
                const uint64_t sc2 = f2_pack(scale_log2, scale_log2), nm2 = f2_pack(neg_ms, neg_ms);
                uint64_t l2 = f2_pack(0.f, 0.f);
                float l = 0.f;
                if (warp_lim > 0) {
                    for (int c = cs; c < ce; ++c) {
                        uint32_t pk[8];
                        if (c < cend) {
                            uint32_t s[16];
                            tmem_ld_x16(tS + 16 * c, s);
                            tmem_wait_ld();
                            const int live = lim - 16 * c;
                            if (__all_sync(0xffffffffu, live >= 16)) {
#pragma unroll
                                for (int i = 0; i < 16; i += 2) {
                                    float x0, x1;
                                    f2_unpack(f2_fma(f2_pack(__uint_as_float(s[i]), __uint_as_float(s[i + 1])), sc2, nm2), x0, x1);
                                    const float e0 = fast_exp2(x0), e1 = fast_exp2(x1);
                                    l2 = f2_add(l2, f2_pack(e0, e1));
                                    pk[i >> 1] = pack2<T>(e0, e1);
                                }
                            } else {
#pragma unroll
                                for (int i = 0; i < 16; i += 2) {
                                    const float e0 = (i < live) ? fast_exp2(fmaf(__uint_as_float(s[i]), scale_log2, neg_ms)) : 0.f;
                                    const float e1 = (i + 1 < live) ? fast_exp2(fmaf(__uint_as_float(s[i + 1]), scale_log2, neg_ms)) : 0.f;
                                    l += e0 + e1;
                                    pk[i >> 1] = pack2<T>(e0, e1);
                                }
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i) pk[i] = 0u;
                        }
                        tmem_st_x8(tP + 8 * (c - cs), pk);
                    }
                    float la, lb;
                    f2_unpack(l2, la, lb);
                    l += la + lb;
                    tmem_wait_st();
                }
                *hl_mine = l;
                tc_fence_before();
                mbar_arrive(d64_bar(bar0, d64b::p_full + 2 * pr + hf));
                // ---- epilogue: O / l and LSE = max * scale + ln l; a thread writes 32 of its row's 64 columns
                if (!d64_warp_wait(d64_bar(bar0, d64b::o_full + pr), ph, abort_flag, 314 + pr)) { ok = false; break; }
                tc_fence_after();
                // (the partner's sum was written before its arrival on its p_full, which the MMAs behind o_full waited for)
                const float lt = l + *hl_partner;
                if (warp_lim > 0) {
                    uint32_t o[32];
                    tmem_ld_x32(tO, o);
                    tmem_wait_ld();
                    // O is in registers: the buffer may take the scores of the pair's next unit
                    tc_fence_before();
                    mbar_arrive(d64_bar(bar0, d64b::s_free + pr));
                    const float inv_l = (lt > 0.f) ? 1.f / lt : 0.f;
                    if (row < p.Sq) {
                        const long long obase = (long long)it.b * p.o_sb + (long long)row * p.o_ss + (long long)it.h * p.o_sh + 32 * hf;
                        if (p.o_fp32) {
                            float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.o) + obase);
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                dst[i] = make_float4(__uint_as_float(o[4 * i]) * inv_l, __uint_as_float(o[4 * i + 1]) * inv_l,
                                                     __uint_as_float(o[4 * i + 2]) * inv_l, __uint_as_float(o[4 * i + 3]) * inv_l);
                        } else {
                            uint32_t w[16];
#pragma unroll
                            for (int i = 0; i < 16; ++i) w[i] = pack2<T>(__uint_as_float(o[2 * i]) * inv_l, __uint_as_float(o[2 * i + 1]) * inv_l);
                            T* dst = static_cast<T*>(p.o) + obase;
                            if (p.o_align32) {   // a thread's 64 bytes as two 256-bit stores: half the requests
                                st_global_v8(dst, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
                                st_global_v8(dst + 16, w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]);
                            } else {
#pragma unroll
                                for (int i = 0; i < 4; ++i)
                                    reinterpret_cast<uint4*>(dst)[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
                            }
                        }
                        if (hf == 0 && p.lse != nullptr)
                            p.lse[((long long)it.b * p.Hq + it.h) * p.Sq + row] =
                                (lt > 0.f) ? (m_use * scale_log2 + log2f(lt)) * 0.6931471805599453f : -INFINITY;
                    }
                }
                if (warp_lim <= 0) {   // a warp that read nothing hands the buffer back all the same
                    tc_fence_before();
                    mbar_arrive(d64_bar(bar0, d64b::s_free + pr));
                }
            }
        }
    } else if (lane == 0) {
        const uint32_t sStage0 = smem_base;
        if (warp == 16) {
            // ============================================================ S = Q K^T
            const uint32_t n1 = 16u * (uint32_t)(nch - c0);
            const uint32_t idesc0 = instr_desc_f16(kBf16, 128, 16 * c0, false, false), idesc1 = instr_desc_f16(kBf16, 128, (int)n1, false, false);
            uint32_t u = 0;
            D64StItem it;
            bool ok = true;
            for (int ord = 0; ok && d64st_item(p, n_qpairs, total_items, ord, it); ++ord) {
                const uint32_t st = ord & 1;
                const uint32_t sQ = sStage0 + st * kD64StStageBytes, sK = sQ + 2 * kD64TileBytes;
                if (!mbar_wait(d64_bar(bar0, d64b::qk_full + st), (ord >> 1) & 1, abort_flag, 330)) break;
                for (int t = 0; t < it.nq; ++t, ++u) {
                    const uint32_t buf = u & 1;
                    // the pair has read O of its previous unit out of this buffer
                    if (u >= 2 && !mbar_wait(d64_bar(bar0, d64b::s_free + buf), ((u >> 1) - 1) & 1, abort_flag, 331)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_lo = desc_lo(sQ + (uint32_t)(t ^ it.first) * kD64TileBytes, 16);
                    const uint32_t b0_lo = desc_lo(sK, 16), b1_lo = desc_lo(sK + c0 * 2048, 16);   // 16 keys = 2048 bytes
                    const uint32_t tB = tmem_base + 256 * buf;
                    // one chain of four k-steps per half of the keys, each with a barrier of its own
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) mma_ss_lo(tB, a_lo + ks * (32 >> 4), b0_lo + ks * (32 >> 4), idesc0, ks > 0 ? 1u : 0u);
                    mma_commit(d64_bar(bar0, d64b::s_full + 2 * buf));
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) mma_ss_lo(tB + 256 - n1, a_lo + ks * (32 >> 4), b1_lo + ks * (32 >> 4), idesc1, ks > 0 ? 1u : 0u);
                    mma_commit(d64_bar(bar0, d64b::s_full + 2 * buf + 1));
                }
                if (ok) mma_commit(d64_bar(bar0, d64b::qk_empty + st));
            }
        } else if (warp == 18) {
            // ============================================================ O = P V
            constexpr uint32_t idesc = instr_desc_f16(kBf16, 128, 64, false, true);
            uint32_t u = 0;
            D64StItem it;
            bool ok = true;
            for (int ord = 0; ok && d64st_item(p, n_qpairs, total_items, ord, it); ++ord) {
                const uint32_t st = ord & 1;
                const uint32_t sV = sStage0 + st * kD64StStageBytes + 4 * kD64TileBytes;
                if (!mbar_wait(d64_bar(bar0, d64b::v_full + st), (ord >> 1) & 1, abort_flag, 340)) break;
                for (int t = 0; t < it.nq; ++t, ++u) {
                    const uint32_t buf = u & 1;
                    const uint32_t tB = tmem_base + 256 * buf;
                    const uint32_t b_lo = desc_lo(sV, 16);
                    // 16 keys per step: 2048 bytes down the V boxes.  Half 0's keys as soon as its
                    // warpgroup is through, half 1's behind them.
                    if (!mbar_wait(d64_bar(bar0, d64b::p_full + 2 * buf), (u >> 1) & 1, abort_flag, 341)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        if (ks < c0) mma_ts_lo(tB + 64, tB + 8 * ks, b_lo + ks * (2048 >> 4), idesc, ks > 0 ? 1u : 0u);
                    }
                    if (!mbar_wait(d64_bar(bar0, d64b::p_full + 2 * buf + 1), (u >> 1) & 1, abort_flag, 342)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t tP1 = tB + 256 - 16 * (nch - c0), b1_lo = b_lo + c0 * (2048 >> 4);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        if (ks < nch - c0) mma_ts_lo(tB + 64, tP1 + 8 * ks, b1_lo + ks * (2048 >> 4), idesc, 1u);
                    }
                    mma_commit(d64_bar(bar0, d64b::o_full + buf));
                }
                if (ok) mma_commit(d64_bar(bar0, d64b::v_empty + st));
            }
        } else if (warp == 17) {
            // ============================================================ Q and K loads
            tma_prefetch_desc(&tm_q);
            tma_prefetch_desc(&tm_k);
            D64StItem it;
            for (int ord = 0; d64st_item(p, n_qpairs, total_items, ord, it); ++ord) {
                const uint32_t st = ord & 1;
                const uint32_t sQ = sStage0 + st * kD64StStageBytes, sK = sQ + 2 * kD64TileBytes;
                const uint32_t bar = d64_bar(bar0, d64b::qk_full + st);
                // passes at once the first time each stage is used
                if (!mbar_wait(d64_bar(bar0, d64b::qk_empty + st), ((ord >> 1) & 1) ^ 1, abort_flag, 350)) break;
                mbar_expect_tx(bar, (2 + it.nq) * kD64TileBytes);   // rows past the end arrive as zeros
                tma_load_4d(sK, &tm_k, bar, 0, it.hk, 0, it.b);
                tma_load_4d(sK + kD64TileBytes, &tm_k, bar, 0, it.hk, kTile, it.b);
                tma_load_4d(sQ, &tm_q, bar, 0, it.h, it.q0, it.b);
                if (it.nq > 1) tma_load_4d(sQ + kD64TileBytes, &tm_q, bar, 0, it.h, it.q0 + kTile, it.b);
            }
        } else {
            // ============================================================ V loads
            tma_prefetch_desc(&tm_v);
            D64StItem it;
            for (int ord = 0; d64st_item(p, n_qpairs, total_items, ord, it); ++ord) {
                const uint32_t st = ord & 1;
                const uint32_t sV = sStage0 + st * kD64StStageBytes + 4 * kD64TileBytes;
                const uint32_t bar = d64_bar(bar0, d64b::v_full + st);
                if (!mbar_wait(d64_bar(bar0, d64b::v_empty + st), ((ord >> 1) & 1) ^ 1, abort_flag, 351)) break;
                mbar_expect_tx(bar, 2 * kD64TileBytes);
                tma_load_4d(sV, &tm_v, bar, 0, it.hk, 0, it.b);
                tma_load_4d(sV + kD64TileBytes, &tm_v, bar, 0, it.hk, kTile, it.b);
            }
        }
    }
    __syncwarp();

    tc_fence_before();
    __syncthreads();
    if (warp == 16) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

template <typename T>
int launch_d64_stream(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const FwdParams& fp,
                      cudaStream_t st, int* cuda_err) {
    auto kern = fa_fwd_d64_stream_kernel<T>;
    int sm_count = 0;
    if (int ce = prepare_big_smem_kernel(reinterpret_cast<const void*>(kern), kD64StSmem, &sm_count)) { *cuda_err = ce; return -7; }
    const int n_qpairs = (fp.n_qtiles + 1) / 2;
    const long long total = (long long)n_qpairs * fp.B * fp.Hq;
    if (total > 0x7fffffffll) return -3;
    const int grid = (int)(total < sm_count ? total : sm_count);
    kern<<<grid, kD64StThreads, kD64StSmem, st>>>(tq, tk, tv, fp, n_qpairs, (int)total);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { *cuda_err = (int)e; return -7; }
    return 0;
}

}  // namespace fa
