// Prefill forward, pipelined variant (the default kernel).
//
// A persistent CTA (one per SM, 384 threads) walks a static list of work items, longest
// first.  An item is a pair of adjacent 128-row query tiles of one (batch, head); K/V tiles
// of 128 keys stream through a 5-slot TMA ring shared by both query tiles.  Roles:
//   warpgroup 0 / 1 : softmax for query tile 0 / 1, one thread per row.  Reads S from tensor
//                     memory, keeps the running rowmax / rowsum, writes P (16-bit, packed)
//                     back over the columns S occupied, rescales O when the row max grew by
//                     more than 2^8, and at the end of an item normalises and stores O, LSE.
//   warp 8          : one thread issues every tcgen05.mma: S_t = Q_t K_j^T (operands in shared
//                     memory) and O_t += P_t V_j (P from tensor memory, V N-major from shared
//                     memory).  The S MMA for a tile's next step is issued right behind the
//                     PV MMA of its current step, so the tensor core works on one query tile
//                     while the other tile's softmax runs (the Cube/Vector overlap of
//                     Section 4.1 on this hardware), also across item boundaries.
//   warp 9          : one thread issues every TMA load.
// Tensor memory: columns [0,128) S_0/P_0, [128,256) S_1/P_1, [256,384) O_0, [384,512) O_1.
// Synchronisation is mbarrier-only; every wait is bounded (see mbar_wait).
#pragma once

#include <type_traits>

#include "prefill_simple.cuh"
#include "sm100_ptx.cuh"

namespace fa {

constexpr int kStages = 5;                  // K/V ring slots of one 128x128 16-bit tile each
constexpr int kPipeThreads = 384;
constexpr float kRescaleThreshold = 8.0f;   // in log2 units: P stays below 2^8

struct Item {
    int b, h, hk;
    int q0[2];   // first query row of the tile handled by role "tile 0" / "tile 1"
    int n[2];    // kv tiles each of them visits; they differ by at most one
};

// Decodes work item `idx` and assigns its two query tiles to the two tile roles.  Under the
// causal mask the upper tile visits one kv tile more than the lower one.  `lead` is how many
// steps role 0 is ahead of role 1 in the shared K/V ring (0 or 1): with no lead role 0 takes
// the shorter tile (and gains a step), with a lead it takes the longer one (and loses it), so
// both roles carry the same load and role 0 is never behind role 1.  Every warp role replays
// this sequence with its own copy of `lead`.
__device__ __forceinline__ Item decode_item(const FwdParams& p, int idx, int n_qpairs, int& lead) {
    Item it;
    const int bh_count = p.B * p.Hq;
    const int qp = n_qpairs - 1 - idx / bh_count;  // long (late) query tiles first
    const int bh = idx % bh_count;
    it.b = bh / p.Hq;
    it.h = bh % p.Hq;
    it.hk = it.h / (p.Hq / p.Hkv);
    const int q_lo = qp * 2 * kTile;
    const int n_lo = kv_tiles_for(q_lo, kTile, p.Sq, p.Skv, p.causal);
    // a second tile that starts past the last row still runs (on zero-filled rows, never
    // stored) so that both roles always have work in every item
    const int n_hi = (q_lo + kTile < p.Sq) ? kv_tiles_for(q_lo + kTile, kTile, p.Sq, p.Skv, p.causal) : n_lo;
    const int r_lo = lead ? 1 : 0;  // role that takes the lower (shorter) tile
    it.q0[r_lo] = q_lo;
    it.n[r_lo] = n_lo;
    it.q0[1 - r_lo] = q_lo + kTile;
    it.n[1 - r_lo] = n_hi;
    lead += lead ? -(n_hi - n_lo) : (n_hi - n_lo);
    return it;
}

// ---- softmax for one step of one query tile; `s` holds this thread's row of S (raw scores)
template <typename T, bool kMasked>
__device__ __forceinline__ void softmax_step(uint32_t (&s)[128], uint32_t tS, uint32_t tO, float scale_log2,
                                             int lim, bool first, float& m_ref, float& l_run) {
    // row max over the visible columns
    float mx;
    if (kMasked) {
        mx = -INFINITY;
#pragma unroll
        for (int i = 0; i < 128; ++i)
            if (i < lim) mx = fmaxf(mx, __uint_as_float(s[i]));
    } else {
        float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
        for (int i = 0; i < 128; i += 8) {
            m0 = max3(m0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
            m1 = max3(m1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
            m2 = max3(m2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
            m3 = max3(m3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
        }
        mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
    }
    // lazy reference update: move the reference max only when the row max outgrew it by more
    // than the threshold; O and l then carry the same (stale) reference, so O / l is exact
    bool grow = first ? true : ((mx - m_ref) * scale_log2 > kRescaleThreshold);
    if (mx == -INFINITY) grow = false;  // nothing visible in this tile for this row
    float alpha = 1.f;
    if (grow) {
        alpha = (m_ref == -INFINITY) ? 0.f : fast_exp2((m_ref - mx) * scale_log2);
        m_ref = mx;
    }
    if (!first && __any_sync(0xffffffffu, grow)) {
        // O_t holds every P V issued so far: the S MMA we just waited for was committed after them
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld_x32(tO + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st_x32(tO + c * 32, r);
        }
    }
    l_run *= alpha;
    const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
    const float neg_ms = -m_use * scale_log2;
    if (kMasked) {
        float l0 = 0.f, l1 = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const int e = c * 32 + i;
                float p0 = fast_exp2(fmaf(__uint_as_float(s[e]), scale_log2, neg_ms));
                float p1 = fast_exp2(fmaf(__uint_as_float(s[e + 1]), scale_log2, neg_ms));
                p0 = (e < lim) ? p0 : 0.f;  // exact zeros whatever the scale
                p1 = (e + 1 < lim) ? p1 : 0.f;
                l0 += p0;
                l1 += p1;
                pk[i / 2] = pack2<T>(p0, p1);
            }
            tmem_st_x16(tS + c * 16, pk);
        }
        l_run += l0 + l1;
    } else {
        // packed f32x2 arithmetic: one FMA and one add per pair of columns
        const uint64_t sc2 = f2_pack(scale_log2, scale_log2), nm2 = f2_pack(neg_ms, neg_ms);
        uint64_t la = f2_pack(0.f, 0.f), lb = la;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
                const int e = c * 32 + i;
                const uint64_t x01 = f2_fma(f2_pack(__uint_as_float(s[e]), __uint_as_float(s[e + 1])), sc2, nm2);
                const uint64_t x23 = f2_fma(f2_pack(__uint_as_float(s[e + 2]), __uint_as_float(s[e + 3])), sc2, nm2);
                float x0, x1, x2, x3;
                f2_unpack(x01, x0, x1);
                f2_unpack(x23, x2, x3);
                const float p0 = fast_exp2(x0), p1 = fast_exp2(x1), p2 = fast_exp2(x2), p3 = fast_exp2(x3);
                la = f2_add(la, f2_pack(p0, p1));
                lb = f2_add(lb, f2_pack(p2, p3));
                pk[i / 2] = pack2<T>(p0, p1);
                pk[i / 2 + 1] = pack2<T>(p2, p3);
            }
            tmem_st_x16(tS + c * 16, pk);
        }
        float a0, a1, b0, b1;
        f2_unpack(la, a0, a1);
        f2_unpack(lb, b0, b1);
        l_run += (a0 + a1) + (b0 + b1);
    }
}

template <typename T>
__global__ void __launch_bounds__(kPipeThreads, 1)
fa_fwd_pipelined_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                        const __grid_constant__ CUtensorMap tm_v, const FwdParams p, const int total_items,
                        const int n_qpairs) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;                      // 2 tiles
    const uint32_t sKV = smem_base + 2 * kTileBytes;    // kStages tiles
    __shared__ __align__(8) uint64_t bars[4 + 2 * kStages + 6];
    __shared__ uint32_t tmem_holder;
    __shared__ volatile uint32_t abort_flag;

    const uint32_t bar0 = smem_u32(&bars[0]);
    auto q_full = [&](int t) { return bar0 + 8 * t; };
    auto q_empty = [&](int t) { return bar0 + 8 * (2 + t); };
    auto kv_full = [&](int s) { return bar0 + 8 * (4 + s); };
    auto kv_empty = [&](int s) { return bar0 + 8 * (4 + kStages + s); };
    auto s_full = [&](int t) { return bar0 + 8 * (4 + 2 * kStages + t); };
    auto p_full = [&](int t) { return bar0 + 8 * (6 + 2 * kStages + t); };
    auto o_final = [&](int t) { return bar0 + 8 * (8 + 2 * kStages + t); };

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;

    if (tid == 0) {
        for (int i = 0; i < 4 + 2 * kStages + 6; ++i) {
            const bool is_p_full = (i == 6 + 2 * kStages) || (i == 7 + 2 * kStages);
            mbar_init(bar0 + 8 * i, is_p_full ? 4 : 1);  // p_full: one arrival per softmax warp
        }
        abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 8) {
        tmem_alloc(smem_u32(&tmem_holder), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;
    const int off = p.Skv - p.Sq;
    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;

    if (warp < 8) {
        // ================================================================ softmax + epilogue
        setmaxnreg_inc<224>();  // a whole row of S lives in registers
        const int t = warp >> 2;                    // query tile of this warpgroup
        const int r_in_tile = tid & 127;
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + lane_sel + t * 128;
        const uint32_t tO = tmem_base + lane_sel + 256 + t * 128;
        uint32_t ph_s = 0, ph_o = 0;
        bool ok = true;
        int lead = 0;
        for (int idx = blockIdx.x; idx < total_items && ok; idx += gridDim.x) {
            const Item it = decode_item(p, idx, n_qpairs, lead);
            const int n = it.n[t];
            const int q0 = it.q0[t];
            const int row = q0 + r_in_tile;
            float m_ref = -INFINITY, l_run = 0.f;
            for (int j = 0; j < n; ++j) {
                ok = mbar_wait(s_full(t), ph_s, &abort_flag, 10 + t);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                ph_s ^= 1;
                tc_fence_after();
                uint32_t s[128];
                tmem_ld_x32(tS, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
                tmem_ld_x32(tS + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
                tmem_ld_x32(tS + 64, *reinterpret_cast<uint32_t(*)[32]>(&s[64]));
                tmem_ld_x32(tS + 96, *reinterpret_cast<uint32_t(*)[32]>(&s[96]));
                tmem_wait_ld();
                const int kv0 = j * kTile;
                const bool need_mask = (p.causal && kv0 + kTile - 1 > q0 + off) || (kv0 + kTile > p.Skv);
                if (need_mask) {
                    int lim = p.Skv - kv0;
                    if (p.causal) lim = min(lim, row + off - kv0 + 1);
                    softmax_step<T, true>(s, tS, tO, p.scale_log2, lim, j == 0, m_ref, l_run);
                } else {
                    softmax_step<T, false>(s, tS, tO, p.scale_log2, 128, j == 0, m_ref, l_run);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(t));
            }
            if (!ok) break;
            // ---- epilogue of this item for tile t
            ok = mbar_wait(o_final(t), ph_o, &abort_flag, 12 + t);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            ph_o ^= 1;
            tc_fence_after();
            const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
            const bool live = row < p.Sq;
            const long long obase = (long long)it.b * p.o_sb + (long long)row * p.o_ss + (long long)it.h * p.o_sh;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
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
                const float lse = (l_run > 0.f) ? (m_ref * p.scale_log2 + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
                p.lse[((long long)it.b * p.Hq + it.h) * p.Sq + row] = lse;
            }
            // the next item's first P V (accumulate off) is only issued after this warp's next
            // p_full arrival, i.e. after these reads of O
            tc_fence_before();
        }
    } else {
        setmaxnreg_dec<56>();
    }
    if (warp == 8) {
        // ================================================================ MMA issue
        if (lane == 0) {
            constexpr uint32_t idesc_qk = instr_desc_f16(kBf16, 128, 128, false, false);
            constexpr uint32_t idesc_pv = instr_desc_f16(kBf16, 128, 128, false, true);
            struct Cursor {
                int idx;       // work item index (global)
                int ord;       // ordinal of the item in this CTA's sequence
                int lead;      // this cursor's replay of the role assignment
                int j, n;      // step within the item, steps of this role's tile
                int n_other;   // steps of the other role's tile in the same item
                uint32_t base; // ring index of the item's K_0
                bool valid;
            } cur[2];
            bool ok = true;
            auto load_item = [&](Cursor& c, int t) {
                c.valid = c.idx < total_items;
                if (c.valid) {
                    const Item it = decode_item(p, c.idx, n_qpairs, c.lead);
                    c.n = it.n[t];
                    c.n_other = it.n[1 - t];
                    c.j = 0;
                }
            };
            for (int t = 0; t < 2; ++t) {
                cur[t].idx = blockIdx.x;
                cur[t].ord = 0;
                cur[t].lead = 0;
                cur[t].base = 0;
                load_item(cur[t], t);
            }
            uint32_t ph_p[2] = {0, 0};
            auto issue_s = [&](int t) {
                Cursor& c = cur[t];
                if (c.j == 0) ok = ok && mbar_wait(q_full(t), c.ord & 1, &abort_flag, 30 + t);
                const uint32_t g = c.base + 2 * c.j;
                const uint32_t slot = g % kStages;
                ok = ok && mbar_wait(kv_full(slot), (g / kStages) & 1, &abort_flag, 32 + t);
                if (!ok) return;
                tc_fence_after();
                const uint32_t a0 = sQ + t * kTileBytes, b0 = sKV + slot * kTileBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t koff = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                    mma_ss(tmem_base + t * 128, smem_desc_sw128(a0 + koff, 16, 1024),
                           smem_desc_sw128(b0 + koff, 16, 1024), idesc_qk, ks > 0);
                }
                mma_commit(s_full(t));
                // role 1 trails role 0 in ring order, so it is the last reader of every entry it
                // reads; role 0 frees the entries role 1 never reads
                if (t == 1 || c.j >= c.n_other) mma_commit(kv_empty(slot));
                if (c.j == c.n - 1) mma_commit(q_empty(t));     // Q_t of this item is no longer needed
            };
            auto issue_pv = [&](int t) {
                Cursor& c = cur[t];
                const uint32_t g = c.base + 2 * c.j + 1;
                const uint32_t slot = g % kStages;
                ok = ok && mbar_wait(kv_full(slot), (g / kStages) & 1, &abort_flag, 34 + t);
                if (!ok) return;
                tc_fence_after();
                const uint32_t b0 = sKV + slot * kTileBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ts(tmem_base + 256 + t * 128, tmem_base + t * 128 + ks * 8,
                           smem_desc_sw128(b0 + ks * 2048, kHalfBytes, 1024), idesc_pv, (c.j > 0) || (ks > 0));
                if (t == 1 || c.j >= c.n_other) mma_commit(kv_empty(slot));
                if (c.j == c.n - 1) mma_commit(o_final(t));
            };
            if (cur[0].valid) issue_s(0);
            if (cur[1].valid) issue_s(1);
            while (ok && (cur[0].valid || cur[1].valid)) {
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    Cursor& c = cur[t];
                    if (!c.valid || !ok) continue;
                    ok = mbar_wait(p_full(t), ph_p[t], &abort_flag, 36 + t);
                    if (!ok) break;
                    ph_p[t] ^= 1;
                    issue_pv(t);
                    // advance this tile to its next step, possibly in the next item
                    if (++c.j == c.n) {
                        c.base += 2 * max(c.n, c.n_other);
                        c.idx += gridDim.x;
                        c.ord += 1;
                        load_item(c, t);
                    }
                    if (c.valid && ok) issue_s(t);
                }
            }
        }
        __syncwarp();
    } else if (warp == 9) {
        // ================================================================ TMA loads
        if (lane == 0) {
            tma_prefetch_desc(&tm_q);
            tma_prefetch_desc(&tm_k);
            tma_prefetch_desc(&tm_v);
            uint32_t g = 0;
            int ord = 0, lead = 0;
            bool ok = true;
            for (int idx = blockIdx.x; idx < total_items && ok; idx += gridDim.x, ++ord) {
                const Item it = decode_item(p, idx, n_qpairs, lead);
                const int n_kv = max(it.n[0], it.n[1]);
                const uint32_t q_par = (ord & 1) ^ 1;  // passes at once the first time
                ok = mbar_wait(q_empty(0), q_par, &abort_flag, 50);
                if (!ok) break;
                mbar_expect_tx(q_full(0), kTileBytes);
                load_tile(sQ, &tm_q, q_full(0), it.h, it.q0[0], it.b);
                for (int j = 0; j < n_kv && ok; ++j) {
                    for (int kv = 0; kv < 2 && ok; ++kv, ++g) {
                        const uint32_t slot = g % kStages;
                        ok = mbar_wait(kv_empty(slot), ((g / kStages) & 1) ^ 1, &abort_flag, 52 + kv);
                        if (!ok) break;
                        mbar_expect_tx(kv_full(slot), kTileBytes);
                        load_tile(sKV + slot * kTileBytes, kv ? &tm_v : &tm_k, kv_full(slot), it.hk, j * kTile, it.b);
                        if (j == 0 && kv == 0) {
                            // Q of role 1 goes after K_0 so that role 0 can start the item while
                            // role 1 still finishes the previous one
                            ok = mbar_wait(q_empty(1), q_par, &abort_flag, 51);
                            if (!ok) break;
                            mbar_expect_tx(q_full(1), kTileBytes);
                            load_tile(sQ + kTileBytes, &tm_q, q_full(1), it.h, it.q0[1], it.b);
                        }
                    }
                }
            }
        }
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

template <typename T>
int launch_pipelined(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const FwdParams& fp,
                     cudaStream_t st, int* cuda_err) {
    constexpr int smem = 1024 + (2 + kStages) * kTileBytes;
    auto kern = fa_fwd_pipelined_kernel<T>;
    static int sm_count = 0;
    cudaError_t e;
    if (sm_count == 0) {
        int dev = 0, n = 0;
        if ((e = cudaGetDevice(&dev)) != cudaSuccess) { *cuda_err = (int)e; return -7; }
        if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) { *cuda_err = (int)e; return -7; }
        if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)) != cudaSuccess) { *cuda_err = (int)e; return -7; }
        sm_count = n;
    }
    const int n_qpairs = (fp.n_qtiles + 1) / 2;
    const long long total = (long long)n_qpairs * fp.B * fp.Hq;
    if (total > 0x7fffffffll) return -3;
    const int grid = (int)(total < sm_count ? total : sm_count);
    kern<<<grid, kPipeThreads, smem, st>>>(tq, tk, tv, fp, (int)total, n_qpairs);
    e = cudaGetLastError();
    if (e != cudaSuccess) { *cuda_err = (int)e; return -7; }
    return 0;
}

}  // namespace fa
