// Prefill forward, paired-tile pipelined variant (the library's choice below 1024 keys).
//
// A persistent CTA (one per SM, 384 threads) walks a static list of work items, longest
// first, in boustrophedon order over the CTAs.  An item is a pair of adjacent 128-row query
// tiles of one (batch, head); K/V tiles of 128 keys stream through a 5-slot TMA ring shared by
// both query tiles.  The two tiles are handled by two "tile roles":
//   warpgroup 0 / 1 : softmax of role 0 / 1, one thread per query row.  Reads S from tensor
//                     memory, keeps the running rowmax / rowsum, writes P (16-bit, packed)
//                     back over the columns S occupied, rescales O when the row max grew by
//                     more than 2^8, and at the end of an item normalises and stores O, LSE.
//   warp 8 / 10     : one thread each issues the tcgen05.mma of role 0 / 1: S = Q K_j^T
//                     (operands in shared memory) and O += P V_j (P from tensor memory, V
//                     N-major from shared memory).  A role's round is "wait for P, issue P V,
//                     issue S of the role's next step", so the tensor core works on one role
//                     while the other role's softmax runs (the Cube/Vector overlap of
//                     Section 4.1 on this hardware), also across item boundaries.  The two
//                     threads pass a turn token so that their MMA batches alternate back to
//                     back while each thread's waits and commits overlap the other's batch.
//   warp 9          : one thread issues every TMA load.
// Under the causal mask the upper tile of a pair visits one kv tile more than the lower one;
// the roles swap which tile they take whenever role 0 is a step ahead, so both carry the same
// load and role 0 is never behind role 1 in the ring.
// Tensor memory: columns [0,128) S_0/P_0, [128,256) S_1/P_1, [256,384) O_0, [384,512) O_1.
// Synchronisation is mbarrier-only; every wait is bounded (see mbar_wait).
#pragma once

#include <type_traits>

#include "prefill_simple.cuh"
#include "sm100_ptx.cuh"

namespace fa {

constexpr int kStages = 5;                  // K/V ring slots of one 128x128 16-bit tile each
constexpr int kPipeThreads = 384;
// Register reallocation (setmaxnreg moves registers between warpgroups of the CTA only; an
// increase that the other warpgroups' decrease does not cover would wait forever).
constexpr int kPipeLaunchRegs = (65536 / kPipeThreads) & ~7;  // 168
constexpr int kPipeSoftmaxRegs = 224, kPipeOtherRegs = 56;
static_assert(256 * (kPipeSoftmaxRegs - kPipeLaunchRegs) <= 128 * (kPipeLaunchRegs - kPipeOtherRegs),
              "setmaxnreg.inc would wait for registers nobody releases");
constexpr float kRescaleThreshold = 8.0f;   // in log2 units: P stays below 2^8

// Work item taken by this CTA in its k-th round.  Items are listed longest first; rounds
// alternate direction across the CTAs (boustrophedon) so that every CTA gets nearly the same
// total length.  Returns a value >= total_items when the CTA has no k-th item.
__device__ __forceinline__ int item_of_round(int k, int total_items) {
    const int g = gridDim.x, b = blockIdx.x;
    return k * g + ((k & 1) ? (g - 1 - b) : b);
}

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
    // Item order.  Normally the longest (last) query tile pairs of all heads come first, which
    // balances the CTAs best.  When one head alone has at least one round of items for every
    // CTA (very long sequences, whose K and V per head no longer fit in L2), the list goes head
    // by head instead: all CTAs then walk the same head's K/V at about the same pace and share
    // it through L2 rather than each streaming its own head from HBM.
    const bool head_major = n_qpairs >= (int)gridDim.x;
    int major, minor;  // idx = major * (inner count) + minor
    if (head_major) p.by_qpairs.divmod(idx, major, minor);
    else p.by_bh.divmod(idx, major, minor);
    const int qp = n_qpairs - 1 - (head_major ? minor : major);  // long (late) tiles first
    const int bh = head_major ? major : minor;
    p.by_hq.divmod(bh, it.b, it.h);
    it.hk = p.by_group.div(it.h);
    const int q_lo = qp * 2 * kTile;
    const int n_lo = kv_tiles_for(q_lo, kTile, p.Sq, p.Skv, p.causal);
    // a second tile that starts past the last row still runs (on zero-filled rows, never
    // stored) so that both roles always have work in every item
    const int n_hi = (q_lo + kTile < p.Sq) ? kv_tiles_for(q_lo + kTile, kTile, p.Sq, p.Skv, p.causal) : n_lo;
    const bool swap = lead != 0;  // role 0 takes the upper (longer) tile when it is a step ahead
    it.q0[0] = swap ? q_lo + kTile : q_lo;
    it.n[0] = swap ? n_hi : n_lo;
    it.q0[1] = swap ? q_lo : q_lo + kTile;
    it.n[1] = swap ? n_lo : n_hi;
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
            for (int i = 0; i < 32; i += 8) {
                const int e = c * 32 + i;
                float pv[8];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const uint64_t x01 =
                        f2_fma(f2_pack(__uint_as_float(s[e + 2 * q]), __uint_as_float(s[e + 2 * q + 1])), sc2, nm2);
                    float x0, x1;
                    f2_unpack(x01, x0, x1);
                    pv[2 * q] = fast_exp2(x0);
                    pv[2 * q + 1] = fast_exp2(x1);
                }
                la = f2_add(la, f2_pack(pv[0], pv[1]));
                lb = f2_add(lb, f2_pack(pv[2], pv[3]));
                la = f2_add(la, f2_pack(pv[4], pv[5]));
                lb = f2_add(lb, f2_pack(pv[6], pv[7]));
#pragma unroll
                for (int q = 0; q < 4; ++q) pk[i / 2 + q] = pack2<T>(pv[2 * q], pv[2 * q + 1]);
            }
            tmem_st_x16(tS + c * 16, pk);
        }
        float a0, a1, b0, b1;
        f2_unpack(la, a0, a1);
        f2_unpack(lb, b0, b1);
        l_run += (a0 + a1) + (b0 + b1);
    }
}

// ---- barrier addresses (shared by all roles): byte offsets from the first barrier
__device__ __forceinline__ uint32_t bar_q_full(uint32_t b0, int t) { return b0 + 8 * t; }
__device__ __forceinline__ uint32_t bar_q_empty(uint32_t b0, int t) { return b0 + 8 * (2 + t); }
__device__ __forceinline__ uint32_t bar_kv_full(uint32_t b0, uint32_t s) { return b0 + 8 * (4 + s); }
__device__ __forceinline__ uint32_t bar_kv_empty(uint32_t b0, uint32_t s) { return b0 + 8 * (4 + kStages + s); }
__device__ __forceinline__ uint32_t bar_s_full(uint32_t b0, int t) { return b0 + 8 * (4 + 2 * kStages + t); }
__device__ __forceinline__ uint32_t bar_p_full(uint32_t b0, int t) { return b0 + 8 * (6 + 2 * kStages + t); }
__device__ __forceinline__ uint32_t bar_o_final(uint32_t b0, int t) { return b0 + 8 * (8 + 2 * kStages + t); }
__device__ __forceinline__ uint32_t bar_turn(uint32_t b0, int t) { return b0 + 8 * (10 + 2 * kStages + t); }
constexpr int kNumBars = 12 + 2 * kStages;

// High word shared by every shared-memory operand descriptor used here: SBO = 1024 bytes,
// version 1, 128-byte swizzle.  The low word carries the address and the leading offset, so a
// k-step only adds a constant to it.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
    return ((saddr & 0x3ffffu) >> 4) | ((lbo_bytes >> 4) << 16);
}
__device__ __forceinline__ void mma_ss_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
        : "memory");
}
__device__ __forceinline__ void mma_ts_lo(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
        : "memory");
}
// The same two forms for FP8 operands (kind::f8f6f4).
__device__ __forceinline__ void mma_ss_lo_f8(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], da, db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
        : "memory");
}
__device__ __forceinline__ void mma_ts_lo_f8(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], db, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
        : "memory");
}

// The single thread that issues every tcgen05.mma of the CTA.  It keeps one cursor per tile
// role; a round is: wait for the role's P, issue its O += P V, then issue S for the role's
// next step (possibly of the next item).  All state lives in registers.
template <typename T>
struct MmaIssuer {
    uint32_t bar0, sQ, sKV, tmem;
    volatile uint32_t* abort_flag;

    struct Cursor {
        int idx, ord, lead;   // work item, its ordinal in this CTA's sequence, role-assignment replay
        int j, n, n_other;    // step, steps of this role's tile, steps of the other role's tile
        uint32_t slot, par;   // ring slot / parity of this step's K entry (V is the next entry)
        bool valid;
    };
    static constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
    static constexpr uint32_t kIdescQK = instr_desc_f16(kBf16, 128, 128, false, false);
    static constexpr uint32_t kIdescPV = instr_desc_f16(kBf16, 128, 128, false, true);

    __device__ __forceinline__ static void ring_add(uint32_t& slot, uint32_t& par, uint32_t k) {
        slot += k;  // k < kStages
        if (slot >= kStages) {
            slot -= kStages;
            par ^= 1;
        }
    }
    template <int t>
    __device__ __forceinline__ void load_item(Cursor& c, const FwdParams& p, int total_items, int n_qpairs) {
        c.valid = c.idx < total_items;
        if (c.valid) {
            const Item it = decode_item(p, c.idx, n_qpairs, c.lead);
            c.n = it.n[t];
            c.n_other = it.n[1 - t];
            c.j = 0;
        }
    }
    // S = Q K^T for the step the cursor points at (operands already waited for)
    template <int t>
    __device__ __forceinline__ void mma_s(const Cursor& c) {
        const uint32_t a_lo = desc_lo(sQ + t * kTileBytes, 16);
        const uint32_t b_lo = desc_lo(sKV + c.slot * kTileBytes, 16);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint32_t koff = ((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4;
            mma_ss_lo(tmem + t * 128, a_lo + koff, b_lo + koff, kIdescQK, ks > 0 ? 1u : 0u);
        }
        mma_commit(bar_s_full(bar0, t));
    }
    // Commits that only free resources; they go after the turn has been handed over.
    // A ring slot is free once both roles' MMAs on it are done: each reader commits one arrival,
    // and the only reader of an entry the other role never visits commits both.
    template <int t>
    __device__ __forceinline__ void release_s(const Cursor& c) {
        mma_commit(bar_kv_empty(bar0, c.slot));
        if (c.j >= c.n_other) mma_commit(bar_kv_empty(bar0, c.slot));
        if (c.j == c.n - 1) mma_commit(bar_q_empty(bar0, t));  // Q of this item is no longer needed
    }
    template <int t>
    __device__ __forceinline__ bool wait_s_operands(const Cursor& c) {
        if (c.j == 0 && !mbar_wait(bar_q_full(bar0, t), c.ord & 1, abort_flag, 30 + t)) return false;
        return mbar_wait(bar_kv_full(bar0, c.slot), c.par, abort_flag, 32 + t);
    }
    // One round of a role: O += P V for the current step, then S for the next step (possibly of
    // the next item).  Everything that can be waited for in advance is waited for before the
    // role takes its turn on the tensor core; the turn passes to the other role right after the
    // MMAs and the S commit, so the two roles' MMA batches alternate back to back while each
    // role's bookkeeping overlaps the other's batch.
    template <int t>
    __device__ __forceinline__ bool round(Cursor& c, uint32_t& ph_p, uint32_t& turn_k, const FwdParams& p,
                                          int total_items, int n_qpairs) {
        uint32_t v_slot = c.slot, v_par = c.par;
        ring_add(v_slot, v_par, 1);
        if (!mbar_wait(bar_kv_full(bar0, v_slot), v_par, abort_flag, 34 + t)) return false;
        Cursor nx = c;  // the role's next step
        ring_add(nx.slot, nx.par, 2);
        if (++nx.j == nx.n) {  // next item: skip the entries only the other role reads
            if (nx.n_other > nx.n) ring_add(nx.slot, nx.par, 2);
            nx.ord += 1;
            nx.idx = item_of_round(nx.ord, total_items);
            load_item<t>(nx, p, total_items, n_qpairs);
        }
        if (nx.valid && !wait_s_operands<t>(nx)) return false;
        if (!mbar_wait(bar_p_full(bar0, t), ph_p, abort_flag, 36 + t)) return false;
        ph_p ^= 1;
        if (!mbar_wait(bar_turn(bar0, t), (turn_k & 1) ^ (t == 0 ? 1u : 0u), abort_flag, 38 + t)) return false;
        ++turn_k;
        tc_fence_after();
        const uint32_t b_lo = desc_lo(sKV + v_slot * kTileBytes, kHalfBytes);  // V: N-major, 16 kv rows per step
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
            mma_ts_lo(tmem + 256 + t * 128, tmem + t * 128 + ks * 8, b_lo + ks * (2048 >> 4), kIdescPV,
                      (ks > 0) ? 1u : (c.j > 0 ? 1u : 0u));
        if (nx.valid) mma_s<t>(nx);
        mbar_arrive(bar_turn(bar0, 1 - t));
        // bookkeeping, off the other role's critical path
        mma_commit(bar_kv_empty(bar0, v_slot));
        if (c.j >= c.n_other) mma_commit(bar_kv_empty(bar0, v_slot));
        if (c.j == c.n - 1) mma_commit(bar_o_final(bar0, t));
        if (nx.valid) release_s<t>(nx);
        c = nx;
        return true;
    }
    // One issuing thread per role (they sit in different warps).  MMAs of one thread execute in
    // issue order, which is all the P/S aliasing needs; the two roles share the K/V ring and
    // the turn tokens.  Role 0 never has more rounds than role 1 and at most one fewer, so one
    // empty turn at its end keeps the token moving for role 1's last round.
    template <int t>
    __device__ __forceinline__ void run(const FwdParams& p, int total_items, int n_qpairs) {
        Cursor c;
        c.idx = item_of_round(0, total_items);
        c.ord = 0;
        c.lead = 0;
        c.slot = 0;
        c.par = 0;
        load_item<t>(c, p, total_items, n_qpairs);
        uint32_t ph = 0, turn_k = 0;
        bool ok = true;
        if (c.valid) {
            ok = wait_s_operands<t>(c);
            if (ok) {
                tc_fence_after();
                mma_s<t>(c);
                release_s<t>(c);
            }
        }
        while (ok && c.valid) ok = round<t>(c, ph, turn_k, p, total_items, n_qpairs);
        if (t == 0 && ok) {
            if (mbar_wait(bar_turn(bar0, 0), (turn_k & 1) ^ 1u, abort_flag, 40)) mbar_arrive(bar_turn(bar0, 1));
        }
    }
};

// The single thread that issues every TMA load of the CTA: per item Q of role 0, K_0, Q of
// role 1, V_0, K_1, V_1, ... through the K/V ring.
__device__ __forceinline__ void run_loader(uint32_t bar0, uint32_t sQ, uint32_t sKV, const CUtensorMap* tm_q,
                                           const CUtensorMap* tm_k, const CUtensorMap* tm_v, const FwdParams& p,
                                           int total_items, int n_qpairs, volatile uint32_t* abort_flag) {
        tma_prefetch_desc(tm_q);
        tma_prefetch_desc(tm_k);
        tma_prefetch_desc(tm_v);
        const uint64_t pol_q = l2_policy_evict_first(), pol_kv = l2_policy_evict_last();
        uint32_t g = 0;
        int ord = 0, lead = 0;
        bool ok = true;
        for (;; ++ord) {
            const int idx = item_of_round(ord, total_items);
            if (idx >= total_items || !ok) break;
            const Item it = decode_item(p, idx, n_qpairs, lead);
            const int n_kv = max(it.n[0], it.n[1]);
            const uint32_t q_par = (ord & 1) ^ 1;  // passes at once the first time
            ok = mbar_wait(bar_q_empty(bar0, 0), q_par, abort_flag, 50);
            if (!ok) break;
            mbar_expect_tx(bar_q_full(bar0, 0), kTileBytes);
            load_tile_hint(sQ, tm_q, bar_q_full(bar0, 0), it.h, it.q0[0], it.b, pol_q);
            for (int j = 0; j < n_kv && ok; ++j) {
                for (int kv = 0; kv < 2 && ok; ++kv, ++g) {
                    const uint32_t slot = g % kStages;
                    ok = mbar_wait(bar_kv_empty(bar0, slot), ((g / kStages) & 1) ^ 1, abort_flag, 52 + kv);
                    if (!ok) break;
                    mbar_expect_tx(bar_kv_full(bar0, slot), kTileBytes);
                    load_tile_hint(sKV + slot * kTileBytes, kv ? tm_v : tm_k, bar_kv_full(bar0, slot), it.hk, j * kTile, it.b, pol_kv);
                    if (j == 0 && kv == 0) {
                        // Q of role 1 goes after K_0 so that role 0 can start the item while
                        // role 1 still finishes the previous one
                        ok = mbar_wait(bar_q_empty(bar0, 1), q_par, abort_flag, 51);
                        if (!ok) break;
                        mbar_expect_tx(bar_q_full(bar0, 1), kTileBytes);
                        load_tile_hint(sQ + kTileBytes, tm_q, bar_q_full(bar0, 1), it.h, it.q0[1], it.b, pol_q);
                    }
                }
            }
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
    __shared__ __align__(8) uint64_t bars[kNumBars];
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
        for (int i = 0; i < kNumBars; ++i) {
            const bool is_p_full = (i == 6 + 2 * kStages) || (i == 7 + 2 * kStages);
            const bool is_kv_empty = (i >= 4 + kStages) && (i < 4 + 2 * kStages);
            // p_full: one arrival per softmax warp; kv_empty: one per reading role
            mbar_init(bar0 + 8 * i, is_p_full ? 4 : (is_kv_empty ? 2 : 1));
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

    if (warp < 8) {
        // ================================================================ softmax + epilogue
        setmaxnreg_inc<kPipeSoftmaxRegs>();  // a whole row of S lives in registers
        const int t = warp >> 2;                    // query tile of this warpgroup
        const int r_in_tile = tid & 127;
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tS = tmem_base + lane_sel + t * 128;
        const uint32_t tO = tmem_base + lane_sel + 256 + t * 128;
        uint32_t ph_s = 0, ph_o = 0;
        bool ok = true;
        int lead = 0;
        for (int k = 0; ok; ++k) {
            const int idx = item_of_round(k, total_items);
            if (idx >= total_items) break;
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
                    // tiles crossed by the diagonal or by the end of the keys: hidden scores
                    // become -inf (the scale is strictly positive, so they come out as exact
                    // zeros) and the tile then takes the common path
                    int lim = p.Skv - kv0;
                    if (p.causal) lim = min(lim, row + off - kv0 + 1);
#pragma unroll
                    for (int i = 0; i < 128; ++i)
                        if (i >= lim) s[i] = 0xff800000u;
                }
                softmax_step<T, false>(s, tS, tO, p.scale_log2, 128, j == 0, m_ref, l_run);
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
            if (!p.o_fp32 && p.o_align32) {
                // 16-bit output, rows 32-byte aligned: whole-line stores through a lane exchange
                uint32_t wv[64];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tmem_ld_x32(tO + c * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        wv[c * 16 + i] = pack2<T>(__uint_as_float(r[2 * i]) * inv_l, __uint_as_float(r[2 * i + 1]) * inv_l);
                }
                store_rows_coalesced<T>(static_cast<T*>(p.o) + obase, p.o_ss, p.Sq - (row - lane), wv);
            } else {
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
                            T* dst = static_cast<T*>(p.o) + obase + c * 32;
                            uint32_t w[16];
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                w[i] = pack2<T>(__uint_as_float(r[2 * i]) * inv_l, __uint_as_float(r[2 * i + 1]) * inv_l);
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                reinterpret_cast<uint4*>(dst)[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
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
        setmaxnreg_dec<kPipeOtherRegs>();
    }
    if (warp == 8 || warp == 10) {
        // ================================================================ MMA issue (role 0 / 1)
        if (lane == 0) {
            MmaIssuer<T> mi;
            mi.bar0 = bar0;
            mi.sQ = sQ;
            mi.sKV = sKV;
            mi.tmem = tmem_base;
            mi.abort_flag = &abort_flag;
            if (warp == 8) mi.template run<0>(p, total_items, n_qpairs);
            else mi.template run<1>(p, total_items, n_qpairs);
        }
        __syncwarp();
    } else if (warp == 9) {
        // ================================================================ TMA loads
        if (lane == 0) run_loader(bar0, sQ, sKV, &tm_q, &tm_k, &tm_v, p, total_items, n_qpairs, &abort_flag);
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
    int sm_count = 0;
    cudaError_t e;
    if (int ce = prepare_big_smem_kernel(reinterpret_cast<const void*>(kern), smem, &sm_count)) { *cuda_err = ce; return -7; }
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
