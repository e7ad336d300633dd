// Prefill forward, ping-pong variant.
//
// A persistent CTA (one per SM, 384 threads) walks a static list of work items; an item is one
// 128-row query tile of one (batch, head).  The kv steps of the CTA are numbered g = 0, 1, 2, ...
// across items, and everything a step needs is double-buffered on the parity of g:
//   tensor memory : O [0,128)   S_0 [128,256)  S_1 [256,384)  P_0 [384,448)  P_1 [448,512)
//   warpgroup g&1 : softmax of step g, one thread per query row: reads S_{g&1}, keeps its part
//                   of the row sum, writes P (16-bit, packed) to P_{g&1}.
//   warp 8        : one thread issues S_{g&1} = Q K_g^T for every step, as soon as K_g has
//                   landed and the softmax of step g-2 has read its scores out of the buffer.
//   warp 10       : one thread issues O += P_{g&1} V_g for every step, as soon as P is written.
//   warp 9 / 11   : one thread each issues the TMA loads of Q and K / of V (separate rings, as
//                   K is consumed about two steps ahead of V).
// Because P has columns of its own, Q K^T of step g+1 and g+2 run on the tensor core while the
// softmax of step g is still at work: the tensor core never waits for a softmax of the same
// tile (the Cube/Vector overlap of Section 4.1 within one query tile), and the two warpgroups
// give the exponentials two steps of time per step of tensor work.
//
// The online-softmax recurrence (Appendix A) is carried from step to step through shared
// memory: the warpgroup of step g takes the reference max left by step g-1, decides whether its
// own row max moves it (only when it outgrew it by more than 2^8, see kRescaleThreshold),
// publishes the result for step g+1 right away, and, in the rare case that it moved, rescales O
// once O += P V of step g-1 has completed.  Each warpgroup keeps the row sum of its own steps;
// the one that runs an item's last step adds the other's and writes O and LSE.
// Synchronisation is mbarrier-only; every wait is bounded (see mbar_wait).
#pragma once

#include <type_traits>

#include "prefill_pipelined.cuh"

namespace fa {

#ifndef FA_PP_NK
#define FA_PP_NK 3
#endif
#ifndef FA_PP_NV
#define FA_PP_NV 2
#endif
constexpr int kPpNK = FA_PP_NK;   // K ring slots
constexpr int kPpNV = FA_PP_NV;   // V ring slots
constexpr int kPpQBufs = 2;
static_assert((kPpQBufs + kPpNK + kPpNV) * kTileBytes + 3072 <= 232448, "shared memory budget");

// What changes with FP8 e4m3 operands (kF8; Appendix D.2 evaluates the operator with 8-bit
// operands): a tile of 128 rows x 128 bytes is one swizzled TMA box of 16 KiB (a Q slot keeps its
// 32 KiB, because the 16-bit output tile is staged there); one MMA covers 32 elements of the
// contraction, so a product takes four instead of eight; the probabilities are rounded to e4m3
// four to a 32-bit column of tensor memory, times kP8Scale so that they use the format's range:
// with the reference max at most 2^kP8Threshold behind the row max they stay below 2^8 < 448.
// Head dimension 64 (D; 16-bit operands only) has the same byte layout: a row of a Q, K or V tile
// is 64 elements = 128 bytes, one box; Q K^T then contracts over four MMAs of 16 elements, P V is
// eight MMAs of 16 keys with N = 64, and O takes 64 columns of tensor memory.
template <bool kF8, int D = 128>
struct PpOperands {
    static_assert(D == 128 || (D == 64 && !kF8), "head dimension 128, or 64 with 16-bit operands");
    static constexpr bool kOneBox = kF8 || D == 64;                     // a tile row is 128 bytes
    static constexpr int kKvSlotBytes = kOneBox ? 16384 : kTileBytes;   // one K or V ring slot
    static constexpr int kQBytes = kOneBox ? 16384 : kTileBytes;        // bytes a Q load delivers
    static constexpr int kSteps = kOneBox ? 4 : 8;                      // MMAs of Q K^T (32 bytes of every row each)
    static constexpr int kPvSteps = kF8 ? 4 : 8;                        // MMAs of P V (32 or 16 keys each)
    static constexpr int kPCols = kF8 ? 8 : 16;                         // tensor-memory columns of 32 probabilities
};
constexpr float kP8Threshold = 4.0f;   // log2 units: how far the row max may outgrow the reference (FP8)
constexpr float kP8ScaleLog2 = 4.0f;   // log2 of the factor on the FP8 probabilities

// ---- barriers: indices into one array
namespace ppb {
constexpr int q_full = 0;                       // [2]  TMA -> S thread
constexpr int q_empty = 2;                      // [2]  S thread (commit) -> loader; with the output staged in the
                                                //      Q buffer, the four epilogue warps (count 4) -> loader
constexpr int k_full = 4;                       // [NK]
constexpr int k_empty = k_full + kPpNK;         // [NK]
constexpr int v_full = k_empty + kPpNK;         // [NV]
constexpr int v_empty = v_full + kPpNV;         // [NV]
constexpr int s_full = v_empty + kPpNV;         // [2]  S thread (commit) -> softmax
constexpr int pv_done = s_full + 2;             // [2]  PV thread (commit) -> softmax
constexpr int o_final = pv_done + 2;            // [2]  PV thread (commit) -> epilogue, by item parity
// barriers every thread of a softmax warpgroup arrives on (count 128)
constexpr int p_full = o_final + 2;             // [2]  softmax -> PV thread
constexpr int m_ready = p_full + 2;             // [2]  softmax of step g -> softmax of step g+1 (reference max
                                                //      published) and -> S thread (scores read out of S_{g&1})
constexpr int l_pub = m_ready + 2;              // [2]  softmax of an item's last-but-one step -> of its last step
constexpr int o_free = l_pub + 2;               // [1]  epilogue -> PV thread
constexpr int count = o_free + 1;
}  // namespace ppb

struct PpStatic {
    uint64_t bars[ppb::count];
    uint32_t tmem_holder;
    uint32_t abort_flag;
    float m_xch[2][128];   // [warpgroup][row]: reference max after that warpgroup's latest step
    float l_xch[2][128];   // [item parity][row]: row sum of the warpgroup that does not run the last step
    uint8_t pad[3072 - ppb::count * 8 - 8 - 4 * 128 * 4];
};
static_assert(sizeof(PpStatic) == 3072, "static shared state must fill exactly 3 KiB");

struct PpItem {
    int b, h, hk, q0, n;
    // packed variable-length batches only: first row of the sequence in q/o and in k/v, and
    // the sequence's own lengths
    int q_base, k_base, Sq, Skv;
    int page0;   // paged K/V: the sequence's first table entry (-1 for a sequence without keys)
};

// Work item `idx`.  The query tiles of a head are taken in classes of C = 2^cls_log2 consecutive
// tiles, the class of the last (longest) tiles first; inside a class the items go head by head,
// a head's tiles longest first.  With the items dealt to the CTAs round by round, a round then
// works on about gridDim.x / C heads, whose K and V stay in L2 while the C tiles of each head
// read them, and the rounds still get shorter and shorter items, which keeps the static
// assignment balanced (the launcher picks C from the K/V bytes of a head, see launch_pingpong).
// C >= n_qtiles is the plain head-by-head order used for very long sequences.
// kVarlen: the sequence's lengths come from the prefix sums; n == 0 marks an item past the end
// of its sequence (every role skips it), and a live item visits at least one kv tile (so that
// rows without any visible key are still written, as zeros).
template <bool kVarlen>
__device__ __forceinline__ void pp_class_order(const FwdParams& p, int idx, int& bh, int& qt) {
    int c, rem;  // class, index inside the class
    p.by_class.divmod(idx, c, rem);
    const int first = c << p.cls_log2;  // tiles in the classes before this one
    int j;
    if (p.n_qtiles - first >= (1 << p.cls_log2)) {
        bh = rem >> p.cls_log2;
        j = rem & ((1 << p.cls_log2) - 1);
    } else {
        p.by_lastcls.divmod(rem, bh, j);
    }
    qt = p.n_qtiles - 1 - first - j;
}

// The work item that is query tile qt of (batch, head) pair bh.
template <bool kVarlen>
__device__ __forceinline__ PpItem pp_decode_item(const FwdParams& p, int bh, int qt) {
    PpItem it;
    p.by_hq.divmod(bh, it.b, it.h);
    it.hk = p.by_group.div(it.h);
    it.q0 = qt * kTile;
    if (kVarlen) {
        it.q_base = p.cu_q[it.b];
        it.Sq = p.cu_q[it.b + 1] - it.q_base;
        if (p.block_table) {   // paged K/V: the keys are reached through the table
            it.k_base = 0;
            // the first table entry is fetched together with the lengths, so that a loader does
            // not start an item with two dependent global loads (the entry exists for every
            // sequence; its value is ignored when the sequence has no keys)
            const int first_page = __ldg(p.block_table + (long long)it.b * p.table_stride);
            it.Skv = p.seqlens_k[it.b];
            it.page0 = it.Skv > 0 ? first_page : -1;
        } else {
            it.k_base = p.cu_k[it.b];
            it.Skv = p.cu_k[it.b + 1] - it.k_base;
        }
        it.n = (it.q0 < it.Sq) ? max(1, kv_tiles_for(it.q0, kTile, it.Sq, it.Skv, p.causal)) : 0;
    } else {
        it.n = kv_tiles_for(it.q0, kTile, p.Sq, p.Skv, p.causal);
    }
    return it;
}

// The items of this CTA in order.  `ord` counts the items the CTA works on (it selects the
// double buffers); with variable-length batches the items past the end of their sequence are
// passed over, identically in every role.
// Very long sequences (rounds_per_head > 0; one head's K and V no longer fit in L2) go head by
// head, and every head takes a whole number of rounds of the grid: in round r of a head CTA b
// takes the head's (r * gridDim.x + b)-th longest tile -- b counted from the other end in every
// second round, and the other way around for every second head -- and nothing if the head has no
// such tile (only in a head's last round, whose items are its shortest).  The CTAs of a round
// then all walk the same head's keys from the first on, a few dozen tiles apart at most, and
// stay together from head to head, so a K or V tile is fetched from HBM once per round and
// found in L2 by everyone else.  (Without the padding a round straddles two heads, the CTAs
// that get the next head's longest tiles fall a thousand tiles behind the others, and the
// groups, each walking the head on its own, fetch everything several times.)
template <bool kVarlen>
struct PpItems {
    int round = -1, ord = -1;
    PpItem it;
    __device__ __forceinline__ bool next(const FwdParams& p, int total_items) {
        for (;;) {
            ++round;
            if (!kVarlen && p.rounds_per_head > 0) {
                int bh, r;
                p.by_rph.divmod(round, bh, r);
                if (bh >= p.B * p.Hq) return false;
                const int g = gridDim.x, b = blockIdx.x;
                const int j = r * g + (((r + bh) & 1) ? (g - 1 - b) : b);
                if (j >= p.n_qtiles) continue;
                it = pp_decode_item<kVarlen>(p, bh, p.n_qtiles - 1 - j);
                ++ord;
                return true;
            }
            const int idx = item_of_round(round, total_items);
            if (idx >= total_items) return false;
            int bh, qt;
            pp_class_order<kVarlen>(p, idx, bh, qt);
            it = pp_decode_item<kVarlen>(p, bh, qt);
            if (!kVarlen || it.n > 0) {
                ++ord;
                return true;
            }
        }
    }
};

// Row max of 128 raw scores.
__device__ __forceinline__ float pp_row_max(const uint32_t (&s)[128]) {
    float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
    for (int i = 0; i < 128; i += 8) {
        m0 = max3(m0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
        m1 = max3(m1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
        m2 = max3(m2, __uint_as_float(s[i + 4]), __uint_as_float(s[i + 5]));
        m3 = max3(m3, __uint_as_float(s[i + 6]), __uint_as_float(s[i + 7]));
    }
    return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

// exp2(s * scale_log2 + neg_ms) of 32 scores -> 16 packed 16-bit pairs; adds them to (la, lb).
template <typename T, bool kF8>
__device__ __forceinline__ void pp_exp_chunk(const uint32_t (&s)[128], int c, uint64_t sc2, uint64_t nm2,
                                             uint64_t& la, uint64_t& lb, uint32_t (&pk)[PpOperands<kF8>::kPCols]) {
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
        if (kF8) {
            pk[i / 4] = pack4_e4m3(pv[0], pv[1], pv[2], pv[3]);
            pk[i / 4 + 1] = pack4_e4m3(pv[4], pv[5], pv[6], pv[7]);
        } else {
#pragma unroll
            for (int q = 0; q < 4; ++q) pk[i / 2 + q] = pack2<T>(pv[2 * q], pv[2 * q + 1]);
        }
    }
}
template <bool kF8>
__device__ __forceinline__ void pp_store_p(uint32_t taddr, const uint32_t (&pk)[PpOperands<kF8>::kPCols]);
template <>
__device__ __forceinline__ void pp_store_p<false>(uint32_t taddr, const uint32_t (&pk)[16]) { tmem_st_x16(taddr, pk); }
template <>
__device__ __forceinline__ void pp_store_p<true>(uint32_t taddr, const uint32_t (&pk)[8]) { tmem_st_x8(taddr, pk); }

__device__ __forceinline__ uint32_t pp_bar(uint32_t bar0, int i) { return bar0 + 8 * i; }

// Counter in global memory that one SM raises after its writes and another reads before its loads.
__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu_add(unsigned int* p, unsigned int v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Ring cursor: slot and phase parity of the g-th entry of a ring of N slots.
template <int N>
struct PpRing {
    uint32_t slot = 0, par = 0;
    __device__ __forceinline__ void next() {
        if (++slot == N) {
            slot = 0;
            par ^= 1;
        }
    }
};

// The thread that issues S = Q K^T of every step.
template <typename T, bool kTmaOut, bool kVarlen, bool kF8, int D>
__device__ __forceinline__ void pp_run_s(uint32_t bar0, uint32_t sQ, uint32_t sK, uint32_t tmem, const FwdParams& p,
                                         int total_items, volatile uint32_t* abort_flag) {
    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
    constexpr uint32_t idesc = kF8 ? instr_desc_e4m3(128, 128, false, false) : instr_desc_f16(kBf16, 128, 128, false, false);
    using Op = PpOperands<kF8, D>;
    uint32_t g = 0;
    PpRing<kPpNK> ring;
    PpItems<kVarlen> items;
    while (items.next(p, total_items)) {
        const int ord = items.ord;
        const PpItem& it = items.it;
        const uint32_t qb = ord & 1;
        if (!mbar_wait(pp_bar(bar0, ppb::q_full + qb), (ord >> 1) & 1, abort_flag, 130)) return;
        const uint32_t a_lo = desc_lo(sQ + qb * kTileBytes, 16);
        for (int j = 0; j < it.n; ++j, ++g, ring.next()) {
            const uint32_t buf = g & 1;
            if (!mbar_wait(pp_bar(bar0, ppb::k_full + ring.slot), ring.par, abort_flag, 131)) return;
            // the softmax of step g-2 has read its scores out of this buffer (it says so together
            // with its reference max)
            if (g >= 2 && !mbar_wait(pp_bar(bar0, ppb::m_ready + buf), ((g >> 1) - 1) & 1, abort_flag, 132)) return;
            tc_fence_after();
            const uint32_t b_lo = desc_lo(sK + ring.slot * Op::kKvSlotBytes, 16);
#pragma unroll
            for (int ks = 0; ks < Op::kSteps; ++ks) {
                // one MMA takes 32 bytes of every row: 16 16-bit elements (a row of d = 128 is two
                // 128-byte boxes, one of d = 64 a single one) or 32 8-bit ones (one box)
                const uint32_t koff = Op::kOneBox ? (uint32_t)(ks * 32) >> 4 : ((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4;
                if (kF8) mma_ss_lo_f8(tmem + 128 + 128 * buf, a_lo + koff, b_lo + koff, idesc, ks > 0 ? 1u : 0u);
                else mma_ss_lo(tmem + 128 + 128 * buf, a_lo + koff, b_lo + koff, idesc, ks > 0 ? 1u : 0u);
            }
            mma_commit(pp_bar(bar0, ppb::s_full + buf));
            mma_commit(pp_bar(bar0, ppb::k_empty + ring.slot));
            // with the output staged in the Q buffer the item's epilogue hands the buffer back
            if (!kTmaOut && j == it.n - 1) mma_commit(pp_bar(bar0, ppb::q_empty + qb));
        }
    }
}

// The thread that issues O += P V of every step.
template <typename T, bool kVarlen, bool kF8, int D>
__device__ __forceinline__ void pp_run_pv(uint32_t bar0, uint32_t sV, uint32_t tmem, const FwdParams& p,
                                          int total_items, volatile uint32_t* abort_flag) {
    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
    constexpr uint32_t idesc = kF8 ? instr_desc_e4m3(128, 128, false, true) : instr_desc_f16(kBf16, 128, D, false, true);
    using Op = PpOperands<kF8, D>;
    uint32_t g = 0;
    PpRing<kPpNV> ring;
    PpItems<kVarlen> items;
    while (items.next(p, total_items)) {
        const int ord = items.ord;
        const PpItem& it = items.it;
        for (int j = 0; j < it.n; ++j, ++g, ring.next()) {
            const uint32_t buf = g & 1;
            if (!mbar_wait(pp_bar(bar0, ppb::v_full + ring.slot), ring.par, abort_flag, 140)) return;
            // the previous item's epilogue has read O out of tensor memory
            if (j == 0 && ord > 0 && !mbar_wait(pp_bar(bar0, ppb::o_free), (ord - 1) & 1, abort_flag, 141)) return;
            if (!mbar_wait(pp_bar(bar0, ppb::p_full + buf), (g >> 1) & 1, abort_flag, 142)) return;
            tc_fence_after();
            // V is the N-major operand: a key is a row of d elements.  16-bit, d = 128: two 128-byte
            // column blocks kHalfBytes apart, 16 keys (2048 bytes) per MMA; d = 64: one block, the
            // same 16 keys per MMA; 8-bit: one block, 32 keys (4096 bytes) per MMA.  Either way an
            // MMA reads 8 columns of P.
            const uint32_t b_lo = desc_lo(sV + ring.slot * Op::kKvSlotBytes, D == 64 ? 16 : kHalfBytes);
#pragma unroll
            for (int ks = 0; ks < Op::kPvSteps; ++ks) {
                if (kF8) mma_ts_lo_f8(tmem, tmem + 384 + 64 * buf + ks * 8, b_lo + ks * (4096 >> 4), idesc,
                                      (ks > 0) ? 1u : (j > 0 ? 1u : 0u));
                else mma_ts_lo(tmem, tmem + 384 + 64 * buf + ks * 8, b_lo + ks * (2048 >> 4), idesc,
                               (ks > 0) ? 1u : (j > 0 ? 1u : 0u));
            }
            mma_commit(pp_bar(bar0, ppb::pv_done + buf));
            mma_commit(pp_bar(bar0, ppb::v_empty + ring.slot));
            if (j == it.n - 1) mma_commit(pp_bar(bar0, ppb::o_final + (ord & 1)));
        }
    }
}

// Paged K/V (packed batches only): kv tile j of sequence b lies in one page; its coordinates
// become (row inside the page, page).  The page of tile j + 1 is looked up before the loader
// waits for tile j's ring slot, so that the table read is off the path that refills a slot.
template <bool kVarlen>
__device__ __forceinline__ int pp_page_of(const FwdParams& p, int b, int j, int n, int Skv) {
    // a sequence without keys still runs one (fully masked) step; it has no table entry to read:
    // page -1 is outside the tensor map, so the loads of that step deliver zeros
    if (kVarlen && p.block_table != nullptr && Skv == 0) return -1;
    if (kVarlen && p.block_table != nullptr && j < n) {
        // (volatile: issued here, ahead of the wait that follows, not where the value is used)
        int page;
        asm volatile("ld.global.nc.s32 %0, [%1];"
                     : "=r"(page)
                     : "l"(p.block_table + (long long)b * p.table_stride + p.by_tiles_per_page.div(j)));
        return page;
    }
    return 0;
}
template <bool kVarlen>
__device__ __forceinline__ void pp_paged_tile(const FwdParams& p, int page, int j, int& row, int& slab) {
    if (kVarlen && p.block_table != nullptr) {
        slab = page;
        row = (j - p.by_tiles_per_page.div(j) * (int)p.by_tiles_per_page.d) * kTile;
    }
}

// The thread that loads Q of every item and K of every step.  (Packed batches: the tensor maps
// have one batch entry that holds every sequence back to back.)
// One tile: two 64-element boxes of a 16-bit tensor of d = 128, or one 128-byte box (8-bit, or d = 64).
template <bool kOneBox>
__device__ __forceinline__ void pp_load_tile(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int h, int s0, int b,
                                             uint64_t policy) {
    if (kOneBox) tma_load_4d_hint(dst, tm, bar, 0, h, s0, b, policy);
    else load_tile_hint(dst, tm, bar, h, s0, b, policy);
}

template <bool kVarlen, bool kF8, int D>
__device__ __forceinline__ void pp_run_load_qk(uint32_t bar0, uint32_t sQ, uint32_t sK, const CUtensorMap* tm_q,
                                               const CUtensorMap* tm_k, const FwdParams& p, int total_items,
                                               volatile uint32_t* abort_flag) {
    tma_prefetch_desc(tm_q);
    tma_prefetch_desc(tm_k);
    const uint64_t pol_q = l2_policy_evict_first(), pol_kv = l2_policy_evict_last();
    PpRing<kPpNK> ring;
    PpItems<kVarlen> items;
    while (items.next(p, total_items)) {
        const int ord = items.ord;
        const PpItem& it = items.it;
        const uint32_t qb = ord & 1;
        // passes at once the first time each buffer is used
        if (!mbar_wait(pp_bar(bar0, ppb::q_empty + qb), ((ord >> 1) & 1) ^ 1, abort_flag, 150)) return;
        mbar_expect_tx(pp_bar(bar0, ppb::q_full + qb), PpOperands<kF8, D>::kQBytes);
        pp_load_tile<PpOperands<kF8, D>::kOneBox>(sQ + qb * kTileBytes, tm_q, pp_bar(bar0, ppb::q_full + qb), it.h,
                       kVarlen ? it.q_base + it.q0 : it.q0, kVarlen ? 0 : it.b, pol_q);
        int page = (kVarlen && p.block_table != nullptr) ? it.page0 : 0;
        for (int j = 0; j < it.n; ++j, ring.next()) {
            const int page_next = pp_page_of<kVarlen>(p, it.b, j + 1, it.n, it.Skv);
            if (!mbar_wait(pp_bar(bar0, ppb::k_empty + ring.slot), ring.par ^ 1, abort_flag, 151)) return;
            mbar_expect_tx(pp_bar(bar0, ppb::k_full + ring.slot), PpOperands<kF8, D>::kKvSlotBytes);
            int row = kVarlen ? it.k_base + j * kTile : j * kTile, slab = kVarlen ? 0 : it.b;
            pp_paged_tile<kVarlen>(p, page, j, row, slab);
            page = page_next;
            pp_load_tile<PpOperands<kF8, D>::kOneBox>(sK + ring.slot * PpOperands<kF8, D>::kKvSlotBytes, tm_k, pp_bar(bar0, ppb::k_full + ring.slot), it.hk, row, slab, pol_kv);
        }
    }
}

// The thread that loads V of every step.
template <bool kVarlen, bool kF8, int D>
__device__ __forceinline__ void pp_run_load_v(uint32_t bar0, uint32_t sV, const CUtensorMap* tm_v, const FwdParams& p,
                                              int total_items, volatile uint32_t* abort_flag) {
    tma_prefetch_desc(tm_v);
    const uint64_t pol_kv = l2_policy_evict_last();
    PpRing<kPpNV> ring;
    PpItems<kVarlen> items;
    while (items.next(p, total_items)) {
        const int ord = items.ord;
        const PpItem& it = items.it;
        int page = (kVarlen && p.block_table != nullptr) ? it.page0 : 0;
        for (int j = 0; j < it.n; ++j, ring.next()) {
            const int page_next = pp_page_of<kVarlen>(p, it.b, j + 1, it.n, it.Skv);
            if (!mbar_wait(pp_bar(bar0, ppb::v_empty + ring.slot), ring.par ^ 1, abort_flag, 152)) return;
            mbar_expect_tx(pp_bar(bar0, ppb::v_full + ring.slot), PpOperands<kF8, D>::kKvSlotBytes);
            int row = kVarlen ? it.k_base + j * kTile : j * kTile, slab = kVarlen ? 0 : it.b;
            pp_paged_tile<kVarlen>(p, page, j, row, slab);
            page = page_next;
            pp_load_tile<PpOperands<kF8, D>::kOneBox>(sV + ring.slot * PpOperands<kF8, D>::kKvSlotBytes, tm_v, pp_bar(bar0, ppb::v_full + ring.slot), it.hk, row, slab, pol_kv);
        }
    }
}

// Warp-wide wait: every lane waits, and the warp leaves together if any lane gave up (the
// tensor-memory instructions that follow need the whole warp).
__device__ __forceinline__ bool pp_warp_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                             unsigned int where) {
    const bool ok = mbar_wait(bar, parity, abort_flag, where);
    return __all_sync(0xffffffffu, ok);
}

// One thread of a softmax warpgroup: its state across the steps of an item, and the step.
template <typename T, bool kVarlen, bool kF8, int D>
struct PpSoftmax {
    static_assert(!(kF8 && kVarlen), "packed batches take 16-bit operands");
    using Op = PpOperands<kF8, D>;
    // fixed for the kernel
    uint32_t bar0;
    volatile uint32_t* abort_flag;
    float* m_mine;          // this row's slot in the reference-max exchange, written by this warpgroup
    const float* m_other;   // the same row's slot written by the other warpgroup
    int w;                  // warpgroup: runs the steps with g & 1 == w
    uint32_t tO, tS, tP;    // this warp's lane quarter of O, S_w, P_w in tensor memory
    float scale_log2;
    int causal, Skv, off;
    uint32_t sV;            // V ring in shared memory (packed batches: see the end of step())
    int r;                  // this thread's row of the tile
    // per item
    int row;                // query row of this thread
    float l_part;           // row sum over this warpgroup's steps, relative to m_loc
    float m_loc;            // reference max after this warpgroup's latest step
    float m_before;         // reference max that step received from the step before it

    // Step g of the CTA = step j of the item.  kMasked: the tile is crossed by the diagonal or by
    // the end of the keys.  Returns false when a wait gave up.
    template <int kMasked>  // 0: no mask code; 1: masked tile; 2: decided at run time by `masked`
    __device__ __forceinline__ bool step(uint32_t (&s)[128], uint32_t g, int j, bool masked = false) {
        if (!pp_warp_wait(pp_bar(bar0, ppb::s_full + w), (g >> 1) & 1, abort_flag, 110 + w)) return false;
        tc_fence_after();
        tmem_ld_x32(tS, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
        tmem_ld_x32(tS + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
        tmem_ld_x32(tS + 64, *reinterpret_cast<uint32_t(*)[32]>(&s[64]));
        tmem_ld_x32(tS + 96, *reinterpret_cast<uint32_t(*)[32]>(&s[96]));
        tmem_wait_ld();
        tc_fence_before();  // for the arrival below that hands the S buffer back
        // probe early, look at the answer after the row max
        const bool m_there = g > 0 && mbar_test(pp_bar(bar0, ppb::m_ready + (1 - w)), ((g - 1) >> 1) & 1);
        if (kMasked == 1 || (kMasked == 2 && masked)) {
            // hidden scores become -inf (the scale is strictly positive, so they come out as exact zeros)
            const int kv0 = j * kTile;
            int lim = Skv - kv0;
            if (causal) lim = min(lim, row + off - kv0 + 1);
#pragma unroll
            for (int i = 0; i < 128; ++i)
                if (i >= lim) s[i] = 0xff800000u;
        }
        const float mx = pp_row_max(s);
        // reference max left by step g-1 (of the other warpgroup); an item starts afresh
        float m_prev = -INFINITY;
        if (g > 0) {
            if (!__all_sync(0xffffffffu, m_there) &&
                !pp_warp_wait(pp_bar(bar0, ppb::m_ready + (1 - w)), ((g - 1) >> 1) & 1, abort_flag, 112 + w))
                return false;
            if (j > 0) m_prev = *m_other;
        }
        m_before = m_prev;
        // lazy reference update: the reference moves only when the row max outgrew it by more than
        // the threshold (always on the first visible score; never on -inf)
        const bool grow = (mx - m_prev) * scale_log2 > (kF8 ? kP8Threshold : kRescaleThreshold);
        const float m_new = grow ? mx : m_prev;
        *m_mine = m_new;
        // one arrival per thread: publishes its reference max and, the scores being in registers,
        // lets Q K^T of step g+2 overwrite the S buffer
        mbar_arrive(pp_bar(bar0, ppb::m_ready + w));
        if (m_loc != m_new) {  // this warpgroup's row sum follows the reference
            if (l_part > 0.f) l_part *= fast_exp2((m_loc - m_new) * scale_log2);
            m_loc = m_new;
        }
        const float neg_ms = -((m_new == -INFINITY) ? 0.f : m_new) * scale_log2 + (kF8 ? kP8ScaleLog2 : 0.f);
        const uint64_t sc2 = f2_pack(scale_log2, scale_log2), nm2 = f2_pack(neg_ms, neg_ms);
        uint64_t la = f2_pack(0.f, 0.f), lb = la;
        {
            uint32_t pk[Op::kPCols];
            const bool p_free = g < 2 || mbar_test(pp_bar(bar0, ppb::pv_done + w), ((g >> 1) - 1) & 1);
            pp_exp_chunk<T, kF8>(s, 0, sc2, nm2, la, lb, pk);
            if (g >= 2) {
                // O += P V of step g-2 has read this P buffer
                if (!__all_sync(0xffffffffu, p_free) &&
                    !pp_warp_wait(pp_bar(bar0, ppb::pv_done + w), ((g >> 1) - 1) & 1, abort_flag, 116 + w))
                    return false;
                tc_fence_after();
            }
            if (__builtin_expect(j > 0 && __any_sync(0xffffffffu, grow), 0)) {
                // rare: the reference moved.  O holds the P V sums up to step g-1 once that step's
                // MMAs have completed (those of step g-2 have, see above, so the parity wait on the
                // other buffer's barrier is one phase at most behind).
                if (!pp_warp_wait(pp_bar(bar0, ppb::pv_done + (1 - w)), ((g - 1) >> 1) & 1, abort_flag, 114 + w)) return false;
                tc_fence_after();
                const float alpha = grow ? ((m_prev == -INFINITY) ? 0.f : fast_exp2((m_prev - mx) * scale_log2)) : 1.f;
#pragma unroll 1
                for (int c = 0; c < D / 16; ++c) {
                    uint32_t o[16];
                    tmem_ld_x16(tO + c * 16, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    tmem_st_x16(tO + c * 16, o);
                }
            }
            pp_store_p<kF8>(tP, pk);
        }
#pragma unroll
        for (int c = 1; c < 4; ++c) {
            uint32_t pk[Op::kPCols];
            pp_exp_chunk<T, kF8>(s, c, sc2, nm2, la, lb, pk);
            pp_store_p<kF8>(tP + c * Op::kPCols, pk);
        }
        {
            float a0, a1, b0, b1;
            f2_unpack(la, a0, a1);
            f2_unpack(lb, b0, b1);
            l_part += (a0 + a1) + (b0 + b1);
        }
        if (kVarlen && (kMasked == 1 || (kMasked == 2 && masked)) && Skv - j * kTile < kTile) {
            // Packed batches, the tile that holds a sequence's last key: the rows of V after it
            // belong to the next sequence, or to the unused rest of a page, and may hold anything.
            // Their probabilities are exact zeros, but 0 * NaN would still poison O, so those
            // rows are cleared in shared memory before P V of this step may start (a contiguous
            // tensor gets the same from the zero fill of its TMA loads).  Thread r owns key row r:
            // its bytes are one 128-byte line in each 64-element half of the tile, whatever the swizzle.
            static_assert(kPpNV == 2, "the V slot of step g is taken to be g & 1");
            if (!pp_warp_wait(pp_bar(bar0, ppb::v_full + w), (g >> 1) & 1, abort_flag, 124 + w)) return false;
            if (r >= Skv - j * kTile) {
                const uint32_t line = sV + (uint32_t)w * Op::kKvSlotBytes + (uint32_t)r * 128u;
#pragma unroll
                for (int c = 0; c < D / 8; ++c)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(line + (uint32_t)(c >> 3) * kHalfBytes + (uint32_t)(c & 7) * 16u), "r"(0u) : "memory");
            }
            fence_proxy_async_smem();
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(pp_bar(bar0, ppb::p_full + w));
        return true;
    }
};

// kTmaOut: the output has the operands' 16-bit type; an item's O goes, scaled and rounded, into
// the item's Q buffer (which Q K^T has finished with by then) in the swizzled layout of a tile,
// and each warp sends its 32 rows to global memory with two TMA stores (tm_o: boxes of 32 rows x
// 64 columns).  Rows past the end of the queries are clipped by the tensor map.  Otherwise
// (fp32 output) every thread stores its own row.
// kSingle: the step exists once, and a branch skips its mask code on tiles every row sees in
// full; otherwise those tiles take a loop of their own without mask code.  The single copy is a
// little slower per step and much smaller: with it, what an item executes from its first step
// to its epilogue stays within the 32 KB the instruction cache serves at full rate, which is
// what counts when an item has few steps.
// kVarlen (needs kTmaOut): a packed batch of sequences of different lengths (see FwdParams).
// kF8: q, k, v hold FP8 e4m3 bytes (see PpOperands); T is then the type of the output only.
// kProj (needs kTmaOut): a projection phase follows in the same launch (proj_gemm.cuh): a warp
// that has stored its rows of an item's output waits until the stores have reached global memory
// and counts them in done[batch * n_qtiles + query tile]; four warps and Hq heads make a row
// block of O complete.
// The whole kernel but for the release of tensor memory; returns false if nothing was set up.
template <typename T, bool kTmaOut, bool kSingle, bool kVarlen, bool kF8, bool kProj, int D = 128>
__device__ __forceinline__ bool pp_attention(const CUtensorMap& tm_q, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                             const CUtensorMap& tm_o, const FwdParams& p, const int total_items,
                                             PpStatic& ss, const uint32_t smem_base, unsigned int* done) {
    static_assert(!kProj || (kTmaOut && !kVarlen && D == 128), "the projection phase reads a contiguous 16-bit O of d = 128");
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + kPpQBufs * kTileBytes;
    const uint32_t sV = sK + kPpNK * PpOperands<kF8, D>::kKvSlotBytes;
    const uint32_t bar0 = smem_u32(&ss.bars[0]);
    volatile uint32_t* abort_flag = &ss.abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    if (smem_base & 1023u) {  // uniform for the CTA: nothing has been set up yet
        if (tid == 0) record_timeout(900);
        return false;
    }
    if (tid == 0) {
        for (int i = 0; i < ppb::count; ++i) {
            const bool q_back = kTmaOut && (i == ppb::q_empty || i == ppb::q_empty + 1);
            mbar_init(pp_bar(bar0, i), i >= ppb::p_full ? 128 : (q_back ? 4 : 1));
        }
        ss.abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 8) {
        tmem_alloc(smem_u32(&ss.tmem_holder), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ss.tmem_holder;
    const int off = p.Skv - p.Sq;

    if (warp < 8) {
        // ================================================================ softmax + epilogue
        setmaxnreg_inc<kPipeSoftmaxRegs>();  // a whole row of S lives in registers
        const int w = warp >> 2;             // this warpgroup runs the steps with g & 1 == w
        const int r = tid & 127;
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tO = tmem_base + lane_sel;
        const uint32_t tS = tmem_base + lane_sel + 128 + 128 * w;
        const uint32_t tP = tmem_base + lane_sel + 384 + 64 * w;
        const float scale_log2 = p.scale_log2;
        PpSoftmax<T, kVarlen, kF8, D> sm;
        sm.sV = sV;
        sm.r = r;
        sm.bar0 = bar0;
        sm.abort_flag = abort_flag;
        sm.m_mine = &ss.m_xch[w][r];
        sm.m_other = &ss.m_xch[1 - w][r];
        sm.w = w;
        sm.tO = tO;
        sm.tS = tS;
        sm.tP = tP;
        sm.scale_log2 = scale_log2;
        sm.causal = p.causal;
        sm.Skv = p.Skv;
        sm.off = off;
        uint32_t g = 0;        // step counter of the CTA
        uint32_t items2 = 0;   // items with at least two steps seen so far
        bool ok = true;
        // Q buffer whose TMA stores this warp has issued but not yet waited for (-1: none).  The
        // wait (until the stores have read the buffer) and the hand-back to the loader come after
        // this warp's next step: early enough for the load of the item after the next, and off
        // the path from one item's last step to the next item's first.
        int q_back = -1;
        int done_slot = 0;     // kProj: the row block the pending stores belong to
        auto hand_back_q = [&]() {
            if (kTmaOut && q_back >= 0) {
                if (lane == 0) {
                    if (kProj) {
                        tma_store_wait_all();          // written, not only read out of shared memory
                        red_release_gpu_add(done + done_slot, 1u);
                    } else {
                        tma_store_wait_read();
                    }
                    mbar_arrive(pp_bar(bar0, ppb::q_empty + q_back));
                }
                q_back = -1;
            }
        };
        PpItems<kVarlen> items;
        while (ok && items.next(p, total_items)) {
            const int ord = items.ord;
            const PpItem& it = items.it;
            const int n = it.n;
            const int row = it.q0 + r;   // within the sequence
            const int Sq_i = kVarlen ? it.Sq : p.Sq, Skv_i = kVarlen ? it.Skv : p.Skv;
            const int off_i = kVarlen ? it.Skv - it.Sq : off;
            if (kVarlen) {
                sm.Skv = Skv_i;
                sm.off = off_i;
            }
            sm.row = row;
            sm.l_part = 0.f;
            sm.m_loc = -INFINITY;
            sm.m_before = -INFINITY;
            uint32_t s[128];             // this thread's row of S, later of O
            const uint32_t xb = items2 & 1, xpar = (items2 >> 1) & 1;  // row-sum exchange buffer / phase
            // kv tiles every row of the query tile sees in full: they come first and take the
            // loop without mask code; the few tiles crossed by the diagonal or by the end of the
            // keys follow
            int n_full = Skv_i / kTile;
            if (p.causal) n_full = min(n_full, max(0, (it.q0 + off_i + 1) / kTile));
            n_full = min(n_full, n);
            // this warpgroup's steps of the item: those with an absolute step number of its parity
            const uint32_t g_item = g;
            int j = (int)((g_item ^ (uint32_t)w) & 1u);
            // no step of this warpgroup in the item (one step, the other warpgroup's): the next
            // step it takes belongs to the item whose Q load waits for the buffer, so hand it back now
            if (j >= n) hand_back_q();
            if (kSingle) {
            for (; j < n && ok; j += 2) {
                ok = sm.template step<2>(s, g_item + (uint32_t)j, j, j >= n_full);
                hand_back_q();
                if (ok && j == n - 2) {
                    ss.l_xch[xb][r] = sm.l_part;
                    mbar_arrive(pp_bar(bar0, ppb::l_pub + xb));
                }
            }
            } else {
            for (; j < n_full && ok; j += 2) {
                ok = sm.template step<0>(s, g_item + (uint32_t)j, j);
                hand_back_q();
                if (ok && j == n - 2) {
                    // the other warpgroup runs the last step and the epilogue: hand it this row sum
                    // (it is relative to the reference this step left, which that step receives)
                    ss.l_xch[xb][r] = sm.l_part;
                    mbar_arrive(pp_bar(bar0, ppb::l_pub + xb));
                }
            }
            for (; j < n && ok; j += 2) {
                ok = sm.template step<1>(s, g_item + (uint32_t)j, j);
                hand_back_q();
                if (ok && j == n - 2) {
                    ss.l_xch[xb][r] = sm.l_part;
                    mbar_arrive(pp_bar(bar0, ppb::l_pub + xb));
                }
            }
            }
            const float l_part = sm.l_part, m_loc = sm.m_loc, m_before = sm.m_before;
            if (ok && ((g_item + (uint32_t)n - 1u) & 1u) == (uint32_t)w) {
                // ---- epilogue of the item, by the warpgroup that ran its last step
                float l_run = l_part;
                if (n >= 2) {
                    ok = pp_warp_wait(pp_bar(bar0, ppb::l_pub + xb), xpar, abort_flag, 118 + w);
                    if (!ok) break;
                    const float l_other = ss.l_xch[xb][r];
                    // the other warpgroup's sum is relative to the reference this one's last step received
                    if (l_other > 0.f) l_run += l_other * fast_exp2((m_before - m_loc) * scale_log2);
                }
                ok = pp_warp_wait(pp_bar(bar0, ppb::o_final + (ord & 1)), (ord >> 1) & 1, abort_flag, 120 + w);
                if (!ok) break;
                tc_fence_after();
                tmem_ld_x32(tO, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
                tmem_ld_x32(tO + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
                if (D == 128) {
                    tmem_ld_x32(tO + 64, *reinterpret_cast<uint32_t(*)[32]>(&s[64]));
                    tmem_ld_x32(tO + 96, *reinterpret_cast<uint32_t(*)[32]>(&s[96]));
                }
                tmem_wait_ld();
                // O is in registers: the next item's first P V may overwrite it
                tc_fence_before();
                mbar_arrive(pp_bar(bar0, ppb::o_free));
                // (FP8: O and the row sum carry the same factor on the probabilities; V's own factor goes on O)
                const float inv_l = (l_run > 0.f) ? (kF8 ? p.out_scale / l_run : 1.f / l_run) : 0.f;
                const long long obase = kVarlen ? (long long)(it.q_base + row) * p.o_ss + (long long)it.h * p.o_sh
                                                : (long long)it.b * p.o_sb + (long long)row * p.o_ss + (long long)it.h * p.o_sh;
                if (row < Sq_i && p.lse != nullptr) {
                    const float lse = (l_run > 0.f) ? (m_loc * scale_log2 + log2f(l_run) - (kF8 ? kP8ScaleLog2 : 0.f)) * 0.6931471805599453f
                                                    : -INFINITY;
                    if (kVarlen) p.lse[(long long)it.h * p.total_q + it.q_base + row] = lse;
                    else p.lse[((long long)it.b * p.Hq + it.h) * p.Sq + row] = lse;
                }
                if (kTmaOut) {
                    const uint32_t q_buf = sQ + (uint32_t)(ord & 1) * kTileBytes;
                    const uint32_t row_base = q_buf + (uint32_t)r * 128u;
#pragma unroll
                    for (int c = 0; c < D / 8; ++c) {
                        // 16-byte chunk c & 7 of the row's half c >> 3, at its swizzled place
                        const uint32_t addr = row_base + (uint32_t)(c >> 3) * kHalfBytes + (((uint32_t)(c & 7) ^ ((uint32_t)r & 7u)) << 4);
                        const uint32_t w0 = pack2<T>(__uint_as_float(s[8 * c]) * inv_l, __uint_as_float(s[8 * c + 1]) * inv_l);
                        const uint32_t w1 = pack2<T>(__uint_as_float(s[8 * c + 2]) * inv_l, __uint_as_float(s[8 * c + 3]) * inv_l);
                        const uint32_t w2 = pack2<T>(__uint_as_float(s[8 * c + 4]) * inv_l, __uint_as_float(s[8 * c + 5]) * inv_l);
                        const uint32_t w3 = pack2<T>(__uint_as_float(s[8 * c + 6]) * inv_l, __uint_as_float(s[8 * c + 7]) * inv_l);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    const int row0 = it.q0 + (warp & 3) * 32;   // first row of this warp
                    // packed batches: the rows after a sequence's last belong to the next
                    // sequence, so only a warp whose 32 rows all exist may use the box store
                    const bool box = kVarlen ? (row0 + 32 <= Sq_i) : (row0 < Sq_i);
                    if (lane == 0 && box) {
                        const uint32_t src = q_buf + (uint32_t)(warp & 3) * 4096u;
                        tma_store_4d(&tm_o, src, 0, it.h, kVarlen ? it.q_base + row0 : row0, kVarlen ? 0 : it.b);
                        if (D == 128) tma_store_4d(&tm_o, src + kHalfBytes, 64, it.h, kVarlen ? it.q_base + row0 : row0, kVarlen ? 0 : it.b);
                        tma_store_commit();
                    }
                    q_back = ord & 1;  // handed back to the loader after this warp's next step
                    if (kProj) done_slot = it.b * p.n_qtiles + it.q0 / kTile;
                    __syncwarp();
                    if (kVarlen && !box && row < Sq_i) {
                        // the ragged end of a sequence: each thread writes its own row
                        T* dst = static_cast<T*>(p.o) + obase;
#pragma unroll
                        for (int c = 0; c < D / 8; ++c)
                            reinterpret_cast<uint4*>(dst)[c] =
                                make_uint4(pack2<T>(__uint_as_float(s[8 * c]) * inv_l, __uint_as_float(s[8 * c + 1]) * inv_l),
                                           pack2<T>(__uint_as_float(s[8 * c + 2]) * inv_l, __uint_as_float(s[8 * c + 3]) * inv_l),
                                           pack2<T>(__uint_as_float(s[8 * c + 4]) * inv_l, __uint_as_float(s[8 * c + 5]) * inv_l),
                                           pack2<T>(__uint_as_float(s[8 * c + 6]) * inv_l, __uint_as_float(s[8 * c + 7]) * inv_l));
                    }
                } else if (row < Sq_i) {
                    if (p.o_fp32) {
                        float4* dst = reinterpret_cast<float4*>(static_cast<float*>(p.o) + obase);
#pragma unroll
                        for (int i = 0; i < D / 4; ++i)
                            dst[i] = make_float4(__uint_as_float(s[4 * i]) * inv_l, __uint_as_float(s[4 * i + 1]) * inv_l,
                                                 __uint_as_float(s[4 * i + 2]) * inv_l,
                                                 __uint_as_float(s[4 * i + 3]) * inv_l);
                    } else {
                        T* dst = static_cast<T*>(p.o) + obase;
#pragma unroll
                        for (int c = 0; c < D / 8; ++c)
                            reinterpret_cast<uint4*>(dst)[c] =
                                make_uint4(pack2<T>(__uint_as_float(s[8 * c]) * inv_l, __uint_as_float(s[8 * c + 1]) * inv_l),
                                           pack2<T>(__uint_as_float(s[8 * c + 2]) * inv_l, __uint_as_float(s[8 * c + 3]) * inv_l),
                                           pack2<T>(__uint_as_float(s[8 * c + 4]) * inv_l, __uint_as_float(s[8 * c + 5]) * inv_l),
                                           pack2<T>(__uint_as_float(s[8 * c + 6]) * inv_l, __uint_as_float(s[8 * c + 7]) * inv_l));
                    }
                }
            }
            g = g_item + (uint32_t)n;
            if (n >= 2) ++items2;
        }
        // the stores read shared memory, which has to outlive them
        if (kProj) hand_back_q();
        else if (kTmaOut && lane == 0) tma_store_wait_all();
    } else {
        setmaxnreg_dec<kPipeOtherRegs>();
        if (lane == 0) {
            if (warp == 8) pp_run_s<T, kTmaOut, kVarlen, kF8, D>(bar0, sQ, sK, tmem_base, p, total_items, abort_flag);
            else if (warp == 10) pp_run_pv<T, kVarlen, kF8, D>(bar0, sV, tmem_base, p, total_items, abort_flag);
            else if (warp == 9) pp_run_load_qk<kVarlen, kF8, D>(bar0, sQ, sK, &tm_q, &tm_k, p, total_items, abort_flag);
            else pp_run_load_v<kVarlen, kF8, D>(bar0, sV, &tm_v, p, total_items, abort_flag);
        }
        __syncwarp();
    }
    return true;
}

template <typename T, bool kTmaOut, bool kSingle, bool kVarlen, bool kF8 = false, int D = 128>
__global__ void __launch_bounds__(kPipeThreads, 1)
fa_fwd_pingpong_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                       const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                       const FwdParams p, const int total_items) {
    // Shared memory is used to the last byte: 3 KiB of static state (sized so that the dynamic
    // part that follows it starts on a 1024-byte boundary, which the 128-byte swizzle needs)
    // plus seven 32 KiB tiles.  The alignment is checked rather than assumed.
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(1024) PpStatic ss;
    if (!pp_attention<T, kTmaOut, kSingle, kVarlen, kF8, false, D>(tm_q, tm_k, tm_v, tm_o, p, total_items, ss,
                                                                   smem_u32(smem_raw), nullptr))
        return;
    tc_fence_before();
    __syncthreads();
    if ((threadIdx.x >> 5) == 8) {
        __syncwarp();
        tmem_dealloc(ss.tmem_holder, 512);
    }
}

// to: map over the output with boxes of 32 rows x 64 columns; read only when the output has the
// operands' type (any valid map otherwise).
// The item order of a launch on `grid` CTAs (see pp_class_order and PpItems): returns the
// parameters with the order's fields filled in.  bytes_per_key: K plus V bytes of one key and head.
inline FwdParams pp_plan_items(const FwdParams& fp, int grid, double bytes_per_key) {
    const bool varlen = fp.cu_q != nullptr;
    // Class size of the item order: large enough that the K and V of the kv heads one round of
    // CTAs works on (about grid / (C * group) of them, Skv * 512 bytes each) fit in a fraction of
    // L2, but at most half of a head's tiles and 16 (a class that is the whole head makes all
    // its tiles read the same K/V lines at the same moment, which measured slower).  Under the
    // causal mask the items of a class differ in length, which costs balance when a head has few
    // tiles: heads with fewer than 16 keep the plain longest-first order.  When one head alone
    // fills every CTA, a single class: the plain head-by-head order.
    FwdParams fpc = fp;
    int cls_log2 = 0;
    if (fp.n_qtiles >= grid) {
        while ((1 << cls_log2) < fp.n_qtiles) ++cls_log2;
    } else {
        const double head_bytes = bytes_per_key * fp.Skv / (fp.Hq / fp.Hkv);
        const double budget = 32.0 * 1024 * 1024;
        const int half = fp.n_qtiles / 2 < 16 ? fp.n_qtiles / 2 : 16;
        const int cap = (fp.causal && fp.n_qtiles < 16) ? 1 : half;
        while ((grid >> cls_log2) * head_bytes > budget && (2 << cls_log2) <= cap) ++cls_log2;
        while (cls_log2 > 0 && (1 << cls_log2) > fp.n_qtiles) --cls_log2;
    }
    if (varlen) {
        // Packed batches: sequence by sequence and head by head, a head's tiles longest first (a
        // single class).  The lengths differ from sequence to sequence, so classes of tiles across
        // heads would mix long and short items in a round; head by head a round holds the tiles
        // of two or three neighbouring heads, which are of a size and share their K and V
        // (measured on 32 requests of 256 to 8192 tokens: 6.0 ms against 6.8 to 7.7 ms with
        // classes of 1 to 16 tiles).
        cls_log2 = 0;
        while ((1 << cls_log2) < fp.n_qtiles) ++cls_log2;
    }
    // From three rounds per head on (56K keys on 148 SMs) and once a head's K and V are past what
    // L2 keeps, the head-by-head order with whole rounds per head (see PpItems); the empty slots of
    // a head's last round cost little there because its items are the head's shortest.
    const double kv_bytes_per_head = bytes_per_key * fp.Skv;
    if (!varlen && fp.n_qtiles >= 3 * grid && kv_bytes_per_head > 24.0 * 1024 * 1024) {
        fpc.rounds_per_head = (fp.n_qtiles + grid - 1) / grid;
        fpc.by_rph.set(fpc.rounds_per_head);
    }
    fpc.cls_log2 = cls_log2;
    const long long class_items = ((long long)fp.B * fp.Hq) << cls_log2;  // > total only for a single class
    fpc.by_class.set(class_items > 0x7fffffffll ? 0x7fffffff : (int)class_items);
    const int last = fp.n_qtiles & ((1 << cls_log2) - 1);
    fpc.by_lastcls.set(last ? last : 1);
    return fpc;
}

// kF8: tq, tk, tv are maps over FP8 e4m3 bytes (boxes of 128 rows x 128 bytes) and T is the output type.
// D: the head dimension, 128, or 64 with 16-bit operands (maps with boxes of 64 elements either way).
template <typename T, bool kF8 = false, int D = 128>
int launch_pingpong(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                    const FwdParams& fp, cudaStream_t st, int* cuda_err) {
    constexpr int smem = kPpQBufs * kTileBytes + (kPpNK + kPpNV) * PpOperands<kF8, D>::kKvSlotBytes;
    // the single-copy step up to 32 kv tiles per item (timed: ahead by 3 % at 2048 keys, level at
    // 4096, behind by 1 % at 8192)
    const bool single = fp.o_fp32 || fp.Skv <= 32 * kTile;
    const bool varlen = fp.cu_q != nullptr;
    if (varlen && fp.o_fp32) return -3;
    if (kF8 && (varlen || fp.o_fp32)) return -3;
    auto kern = kF8 ? fa_fwd_pingpong_kernel<T, true, true, false, kF8, D>
                    : (varlen ? fa_fwd_pingpong_kernel<T, true, true, kF8 ? false : true, false, D>
                              : (fp.o_fp32 ? fa_fwd_pingpong_kernel<T, false, true, false, false, D>
                                           : (single ? fa_fwd_pingpong_kernel<T, true, true, false, false, D>
                                                     : fa_fwd_pingpong_kernel<T, true, false, false, false, D>)));
    int sm_count = 0;
    cudaError_t e;
    if (int ce = prepare_big_smem_kernel(reinterpret_cast<const void*>(kern), smem, &sm_count)) { *cuda_err = ce; return -7; }
    const long long total = (long long)fp.n_qtiles * fp.B * fp.Hq;
    if (total > 0x7fffffffll) return -3;
    const int grid = (int)(total < sm_count ? total : sm_count);
    const FwdParams fpc = pp_plan_items(fp, grid, (kF8 || D == 64) ? 256.0 : 512.0);
    kern<<<grid, kPipeThreads, smem, st>>>(tq, tk, tv, to, fpc, (int)total);
    e = cudaGetLastError();
    if (e != cudaSuccess) { *cuda_err = (int)e; return -7; }
    return 0;
}

}  // namespace fa
