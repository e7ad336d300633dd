// Decode-stage attention (one query row per sequence over the cached K and V), split along
// the cache: each CTA streams one chunk of one (sequence, kv head) through a TMA-fed
// shared-memory ring and keeps running (rowmax, rowsum, O) for the query heads that share
// the kv head; a second kernel merges the per-chunk partial results.  The work is a single
// pass over the cache, so the kernel is written for HBM bandwidth: every cache byte is read
// exactly once and nothing but the partials is written.
#pragma once

#include <type_traits>

#include "sm100_ptx.cuh"

namespace fa {

constexpr int kDecTile = 128;                 // keys per shared-memory tile
constexpr int kDecStages = 3;                 // ring depth (K and V tiles each)
constexpr int kDecTileBytes = 32768;          // a tile of d = 128
constexpr int kDecHalfBytes = 16384;          // one 128-key x 64-element box
// Head dimension D (128 or 64): a tile is 128 keys x D 16-bit elements, one or two swizzled
// boxes, in a ring of three slots per operand.  With D = 64 a CTA's rings are 96 KiB and two
// CTAs share an SM: the bytes in flight per SM are those of D = 128, and twice the consumer
// warps work on them -- a key costs the same instructions whatever D is and brings half the
// bytes (measured on 64 sequences of 1K to 32K keys: 6.99 against 6.00 TB/s with one CTA of six
// slots per SM).
template <int D>
struct DecShape {
    static_assert(D == 64 || D == 128, "head dimensions of the 16-bit decode kernel");
    static constexpr int kTileBytes = kDecTile * D * 2;
    static constexpr int kStages = kDecStages;
    static constexpr int kCtasPerSm = 128 / D;
    static constexpr int kSmem = 1024 + 2 * kStages * kTileBytes;
};

struct DecodeParams {
    const void* q;        // [B,1,Hq,d] 16-bit
    const int* seqlens;   // [B] device
    float* o_part;        // [B,Hq,NC,d]
    float* lse_part;      // [B,Hq,NC]
    int B, Hq, Hkv, Smax;
    int chunk;            // keys per chunk (multiple of kDecTile)
    int n_chunks;         // ceil(Smax / chunk)
    float scale_log2;
    // paged cache (block_table != nullptr): key j of sequence b is row j % page_size of page
    // block_table[b * table_stride + j / page_size]; the tensor maps then run over
    // [pages, page_size, Hkv, d]; page_size is a multiple of kDecTile, or 16, 32 or 64 (then a
    // tile is several pages and the TMA box is one page high)
    const int* block_table;
    int page_size, table_stride;
    float v_scale;        // 8-bit cache only: factor of the stored values
    int Sq;               // query rows per sequence (1; more for the append form of the fp16 kernel)
    // fp16/bf16 kernel with a single chunk per sequence (n_chunks == 1): the split kernel writes
    // the result itself and no merge kernel runs (nullptr otherwise)
    void* o_final;
    float* lse_final;
    int bf16_io = 0;      // 8-bit cache kernel only: q and o are bf16 (fp16 otherwise)
};


// ---------------------------------------------------------------------------------------
// Split kernel.  A CTA takes one chunk of one (sequence, kv head) and up to 16 of the query
// heads that share the kv head (all of them when Hq / Hkv <= 16).  The query rows are padded
// to the 16 rows of a warp-level mma.sync (m16n8k16, fp32 accumulate): the scan is bound by
// the cache stream, and the warp-level tensor path keeps the arithmetic per cache byte far
// below what the FMA pipe would need, for one query head as well as for sixteen.  Each of the
// four consumer warps owns keys [32w, 32w+32) of every 128-key tile and keeps its own running
// (rowmax, rowsum, O) for them, so consumer warps never synchronise with each other until the
// final merge; a fifth warp issues the TMA loads into a 3-slot ring of K and V tiles.
// Cache rows past the sequence may hold NaN: their scores are masked and their V rows are
// zeroed in shared memory before the second MMA touches them.
constexpr int kDecMmaThreads = 160;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_16816_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// The consumer warps' work in the keys-as-rows form (at most 8 rows, i.e. (token, head) pairs,
// per kv head).  A warp-level MMA has 16 rows and 8 columns: with the query heads as rows, as in the
// general form below, a kv head with 1 to 8 query heads leaves half or more of every MMA to
// padding.  Here the KEYS are the rows: S^T = K q^T (A = 16 keys x 16 elements of K by plain
// ldmatrix, B = q^T, the 8 columns are the heads), and O^T += V^T P^T (A = 16 output columns x 16
// keys of V by transposing ldmatrix, B = P^T, which is the accumulator layout of S^T transposed
// 8 x 8 with movmatrix).  A tile then takes half the MMAs, a thread holds half the scores and
// half the accumulators, and the row maxima and sums run over the lanes that share a column.
// q_col: the query row that is this thread's column g of q^T (nullptr: padding).  kMulti: hide0,
// hide1 say how many of the sequence's last keys the rows in this thread's accumulator columns
// 2 t4, 2 t4 + 1 must not see (they came after the row's token).
// Leaves each warp's (max, sum, O) in mo / ml in the layout the merge expects; returns false
// after a wait that gave up.
template <bool kMulti, typename T, int D>
__device__ __forceinline__ bool dec_consume_key_rows(const DecodeParams& p, uint64_t* bars, volatile uint32_t* abort_flag,
                                                     uint32_t sK, uint32_t sV, float* mo, float* ml, int warp, int lane,
                                                     const T* q_col, int hide0, int hide1, int len, int k_begin, int k_end,
                                                     int n_tiles) {
    constexpr int kStages = DecShape<D>::kStages, kTileB = DecShape<D>::kTileBytes;
    constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
    const int g = lane >> 2, t4 = lane & 3;
    // q^T as B fragments: column g is head g, rows 2 t4, 2 t4 + 1 (and + 8) of every 16-element step
    uint32_t qb[D / 16][2];
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        const int d0 = ks * 16 + 2 * t4;
        qb[ks][0] = q_col ? *reinterpret_cast<const uint32_t*>(q_col + d0) : 0u;
        qb[ks][1] = q_col ? *reinterpret_cast<const uint32_t*>(q_col + d0 + 8) : 0u;
    }
    // O^T: block i holds output columns 16 i + g (values 0, 1) and 16 i + 8 + g (values 2, 3) of heads 2 t4, 2 t4 + 1
    float o[D / 16][4];
#pragma unroll
    for (int i = 0; i < D / 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // heads 2 t4 and 2 t4 + 1
    const int key_w = warp * 32;  // this warp's keys inside a tile
    bool ok = true;

    for (int t = 0; t < n_tiles; ++t) {
        const int st = t % kStages;
        const uint32_t parity = (t / kStages) & 1;
        const int valid = min(kDecTile, k_end - (k_begin + t * kDecTile)) - key_w;  // valid keys of this warp's 32
        ok = mbar_wait(smem_u32(&bars[st]), parity, abort_flag, 20);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        uint32_t pt[2][2];   // P^T as B fragments, per block of 16 keys
        if (valid > 0) {
            // ---- S^T = K q^T: two blocks of 16 keys
            float sc[2][4];  // (key 16 mb + g | heads 2 t4, 2 t4 + 1), (key 16 mb + g + 8 | the same heads)
            const uint32_t kt = sK + st * kTileB;
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) {
                sc[mb][0] = sc[mb][1] = sc[mb][2] = sc[mb][3] = 0.f;
                const int key = key_w + mb * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    // matrices: (keys 0-7, chunk 2 ks), (keys 8-15, chunk 2 ks), (keys 0-7, chunk 2 ks + 1), (keys 8-15, ...)
                    const int chunk = 2 * ks + (lane >> 4);
                    const uint32_t addr = kt + (chunk >> 3) * kDecHalfBytes + key * 128 + (((chunk & 7) ^ (key & 7)) << 4);
                    uint32_t a[4];
                    ldsm_x4(addr, a[0], a[1], a[2], a[3]);
                    if (kBf16) mma_16816_bf16(sc[mb], a, qb[ks][0], qb[ks][1]);
                    else mma_16816(sc[mb], a, qb[ks][0], qb[ks][1]);
                }
            }
            // ---- mask, running max, probabilities
            // keys of this warp's 32 that a row may see: all valid ones, minus (several query
            // rows) those among the sequence's last that came after the row's token
            const int seen0 = kMulti ? min(valid, len - hide0 - (k_begin + t * kDecTile) - key_w) : valid;
            const int seen1 = kMulti ? min(valid, len - hide1 - (k_begin + t * kDecTile) - key_w) : valid;
            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) {
                const int k_lo = mb * 16 + g;
                if (k_lo >= seen0) sc[mb][0] = -INFINITY;
                if (k_lo >= seen1) sc[mb][1] = -INFINITY;
                if (k_lo + 8 >= seen0) sc[mb][2] = -INFINITY;
                if (k_lo + 8 >= seen1) sc[mb][3] = -INFINITY;
                mx0 = fmaxf(mx0, fmaxf(sc[mb][0], sc[mb][2]));
                mx1 = fmaxf(mx1, fmaxf(sc[mb][1], sc[mb][3]));
            }
#pragma unroll
            for (int sh = 4; sh <= 16; sh <<= 1) {  // over the lanes that hold other keys of the same heads
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
            }
            // finite when key 0 of the warp is visible (always with one query token; an earlier
            // token of several may see none of the warp's keys: its state then stays empty)
            const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
            const float a0 = (m_run[0] == -INFINITY) ? 0.f : fast_exp2((m_run[0] - mn0) * p.scale_log2);
            const float a1 = (m_run[1] == -INFINITY) ? 0.f : fast_exp2((m_run[1] - mn1) * p.scale_log2);
            m_run[0] = mn0;
            m_run[1] = mn1;
            const float nm0 = (kMulti && mn0 == -INFINITY) ? 0.f : -mn0 * p.scale_log2;
            const float nm1 = (kMulti && mn1 == -INFINITY) ? 0.f : -mn1 * p.scale_log2;
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) {
                const int k_lo = mb * 16 + g;
                float* e = sc[mb];
                e[0] = (k_lo < seen0) ? fast_exp2(fmaf(e[0], p.scale_log2, nm0)) : 0.f;
                e[1] = (k_lo < seen1) ? fast_exp2(fmaf(e[1], p.scale_log2, nm1)) : 0.f;
                e[2] = (k_lo + 8 < seen0) ? fast_exp2(fmaf(e[2], p.scale_log2, nm0)) : 0.f;
                e[3] = (k_lo + 8 < seen1) ? fast_exp2(fmaf(e[3], p.scale_log2, nm1)) : 0.f;
                s0 += e[0] + e[2];
                s1 += e[1] + e[3];
                // (key g | heads 2 t4, 2 t4 + 1) -> transposed: (head g | keys 2 t4, 2 t4 + 1), the B fragment
                const uint32_t lo = pack2<T>(e[0], e[1]), hi = pack2<T>(e[2], e[3]);
                asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pt[mb][0]) : "r"(lo));
                asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pt[mb][1]) : "r"(hi));
            }
            l_run[0] = l_run[0] * a0 + s0;  // per-thread partial of the sum over keys (reduced at the end)
            l_run[1] = l_run[1] * a1 + s1;
#pragma unroll
            for (int i = 0; i < D / 16; ++i) {
                o[i][0] *= a0;
                o[i][1] *= a1;
                o[i][2] *= a0;
                o[i][3] *= a1;
            }
        }
        ok = mbar_wait(smem_u32(&bars[kStages + st]), parity, abort_flag, 21);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (valid > 0) {
            const uint32_t vt = sV + st * kTileB;
            if (valid < 32) {
                // rows past the sequence may hold NaN bits: zero them (0 * NaN would poison O)
                for (int i = lane; i < (32 - valid) * (D / 8); i += 32) {
                    const int key = key_w + valid + i / (D / 8), ch = i % (D / 8);
                    const uint32_t addr = vt + (ch >> 3) * kDecHalfBytes + key * 128 + (((ch & 7) ^ (key & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
                }
                __syncwarp();
            }
            // ---- O^T += V^T P^T: two steps of 16 keys, D / 16 blocks of 16 output columns
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) {
                // matrices: (keys 0-7, chunk 2 i), (keys 0-7, chunk 2 i + 1), (keys 8-15, chunk 2 i), (keys 8-15, chunk 2 i + 1)
                const int key = key_w + mb * 16 + (lane >> 4) * 8 + (lane & 7);
#pragma unroll
                for (int i = 0; i < D / 16; ++i) {
                    const int ch = 2 * i + ((lane >> 3) & 1);
                    const uint32_t addr = vt + (ch >> 3) * kDecHalfBytes + key * 128 + (((ch & 7) ^ (key & 7)) << 4);
                    uint32_t a[4];
                    ldsm_x4_trans(addr, a[0], a[1], a[2], a[3]);
                    if (kBf16) mma_16816_bf16(o[i], a, pt[mb][0], pt[mb][1]);
                    else mma_16816(o[i], a, pt[mb][0], pt[mb][1]);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars[2 * kStages + st]));
    }
#pragma unroll
    for (int sh = 4; sh <= 16; sh <<= 1) {
        l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], sh);
        l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], sh);
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");   // every warp is through with the ring: it becomes the merge buffer
    if (ok) {
        const int h0 = warp * 16 + 2 * t4;
#pragma unroll
        for (int i = 0; i < D / 16; ++i) {
            mo[h0 * D + 16 * i + g] = o[i][0];
            mo[(h0 + 1) * D + 16 * i + g] = o[i][1];
            mo[h0 * D + 16 * i + 8 + g] = o[i][2];
            mo[(h0 + 1) * D + 16 * i + 8 + g] = o[i][3];
        }
        if (g == 0) {
            ml[h0 * 2] = m_run[0];
            ml[h0 * 2 + 1] = l_run[0];
            ml[(h0 + 1) * 2] = m_run[1];
            ml[(h0 + 1) * 2 + 1] = l_run[1];
        }
    }
    return ok;
}

// kMulti: Sq > 1 query rows per sequence, the last Sq positions of its cache (decoding after
// several tokens were appended, Appendix C with more than one new token): the 16 MMA rows of a
// CTA are then (token, head) pairs of one kv head, and query token t sees the keys up to
// position len - Sq + t.  q is [B,Sq,Hq,d], the partials [B,Sq,Hq,NC,...].
// grid: (Hkv * ceil(Sq * g / 16), n_chunks, B) with g = Hq / Hkv.  The kv head is the fastest
// index: CTAs that run at the same time then read the same keys' rows of neighbouring heads,
// which are contiguous in the cache (a key's Hkv * D elements), instead of key ranges whole
// chunks apart (64 sequences of 1K to 32K keys, 32 kv heads: 2.39 against 2.48 ms).
// T: the 16-bit type of q, the cache and the probabilities (__half or __nv_bfloat16).
// D: the head dimension, 128 or 64.
// kKeyRows (at most 8 (token, head) rows per kv head): the consumers work in the keys-as-rows
// form (dec_consume_key_rows).
template <bool kMulti, typename T = __half, int D = 128, bool kKeyRows = false>
__global__ void __launch_bounds__(kDecMmaThreads, DecShape<D>::kCtasPerSm)
fa_decode_split_mma_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                           const DecodeParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    constexpr int kStages = DecShape<D>::kStages, kTileB = DecShape<D>::kTileBytes;
    const uint32_t sK = smem_base;
    const uint32_t sV = smem_base + kStages * kTileB;
    __shared__ __align__(8) uint64_t bars[3 * kStages];  // K full, V full, slot empty
    __shared__ volatile uint32_t abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int c = blockIdx.y;
    const int b = blockIdx.z;
    const int g_all = p.Hq / p.Hkv;
    const int Sq = kMulti ? p.Sq : 1;
    const int rows_all = g_all * Sq;               // (token, head) rows that share a kv head
    const int n_sub = (rows_all + 15) / 16;        // CTAs per kv head when there are more than 16
    const int hk = blockIdx.x / n_sub;
    const int sub = blockIdx.x % n_sub;
    const int G = min(16, rows_all - sub * 16);    // rows of this CTA
    // row r of the CTA: token and head, and its row in q and in the partial results
    auto row_token = [&](int r) { return kMulti ? (sub * 16 + r) / g_all : 0; };
    auto row_index = [&](int r) -> long long {
        const int R = sub * 16 + r;
        const int hh = kMulti ? R % g_all : R;
        return ((long long)b * Sq + row_token(r)) * p.Hq + hk * g_all + hh;
    };

    int len = p.seqlens[b];
    len = max(0, min(len, p.Smax));
    const int k_begin = c * p.chunk;
    const int k_end = min(len, k_begin + p.chunk);
    auto lse_index = [&](int r) -> long long {   // lse is [B,Hq,Sq]
        const int R = sub * 16 + r;
        return ((long long)b * p.Hq + hk * g_all + (kMulti ? R % g_all : R)) * Sq + row_token(r);
    };
    if (k_begin >= k_end) {  // uniform for the CTA
        if (p.o_final != nullptr && tid < D) {   // a sequence without keys, and nobody else writes its rows
            for (int r = 0; r < G; ++r) {
                static_cast<T*>(p.o_final)[row_index(r) * D + tid] = T(0.f);
                if (tid == 0 && p.lse_final) p.lse_final[lse_index(r)] = -INFINITY;
            }
        }
        return;
    }
    const int n_tiles = (k_end - k_begin + kDecTile - 1) / kDecTile;

    if (tid == 0) {
        for (int i = 0; i < 2 * kStages; ++i) mbar_init(smem_u32(&bars[i]), 1);
        for (int i = 0; i < kStages; ++i) mbar_init(smem_u32(&bars[2 * kStages + i]), 4);  // one arrival per consumer warp
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();

    if (warp == 4) {
        // ---------------------------------------------------------------- producer
        // the cache is read once: its lines go first when L2 needs room (q and the partial results stay)
        const uint64_t stream_policy = l2_policy_evict_first();
        // paged cache: the page of a tile is looked up one tile ahead of its loads, so that
        // the table read is not on the path that refills a freed slot
        const int* table = p.block_table ? p.block_table + (long long)b * p.table_stride : nullptr;
        if (table && p.page_size < kDecTile) {
            // pages of 16, 32 or 64 keys: a tile is several pages, each its own TMA box (pages past
            // the sequence's last are not loaded: their scores are masked and their V rows zeroed
            // by the consumers).  Lane i of the warp looks up and loads page i of every tile.
            const int ps = p.page_size, n_sub = kDecTile / ps;
            auto lookup = [&](int first_key) {
                const int key = first_key + lane * ps;
                return (lane < n_sub && key < k_end) ? table[key / ps] : -1;
            };
            int pg_next = lookup(k_begin);
            for (int t = 0; t < n_tiles; ++t) {
                const int st = t % kStages;
                const uint32_t bk = smem_u32(&bars[st]), bv = smem_u32(&bars[kStages + st]);
                const int row0 = k_begin + t * kDecTile;
                const int cur = pg_next;
                if (t + 1 < n_tiles) pg_next = lookup(row0 + kDecTile);
                bool ok = true;
                if (lane == 0) ok = mbar_wait(smem_u32(&bars[2 * kStages + st]), ((t / kStages) & 1) ^ 1, &abort_flag, 22);
                if (!__shfl_sync(0xffffffffu, ok, 0)) break;
                const int live = min(n_sub, (k_end - row0 + ps - 1) / ps);   // pages of this tile that hold keys
                if (lane == 0) {
                    mbar_expect_tx(bk, (uint32_t)(live * ps) * (2u * D));
                    mbar_expect_tx(bv, (uint32_t)(live * ps) * (2u * D));
                }
                __syncwarp();
                if (lane < live) {
                    const uint32_t offs = (uint32_t)(lane * ps) * 128u;
                    tma_load_4d_hint(sK + st * kTileB + offs, &tm_k, bk, 0, hk, 0, cur, stream_policy);
                    if (D == 128) tma_load_4d_hint(sK + st * kTileB + kDecHalfBytes + offs, &tm_k, bk, 64, hk, 0, cur, stream_policy);
                    tma_load_4d_hint(sV + st * kTileB + offs, &tm_v, bv, 0, hk, 0, cur, stream_policy);
                    if (D == 128) tma_load_4d_hint(sV + st * kTileB + kDecHalfBytes + offs, &tm_v, bv, 64, hk, 0, cur, stream_policy);
                }
            }
        } else if (lane == 0) {
            int page_next = table ? table[k_begin / p.page_size] : 0;
            for (int t = 0; t < n_tiles; ++t) {
                const int st = t % kStages;
                const uint32_t bk = smem_u32(&bars[st]), bv = smem_u32(&bars[kStages + st]);
                int row0 = k_begin + t * kDecTile;  // first key of the tile within the sequence
                int slab = b;                        // outermost coordinate: the sequence, or the page
                if (table) {
                    slab = page_next;
                    if (t + 1 < n_tiles) page_next = table[(row0 + kDecTile) / p.page_size];
                    row0 %= p.page_size;
                }
                if (!mbar_wait(smem_u32(&bars[2 * kStages + st]), ((t / kStages) & 1) ^ 1, &abort_flag, 22)) break;
                mbar_expect_tx(bk, kTileB);
                tma_load_4d_hint(sK + st * kTileB, &tm_k, bk, 0, hk, row0, slab, stream_policy);
                if (D == 128) tma_load_4d_hint(sK + st * kTileB + kDecHalfBytes, &tm_k, bk, 64, hk, row0, slab, stream_policy);
                mbar_expect_tx(bv, kTileB);
                tma_load_4d_hint(sV + st * kTileB, &tm_v, bv, 0, hk, row0, slab, stream_policy);
                if (D == 128) tma_load_4d_hint(sV + st * kTileB + kDecHalfBytes, &tm_v, bv, 64, hk, row0, slab, stream_policy);
            }
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------------------- consumers
        const int g = lane >> 2, t4 = lane & 3;  // fragment row (query head g and g + 8) and column pair
        float* mo = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));  // [4 warps][16 rows][D]
        float* ml = mo + 4 * 16 * D;                                                         // [4][16][2]: m, l
        bool ok = true;
        if constexpr (kKeyRows) {
            // column g of q^T is row g of the CTA; accumulator columns 2 t4, 2 t4 + 1 are rows 2 t4, 2 t4 + 1
            const T* q_col = (g < G) ? static_cast<const T*>(p.q) + row_index(g) * D : nullptr;
            const int hide0 = kMulti ? Sq - 1 - row_token(min(2 * t4, G - 1)) : 0;
            const int hide1 = kMulti ? Sq - 1 - row_token(min(2 * t4 + 1, G - 1)) : 0;
            ok = dec_consume_key_rows<kMulti, T, D>(p, bars, &abort_flag, sK, sV, mo, ml, warp, lane, q_col, hide0, hide1,
                                                    len, k_begin, k_end, n_tiles);
        } else {
        // Q as A fragments for the D / 16 k-steps (rows >= G are zero)
        uint32_t qa[D / 16][4];
        {
            const __half* q_lo = static_cast<const __half*>(p.q) + row_index(g) * D;
            const __half* q_hi = static_cast<const __half*>(p.q) + row_index(g + 8) * D;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const int k0 = ks * 16 + 2 * t4;
                qa[ks][0] = (g < G) ? *reinterpret_cast<const uint32_t*>(q_lo + k0) : 0u;
                qa[ks][1] = (g + 8 < G) ? *reinterpret_cast<const uint32_t*>(q_hi + k0) : 0u;
                qa[ks][2] = (g < G) ? *reinterpret_cast<const uint32_t*>(q_lo + k0 + 8) : 0u;
                qa[ks][3] = (g + 8 < G) ? *reinterpret_cast<const uint32_t*>(q_hi + k0 + 8) : 0u;
            }
        }
        // keys an earlier query token must not see: the last Sq - 1 - t of the sequence
        const int hide_lo = kMulti ? Sq - 1 - row_token(g) : 0;
        const int hide_hi = kMulti ? Sq - 1 - row_token(min(g + 8, G - 1)) : 0;
        float o[D / 8][4];
#pragma unroll
        for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;  // rows g and g + 8
        const int key_w = warp * 32;  // this warp's keys inside a tile

        for (int t = 0; t < n_tiles; ++t) {
            const int st = t % kStages;
            const uint32_t parity = (t / kStages) & 1;
            const int valid = min(kDecTile, k_end - (k_begin + t * kDecTile)) - key_w;  // valid keys of this warp's 32
            ok = mbar_wait(smem_u32(&bars[st]), parity, &abort_flag, 20);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            float sc[4][4];
            if (valid > 0) {
                // ---- S = Q K^T for this warp's four blocks of 8 keys
                const uint32_t kt = sK + st * kTileB;
#pragma unroll
                for (int nb = 0; nb < 4; ++nb) {
                    sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
                    const int key = key_w + nb * 8 + (lane & 7);
#pragma unroll
                    for (int c4 = 0; c4 < D / 32; ++c4) {  // 4 d-chunks of 8 per ldmatrix.x4 = two k-steps
                        const int chunk = c4 * 4 + (lane >> 3);
                        const uint32_t addr = kt + (chunk >> 3) * kDecHalfBytes + key * 128 + (((chunk & 7) ^ (key & 7)) << 4);
                        uint32_t b0, b1, b2, b3;
                        ldsm_x4(addr, b0, b1, b2, b3);
                        if (std::is_same<T, __nv_bfloat16>::value) {
                            mma_16816_bf16(sc[nb], qa[2 * c4], b0, b1);
                            mma_16816_bf16(sc[nb], qa[2 * c4 + 1], b2, b3);
                        } else {
                            mma_16816(sc[nb], qa[2 * c4], b0, b1);
                            mma_16816(sc[nb], qa[2 * c4 + 1], b2, b3);
                        }
                    }
                }
                // ---- mask, running max, probabilities
                // keys of this warp's 32 that the row may see: all valid ones, minus (several query
                // rows) those among the sequence's last that came after the row's token
                const int seen_lo = kMulti ? min(valid, len - hide_lo - (k_begin + t * kDecTile) - key_w) : valid;
                const int seen_hi = kMulti ? min(valid, len - hide_hi - (k_begin + t * kDecTile) - key_w) : valid;
                float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
                for (int nb = 0; nb < 4; ++nb) {
                    const int k0 = nb * 8 + 2 * t4;
                    if (k0 >= seen_lo) sc[nb][0] = -INFINITY;
                    if (k0 + 1 >= seen_lo) sc[nb][1] = -INFINITY;
                    if (k0 >= seen_hi) sc[nb][2] = -INFINITY;
                    if (k0 + 1 >= seen_hi) sc[nb][3] = -INFINITY;
                    mx_lo = fmaxf(mx_lo, fmaxf(sc[nb][0], sc[nb][1]));
                    mx_hi = fmaxf(mx_hi, fmaxf(sc[nb][2], sc[nb][3]));
                }
                mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
                mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
                mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
                mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
                // finite when key 0 of the warp is visible (always with one query row; an earlier
                // token of several may see none of the warp's keys: its state then stays empty)
                const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
                const float a_lo = (m_lo == -INFINITY) ? 0.f : fast_exp2((m_lo - mn_lo) * p.scale_log2);
                const float a_hi = (m_hi == -INFINITY) ? 0.f : fast_exp2((m_hi - mn_hi) * p.scale_log2);
                m_lo = mn_lo;
                m_hi = mn_hi;
                const float nm_lo = (mn_lo == -INFINITY) ? 0.f : -mn_lo * p.scale_log2;
                const float nm_hi = (mn_hi == -INFINITY) ? 0.f : -mn_hi * p.scale_log2;
                float s_lo = 0.f, s_hi = 0.f;
#pragma unroll
                for (int nb = 0; nb < 4; ++nb) {
                    const int k0 = nb * 8 + 2 * t4;
                    sc[nb][0] = (k0 < seen_lo) ? fast_exp2(fmaf(sc[nb][0], p.scale_log2, nm_lo)) : 0.f;
                    sc[nb][1] = (k0 + 1 < seen_lo) ? fast_exp2(fmaf(sc[nb][1], p.scale_log2, nm_lo)) : 0.f;
                    sc[nb][2] = (k0 < seen_hi) ? fast_exp2(fmaf(sc[nb][2], p.scale_log2, nm_hi)) : 0.f;
                    sc[nb][3] = (k0 + 1 < seen_hi) ? fast_exp2(fmaf(sc[nb][3], p.scale_log2, nm_hi)) : 0.f;
                    s_lo += sc[nb][0] + sc[nb][1];
                    s_hi += sc[nb][2] + sc[nb][3];
                }
                l_lo = l_lo * a_lo + s_lo;  // per-thread partial of the row sum (the quad is summed at the end)
                l_hi = l_hi * a_hi + s_hi;
#pragma unroll
                for (int i = 0; i < D / 8; ++i) {
                    o[i][0] *= a_lo;
                    o[i][1] *= a_lo;
                    o[i][2] *= a_hi;
                    o[i][3] *= a_hi;
                }
            }
            ok = mbar_wait(smem_u32(&bars[kStages + st]), parity, &abort_flag, 21);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (valid > 0) {
                const uint32_t vt = sV + st * kTileB;
                if (valid < 32) {
                    // rows past the sequence may hold NaN bits: zero them (0 * NaN would poison O)
                    for (int i = lane; i < (32 - valid) * (D / 8); i += 32) {
                        const int key = key_w + valid + i / (D / 8), ch = i % (D / 8);
                        const uint32_t addr = vt + (ch >> 3) * kDecHalfBytes + key * 128 + (((ch & 7) ^ (key & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
                    }
                    __syncwarp();
                }
                // ---- O += P V: two k-steps of 16 keys, D / 8 blocks of 8 output columns
#pragma unroll
                for (int k2 = 0; k2 < 2; ++k2) {
                    uint32_t pa[4];
                    pa[0] = pack2<T>(sc[2 * k2][0], sc[2 * k2][1]);
                    pa[1] = pack2<T>(sc[2 * k2][2], sc[2 * k2][3]);
                    pa[2] = pack2<T>(sc[2 * k2 + 1][0], sc[2 * k2 + 1][1]);
                    pa[3] = pack2<T>(sc[2 * k2 + 1][2], sc[2 * k2 + 1][3]);
                    const int key = key_w + k2 * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                    for (int n2 = 0; n2 < D / 16; ++n2) {  // two output blocks per ldmatrix.x4.trans
                        const int ch = n2 * 2 + (lane >> 4);
                        const uint32_t addr = vt + (ch >> 3) * kDecHalfBytes + key * 128 + (((ch & 7) ^ (key & 7)) << 4);
                        uint32_t b0, b1, b2, b3;
                        ldsm_x4_trans(addr, b0, b1, b2, b3);
                        if (std::is_same<T, __nv_bfloat16>::value) {
                            mma_16816_bf16(o[2 * n2], pa, b0, b1);
                            mma_16816_bf16(o[2 * n2 + 1], pa, b2, b3);
                        } else {
                            mma_16816(o[2 * n2], pa, b0, b1);
                            mma_16816(o[2 * n2 + 1], pa, b2, b3);
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars[2 * kStages + st]));
        }

        // ---- merge the four warps' states and write this chunk's partial result
        // (all tiles this CTA requested have been consumed by every warp before the barrier below,
        // so the ring can be reused as the merge buffer)
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (ok) {
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                const int col = i * 8 + 2 * t4;
                *reinterpret_cast<float2*>(&mo[(warp * 16 + g) * D + col]) = make_float2(o[i][0], o[i][1]);
                *reinterpret_cast<float2*>(&mo[(warp * 16 + g + 8) * D + col]) = make_float2(o[i][2], o[i][3]);
            }
            if (t4 == 0) {
                ml[(warp * 16 + g) * 2] = m_lo;
                ml[(warp * 16 + g) * 2 + 1] = l_lo;
                ml[(warp * 16 + g + 8) * 2] = m_hi;
                ml[(warp * 16 + g + 8) * 2 + 1] = l_hi;
            }
        }
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (ok && tid < D) {
            for (int r = 0; r < G; ++r) {  // thread `tid` owns output column `tid` of every row
                float M = -INFINITY;
#pragma unroll
                for (int w = 0; w < 4; ++w) M = fmaxf(M, ml[(w * 16 + r) * 2]);
                float l = 0.f, acc = 0.f;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const float mw = ml[(w * 16 + r) * 2];
                    const float sw = (mw == -INFINITY) ? 0.f : fast_exp2((mw - M) * p.scale_log2);
                    l += sw * ml[(w * 16 + r) * 2 + 1];
                    acc += sw * mo[(w * 16 + r) * D + tid];
                }
                // (l == 0: a query token that sees none of this chunk's keys)
                const float out = (l > 0.f) ? acc / l : 0.f;
                const float lse = (l > 0.f) ? (M * p.scale_log2 + log2f(l)) * 0.6931471805599453f : -INFINITY;
                if (p.o_final != nullptr) {   // the only chunk: this is the result
                    static_cast<T*>(p.o_final)[row_index(r) * D + tid] = T(out);
                    if (tid == 0 && p.lse_final) p.lse_final[lse_index(r)] = lse;
                } else {
                    const long long slot = row_index(r) * p.n_chunks + c;
                    p.o_part[slot * D + tid] = out;
                    if (tid == 0) p.lse_part[slot] = lse;
                }
            }
        }
    }
}

// Merge of the per-chunk partials (rowmax/rowsum recurrence applied across chunks):
//   M = max_c LSE_c, w_c = exp(LSE_c - M), O = sum_c w_c O_c / sum_c w_c, LSE = M + ln sum_c w_c.
// grid: B * Sq * Hq blocks of D threads (row = (b, token, head)), thread t owns output dim t.
template <typename T, int D = 128>
__global__ void __launch_bounds__(128)
fa_decode_combine_kernel(const DecodeParams p, T* o, float* lse) {
    const int bh = blockIdx.x;
    const int b = bh / (p.Hq * p.Sq);
    // lse is [B,Hq,Sq]
    const long long lse_at = ((long long)b * p.Hq + bh % p.Hq) * p.Sq + (bh / p.Hq) % p.Sq;
    const int tid = threadIdx.x;
    int len = p.seqlens[b];
    len = max(0, min(len, p.Smax));
    const int nc = (len + p.chunk - 1) / p.chunk;
    // launched as a programmatic dependent of the split kernel: its partial results are
    // complete and visible from here on (returns at once in an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const float* lp = p.lse_part + (long long)bh * p.n_chunks;
    const float* op = p.o_part + (long long)bh * p.n_chunks * D;
    float M = -INFINITY;
    for (int c = 0; c < nc; ++c) M = fmaxf(M, lp[c]);
    if (nc == 0 || M == -INFINITY) {   // no keys, or (several query rows) a token that sees none
        o[(long long)bh * D + tid] = T(0.f);
        if (lse && tid == 0) lse[lse_at] = -INFINITY;
        return;
    }
    float wsum = 0.f, acc = 0.f;
    for (int c = 0; c < nc; ++c) {
        const float w = __expf(lp[c] - M);
        wsum += w;
        acc = fmaf(w, op[(long long)c * D + tid], acc);
    }
    o[(long long)bh * D + tid] = T(acc / wsum);
    if (lse && tid == 0) lse[lse_at] = M + logf(wsum);
}

}  // namespace fa
