// Decode-stage attention over an 8-bit cache (Appendix D.2 runs the operator with 8-bit operands;
// here the cached K and V are FP8 e4m3 with one scale each, the queries and the probabilities
// stay fp16): the structure of the split kernel of decode.cuh with half the cache bytes per key.
// K and V tiles of 128 keys x 128 bytes arrive through TMA (one 128-byte-swizzled box each); the
// 8-bit rows go through ldmatrix as if they were 16-bit elements and are widened to fp16 pairs in
// registers (cvt.rn.f16x2.e4m3x2) on their way into warp-level m16n8k16 MMAs, whose rows are keys
// and whose columns are query heads (the products are taken transposed).  The key scale is
// folded into the softmax scale, the value scale into the partial output.
#pragma once

#include "decode.cuh"

namespace fa {

constexpr int kDec8Stages = 3;            // ring slots of one K and one V tile: 97 KiB per CTA, two CTAs per SM
constexpr int kDec8TileBytes = 16384;   // 128 keys x 128 one-byte elements
constexpr int kDec8Warps = 4;            // consumer warps, 32 keys of every tile each (as in the fp16 kernel)
constexpr int kDec8Threads = (kDec8Warps + 1) * 32;

// Four e4m3 bytes -> two fp16 pairs: (byte 0, byte 1) and (byte 2, byte 3).  (Widening on the
// integer pipe instead -- the byte moved into the upper half of a halfword with its low seven
// bits shifted down by one is the fp16 pattern of the value times 2^-8 -- is exact too, but its
// eight integer instructions per four bytes were slower: 2.51 against 1.89 ms on the MHA case.)
__device__ __forceinline__ void e4m3x4_to_f16x2x2(uint32_t in, uint32_t& lo, uint32_t& hi) {
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.rn.f16x2.e4m3x2 %0, a;\n\tcvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
        : "=r"(lo), "=r"(hi)
        : "r"(in));
}

// A pair of bf16 values as a pair of fp16 values: exact for magnitudes in fp16's normal range
// (bf16 carries 8 significant bits, fp16 11); larger ones become infinities, smaller ones lose bits.
__device__ __forceinline__ uint32_t bf16x2_to_f16x2(uint32_t v) {
    const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v));
    const __half2 h = __floats2half2_rn(f.x, f.y);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// grid: (Hkv * ceil(g / 16), n_chunks, B) with g = Hq / Hkv (the kv head fastest, see decode.cuh)
template <int NB>
__global__ void __launch_bounds__(kDec8Threads, 2)
fa_decode_split_fp8_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                           const DecodeParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sK = smem_base;
    const uint32_t sV = smem_base + kDec8Stages * kDec8TileBytes;
    __shared__ __align__(8) uint64_t bars[3 * kDec8Stages];  // K full, V full, slot empty
    __shared__ volatile uint32_t abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int c = blockIdx.y;
    const int b = blockIdx.z;
    const int g_all = p.Hq / p.Hkv;
    const int n_sub = (g_all + 15) / 16;           // CTAs per kv head when more than 16 heads share it
    const int hk = blockIdx.x / n_sub;
    const int sub = blockIdx.x % n_sub;
    const int h0 = hk * g_all + sub * 16;          // first query head of this CTA
    const int G = min(16, g_all - sub * 16);       // its number of query heads

    int len = p.seqlens[b];
    len = max(0, min(len, p.Smax));
    const int k_begin = c * p.chunk;
    const int k_end = min(len, k_begin + p.chunk);
    if (k_begin >= k_end) {  // uniform for the CTA
        if (p.o_final != nullptr && tid < 128) {   // a sequence without keys, and nobody else writes its rows
            for (int r = 0; r < G; ++r) {
                // (sixteen zero bits are 0.0 in fp16 and in bf16)
                static_cast<__half*>(p.o_final)[((long long)b * p.Hq + h0 + r) * 128 + tid] = __half(0.f);
                if (tid == 0 && p.lse_final) p.lse_final[(long long)b * p.Hq + h0 + r] = -INFINITY;
            }
        }
        return;
    }
    const int n_tiles = (k_end - k_begin + kDecTile - 1) / kDecTile;

    if (tid == 0) {
        for (int i = 0; i < 2 * kDec8Stages; ++i) mbar_init(smem_u32(&bars[i]), 1);
        for (int i = 0; i < kDec8Stages; ++i) mbar_init(smem_u32(&bars[2 * kDec8Stages + i]), kDec8Warps);  // one arrival per consumer warp
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();

    if (warp == kDec8Warps) {
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
                const int st = t % kDec8Stages;
                const uint32_t bk = smem_u32(&bars[st]), bv = smem_u32(&bars[kDec8Stages + st]);
                const int row0 = k_begin + t * kDecTile;
                const int cur = pg_next;
                if (t + 1 < n_tiles) pg_next = lookup(row0 + kDecTile);
                bool ok = true;
                if (lane == 0) ok = mbar_wait(smem_u32(&bars[2 * kDec8Stages + st]), ((t / kDec8Stages) & 1) ^ 1, &abort_flag, 22);
                if (!__shfl_sync(0xffffffffu, ok, 0)) break;
                const int live = min(n_sub, (k_end - row0 + ps - 1) / ps);   // pages of this tile that hold keys
                if (lane == 0) {
                    mbar_expect_tx(bk, (uint32_t)(live * ps) * 128u);
                    mbar_expect_tx(bv, (uint32_t)(live * ps) * 128u);
                }
                __syncwarp();
                if (lane < live) {
                    const uint32_t offs = (uint32_t)(lane * ps) * 128u;
                    tma_load_4d_hint(sK + st * kDec8TileBytes + offs, &tm_k, bk, 0, hk, 0, cur, stream_policy);
                    tma_load_4d_hint(sV + st * kDec8TileBytes + offs, &tm_v, bv, 0, hk, 0, cur, stream_policy);
                }
            }
        } else if (lane == 0) {
            int page_next = table ? table[k_begin / p.page_size] : 0;
            for (int t = 0; t < n_tiles; ++t) {
                const int st = t % kDec8Stages;
                const uint32_t bk = smem_u32(&bars[st]), bv = smem_u32(&bars[kDec8Stages + st]);
                int row0 = k_begin + t * kDecTile;  // first key of the tile within the sequence
                int slab = b;                        // outermost coordinate: the sequence, or the page
                if (table) {
                    slab = page_next;
                    if (t + 1 < n_tiles) page_next = table[(row0 + kDecTile) / p.page_size];
                    row0 %= p.page_size;
                }
                if (!mbar_wait(smem_u32(&bars[2 * kDec8Stages + st]), ((t / kDec8Stages) & 1) ^ 1, &abort_flag, 22)) break;
                mbar_expect_tx(bk, kDec8TileBytes);
                tma_load_4d_hint(sK + st * kDec8TileBytes, &tm_k, bk, 0, hk, row0, slab, stream_policy);
                mbar_expect_tx(bv, kDec8TileBytes);
                tma_load_4d_hint(sV + st * kDec8TileBytes, &tm_v, bv, 0, hk, row0, slab, stream_policy);
            }
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------------------- consumers
        // The products are taken transposed, S^T = K q^T and O^T = V^T P^T: the 16 rows of an
        // MMA are keys (or output columns) and its 8 columns are query heads, so that a group of
        // up to 8 heads costs half the MMAs of the head-major form (NB = 1; NB = 2 for 9..16 heads).
        const int g = lane >> 2, t4 = lane & 3;
        // q^T as B fragments: column g = head 8 nbk + g; a k-step's rows (2 t4, 2 t4 + 1) and
        // (2 t4 + 8, 2 t4 + 9) are d = 16 ks + 4 t4 .. + 3, the order in which a thread receives a
        // key's bytes from ldmatrix (the dot product over d does not care about the order)
        uint32_t qb[NB][8][2];
        {
            const __half* qp = static_cast<const __half*>(p.q) + ((long long)b * p.Hq + h0) * 128;
#pragma unroll
            for (int nbk = 0; nbk < NB; ++nbk) {
                const int head = nbk * 8 + g;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const int d0 = ks * 16 + 4 * t4;
                    qb[nbk][ks][0] = (head < G) ? *reinterpret_cast<const uint32_t*>(qp + head * 128 + d0) : 0u;
                    qb[nbk][ks][1] = (head < G) ? *reinterpret_cast<const uint32_t*>(qp + head * 128 + d0 + 2) : 0u;
                    if (p.bf16_io) {   // the products run in fp16 (the widened cache is fp16): q goes there too
                        qb[nbk][ks][0] = bf16x2_to_f16x2(qb[nbk][ks][0]);
                        qb[nbk][ks][1] = bf16x2_to_f16x2(qb[nbk][ks][1]);
                    }
                }
            }
        }
        // O^T: block c holds output columns 16 c .. 16 c + 15 as MMA rows (row g = column
        // 16 c + 2 g, row g + 8 = column 16 c + 2 g + 1) for heads 8 nbk + 2 t4 and + 1
        float o[8][NB][4];
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int nbk = 0; nbk < NB; ++nbk) o[i][nbk][0] = o[i][nbk][1] = o[i][nbk][2] = o[i][nbk][3] = 0.f;
        // running max and (per-thread partial) sum for heads 8 nbk + 2 t4 (index 0) and + 1 (index 1)
        float m_run[NB][2], l_run[NB][2];
#pragma unroll
        for (int nbk = 0; nbk < NB; ++nbk) {
            m_run[nbk][0] = m_run[nbk][1] = -INFINITY;
            l_run[nbk][0] = l_run[nbk][1] = 0.f;
        }
        const int key_w = warp * 32;  // this warp's keys inside a tile
        bool ok = true;

        for (int t = 0; t < n_tiles; ++t) {
            const int st = t % kDec8Stages;
            const uint32_t parity = (t / kDec8Stages) & 1;
            const int valid = min(kDecTile, k_end - (k_begin + t * kDecTile)) - key_w;  // valid keys of this warp's 32
            ok = mbar_wait(smem_u32(&bars[st]), parity, &abort_flag, 20);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            uint32_t pt[2][NB][2];   // P^T as B fragments per 16-key step
            if (valid > 0) {
                // ---- S^T = K q^T: two blocks of 16 keys
                float sc[2][NB][4];  // (key 16 mb + g, heads 2 t4, 2 t4 + 1), (key 16 mb + g + 8, same heads)
                const uint32_t kt = sK + st * kDec8TileBytes;
#pragma unroll
                for (int mb = 0; mb < 2; ++mb) {
#pragma unroll
                    for (int nbk = 0; nbk < NB; ++nbk) sc[mb][nbk][0] = sc[mb][nbk][1] = sc[mb][nbk][2] = sc[mb][nbk][3] = 0.f;
                    const int key = key_w + mb * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {  // two 16-byte chunks (two k-steps) per ldmatrix.x4
                        const int chunk = cc * 2 + (lane >> 4);
                        const uint32_t addr = kt + key * 128 + ((chunk ^ (key & 7)) << 4);
                        // matrices: (keys 0-7, chunk 2 cc), (keys 8-15, chunk 2 cc), (keys 0-7, chunk 2 cc + 1), (keys 8-15, ...)
                        uint32_t w[4];
                        ldsm_x4(addr, w[0], w[1], w[2], w[3]);
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            uint32_t a[4];
                            e4m3x4_to_f16x2x2(w[2 * j], a[0], a[2]);      // keys g: d 4 t4, +1 | +2, +3
                            e4m3x4_to_f16x2x2(w[2 * j + 1], a[1], a[3]);  // keys g + 8
#pragma unroll
                            for (int nbk = 0; nbk < NB; ++nbk)
                                mma_16816(sc[mb][nbk], a, qb[nbk][cc * 2 + j][0], qb[nbk][cc * 2 + j][1]);
                        }
                    }
                }
                // ---- mask, running max, probabilities
#pragma unroll
                for (int nbk = 0; nbk < NB; ++nbk) {
                    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                    for (int mb = 0; mb < 2; ++mb) {
                        const int k_lo = mb * 16 + g;
                        if (k_lo >= valid) sc[mb][nbk][0] = sc[mb][nbk][1] = -INFINITY;
                        if (k_lo + 8 >= valid) sc[mb][nbk][2] = sc[mb][nbk][3] = -INFINITY;
                        mx0 = fmaxf(mx0, fmaxf(sc[mb][nbk][0], sc[mb][nbk][2]));
                        mx1 = fmaxf(mx1, fmaxf(sc[mb][nbk][1], sc[mb][nbk][3]));
                    }
#pragma unroll
                    for (int sh = 4; sh <= 16; sh <<= 1) {  // over the lanes that hold other keys of the same heads
                        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
                        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
                    }
                    const float mn0 = fmaxf(m_run[nbk][0], mx0), mn1 = fmaxf(m_run[nbk][1], mx1);  // finite: key 0 of the warp is valid
                    const float a0 = (m_run[nbk][0] == -INFINITY) ? 0.f : fast_exp2((m_run[nbk][0] - mn0) * p.scale_log2);
                    const float a1 = (m_run[nbk][1] == -INFINITY) ? 0.f : fast_exp2((m_run[nbk][1] - mn1) * p.scale_log2);
                    m_run[nbk][0] = mn0;
                    m_run[nbk][1] = mn1;
                    const float nm0 = -mn0 * p.scale_log2, nm1 = -mn1 * p.scale_log2;
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int mb = 0; mb < 2; ++mb) {
                        const int k_lo = mb * 16 + g;
                        float* e = sc[mb][nbk];
                        e[0] = (k_lo < valid) ? fast_exp2(fmaf(e[0], p.scale_log2, nm0)) : 0.f;
                        e[1] = (k_lo < valid) ? fast_exp2(fmaf(e[1], p.scale_log2, nm1)) : 0.f;
                        e[2] = (k_lo + 8 < valid) ? fast_exp2(fmaf(e[2], p.scale_log2, nm0)) : 0.f;
                        e[3] = (k_lo + 8 < valid) ? fast_exp2(fmaf(e[3], p.scale_log2, nm1)) : 0.f;
                        s0 += e[0] + e[2];
                        s1 += e[1] + e[3];
                        // (keys g | heads 2 t4, 2 t4 + 1) -> transposed: (head g | keys 2 t4, 2 t4 + 1), the B fragment
                        __half2 lo = __floats2half2_rn(e[0], e[1]), hi = __floats2half2_rn(e[2], e[3]);
                        asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pt[mb][nbk][0]) : "r"(*reinterpret_cast<uint32_t*>(&lo)));
                        asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(pt[mb][nbk][1]) : "r"(*reinterpret_cast<uint32_t*>(&hi)));
                    }
                    l_run[nbk][0] = l_run[nbk][0] * a0 + s0;  // per-thread partial of the sum over keys (reduced at the end)
                    l_run[nbk][1] = l_run[nbk][1] * a1 + s1;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        o[i][nbk][0] *= a0;
                        o[i][nbk][1] *= a1;
                        o[i][nbk][2] *= a0;
                        o[i][nbk][3] *= a1;
                    }
                }
            }
            ok = mbar_wait(smem_u32(&bars[kDec8Stages + st]), parity, &abort_flag, 21);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (valid > 0) {
                const uint32_t vt = sV + st * kDec8TileBytes;
                if (valid < 32) {
                    // rows past the sequence may hold NaN bits: zero them (0 * NaN would poison O)
                    for (int i = lane; i < (32 - valid) * 8; i += 32) {
                        const int key = key_w + valid + (i >> 3), ch = i & 7;
                        const uint32_t addr = vt + key * 128 + ((ch ^ (key & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
                    }
                    __syncwarp();
                }
                // ---- O^T += V^T P^T: two k-steps of 16 keys, eight blocks of 16 output columns
#pragma unroll
                for (int k2 = 0; k2 < 2; ++k2) {
                    const int key = key_w + k2 * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {  // two 16-byte chunks per ldmatrix.x4.trans
                        const int ch = q4 * 2 + (lane >> 4);
                        const uint32_t addr = vt + key * 128 + ((ch ^ (key & 7)) << 4);
                        // matrices: (keys 0-7, chunk 2 q4), (keys 8-15, chunk 2 q4), (keys 0-7, chunk 2 q4 + 1), (keys 8-15, ...)
                        uint32_t w[4];
                        ldsm_x4_trans(addr, w[0], w[1], w[2], w[3]);
                        // a transposed 16-bit element is the byte pair (2g, 2g + 1) of one key, held for keys
                        // 2 t4 and 2 t4 + 1; regrouped by byte: column 2g of both keys, then column 2g + 1
                        uint32_t ev[4], od[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint32_t tw;
                            asm("prmt.b32 %0, %1, %1, 0x3120;" : "=r"(tw) : "r"(w[j]));
                            e4m3x4_to_f16x2x2(tw, ev[j], od[j]);
                        }
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            // rows g: even columns, rows g + 8: odd columns; k: keys 2 t4.. | keys 2 t4 + 8..
                            const uint32_t a[4] = {ev[2 * j], od[2 * j], ev[2 * j + 1], od[2 * j + 1]};
#pragma unroll
                            for (int nbk = 0; nbk < NB; ++nbk)
                                mma_16816(o[q4 * 2 + j][nbk], a, pt[k2][nbk][0], pt[k2][nbk][1]);
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars[2 * kDec8Stages + st]));
        }

        // ---- merge the warps' states and write this chunk's partial result (the ring is free:
        // every warp has consumed all tiles this CTA requested before the barrier below)
#pragma unroll
        for (int nbk = 0; nbk < NB; ++nbk)
#pragma unroll
            for (int sh = 4; sh <= 16; sh <<= 1) {
                l_run[nbk][0] += __shfl_xor_sync(0xffffffffu, l_run[nbk][0], sh);
                l_run[nbk][1] += __shfl_xor_sync(0xffffffffu, l_run[nbk][1], sh);
            }
        float* mo = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));  // [warps][16 heads][128]
        float* ml = mo + kDec8Warps * 16 * 128;                                              // [warps][16][2]: m, l
        asm volatile("bar.sync 1, %0;" ::"n"(kDec8Warps * 32) : "memory");
        if (ok) {
#pragma unroll
            for (int nbk = 0; nbk < NB; ++nbk) {
                const int head = nbk * 8 + 2 * t4;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int col = i * 16 + 2 * g;
                    mo[(warp * 16 + head) * 128 + col] = o[i][nbk][0];
                    mo[(warp * 16 + head + 1) * 128 + col] = o[i][nbk][1];
                    mo[(warp * 16 + head) * 128 + col + 1] = o[i][nbk][2];
                    mo[(warp * 16 + head + 1) * 128 + col + 1] = o[i][nbk][3];
                }
                if (g == 0) {
                    ml[(warp * 16 + head) * 2] = m_run[nbk][0];
                    ml[(warp * 16 + head) * 2 + 1] = l_run[nbk][0];
                    ml[(warp * 16 + head + 1) * 2] = m_run[nbk][1];
                    ml[(warp * 16 + head + 1) * 2 + 1] = l_run[nbk][1];
                }
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kDec8Warps * 32) : "memory");
        if (ok) {
            const int col = tid & 127;   // a thread owns one output column
            for (int r = tid >> 7; r < G; r += kDec8Warps / 4) {
                float M = -INFINITY;
#pragma unroll
                for (int w = 0; w < kDec8Warps; ++w) M = fmaxf(M, ml[(w * 16 + r) * 2]);
                float l = 0.f, acc = 0.f;
#pragma unroll
                for (int w = 0; w < kDec8Warps; ++w) {
                    const float mw = ml[(w * 16 + r) * 2];
                    const float sw = (mw == -INFINITY) ? 0.f : fast_exp2((mw - M) * p.scale_log2);
                    l += sw * ml[(w * 16 + r) * 2 + 1];
                    acc += sw * mo[(w * 16 + r) * 128 + col];
                }
                const float out = acc / l * p.v_scale;
                const float lse = (M * p.scale_log2 + log2f(l)) * 0.6931471805599453f;
                if (p.o_final != nullptr) {   // the only chunk: this is the result
                    const long long row = (long long)b * p.Hq + h0 + r;
                    if (p.bf16_io) static_cast<__nv_bfloat16*>(p.o_final)[row * 128 + col] = __nv_bfloat16(out);
                    else static_cast<__half*>(p.o_final)[row * 128 + col] = __half(out);
                    if (col == 0 && p.lse_final) p.lse_final[row] = lse;
                } else {
                    const long long slot = ((long long)b * p.Hq + h0 + r) * p.n_chunks + c;
                    p.o_part[slot * 128 + col] = out;
                    if (col == 0) p.lse_part[slot] = lse;
                }
            }
        }
    }
}

}  // namespace fa
