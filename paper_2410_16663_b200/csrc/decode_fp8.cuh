// Decode-stage attention over an 8-bit cache (Appendix D.2 runs the operator with 8-bit operands;
// here the cached K and V are FP8 e4m3 with one scale each, the queries and the probabilities
// stay fp16): the split kernel of decode.cuh with half the cache bytes per key.  K and V tiles of
// 128 keys x 128 bytes arrive through TMA (one 128-byte-swizzled box each); the 8-bit rows go
// through ldmatrix as if they were 16-bit elements and are widened to fp16 pairs in registers
// (cvt.rn.f16x2.e4m3x2) on their way into the same warp-level m16n8k16 MMAs.  The key scale is
// folded into the softmax scale, the value scale into the partial output.
#pragma once

#include "decode.cuh"

namespace fa {

constexpr int kDec8Stages = 4;
constexpr int kDec8TileBytes = 16384;   // 128 keys x 128 one-byte elements
#ifndef FA_DEC8_WARPS
#define FA_DEC8_WARPS 4
#endif
// Consumer warps: each owns kDec8KeysPerWarp keys of every tile.  Four warps of 32 keys as in the
// fp16 kernel; eight warps of 16 keys (two per scheduler) were 5 % slower: the kernel is bound
// by the throughput of the conversions and the warp-level MMAs, not by their latency.
constexpr int kDec8Warps = FA_DEC8_WARPS;
constexpr int kDec8KeysPerWarp = kDecTile / kDec8Warps;
constexpr int kDec8Threads = (kDec8Warps + 1) * 32;
static_assert(kDec8KeysPerWarp == 16 || kDec8KeysPerWarp == 32, "a warp owns one or two MMA k-steps of keys");

// Four e4m3 bytes -> two fp16 pairs: (byte 0, byte 1) and (byte 2, byte 3).  (Widening on the
// integer pipe instead -- the byte moved into the upper half of a halfword with its low seven
// bits shifted down by one is the fp16 pattern of the value times 2^-8 -- is exact too, but its
// eight integer instructions per four bytes were slower: 2.51 against 1.89 ms on the MHA case.)
__device__ __forceinline__ void e4m3x4_to_f16x2x2(uint32_t in, uint32_t& lo, uint32_t& hi) {
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.rn.f16x2.e4m3x2 %0, a;\n\tcvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
        : "=r"(lo), "=r"(hi)
        : "r"(in));
}

// grid: (n_chunks, Hkv * ceil(g / 16), B) with g = Hq / Hkv
__global__ void __launch_bounds__(kDec8Threads, 1)
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
    const int c = blockIdx.x;
    const int b = blockIdx.z;
    const int g_all = p.Hq / p.Hkv;
    const int n_sub = (g_all + 15) / 16;           // CTAs per kv head when more than 16 heads share it
    const int hk = blockIdx.y / n_sub;
    const int sub = blockIdx.y % n_sub;
    const int h0 = hk * g_all + sub * 16;          // first query head of this CTA
    const int G = min(16, g_all - sub * 16);       // its number of query heads

    int len = p.seqlens[b];
    len = max(0, min(len, p.Smax));
    const int k_begin = c * p.chunk;
    const int k_end = min(len, k_begin + p.chunk);
    if (k_begin >= k_end) return;  // uniform for the CTA
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
        if (lane == 0) {
            // paged cache: the page of a tile is looked up one tile ahead of its loads, so that
            // the table read is not on the path that refills a freed slot
            const int* table = p.block_table ? p.block_table + (long long)b * p.table_stride : nullptr;
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
                tma_load_4d(sK + st * kDec8TileBytes, &tm_k, bk, 0, hk, row0, slab);
                mbar_expect_tx(bv, kDec8TileBytes);
                tma_load_4d(sV + st * kDec8TileBytes, &tm_v, bv, 0, hk, row0, slab);
            }
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------------------- consumers
        const int g = lane >> 2, t4 = lane & 3;  // fragment row (query head g and g + 8) and column pair
        // Q as A fragments for the eight k-steps of d = 128 (rows >= G are zero).  A k-step
        // covers 16 consecutive d, but in the order the 8-bit K rows come out of ldmatrix: a
        // thread's four bytes of a 16-byte chunk are d = 4 t4 .. 4 t4 + 3, which become the
        // k-step's columns (2 t4, 2 t4 + 1) and (2 t4 + 8, 2 t4 + 9).  The dot product over d does
        // not care about the order as long as Q uses the same one.
        uint32_t qa[8][4];
        {
            const __half* qb = static_cast<const __half*>(p.q) + ((long long)b * p.Hq + h0) * 128;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const int k0 = ks * 16 + 4 * t4;
                qa[ks][0] = (g < G) ? *reinterpret_cast<const uint32_t*>(qb + g * 128 + k0) : 0u;
                qa[ks][1] = (g + 8 < G) ? *reinterpret_cast<const uint32_t*>(qb + (g + 8) * 128 + k0) : 0u;
                qa[ks][2] = (g < G) ? *reinterpret_cast<const uint32_t*>(qb + g * 128 + k0 + 2) : 0u;
                qa[ks][3] = (g + 8 < G) ? *reinterpret_cast<const uint32_t*>(qb + (g + 8) * 128 + k0 + 2) : 0u;
            }
        }
        float o[16][4];
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;  // rows g and g + 8
        const int key_w = warp * kDec8KeysPerWarp;  // this warp's keys inside a tile
        bool ok = true;

        for (int t = 0; t < n_tiles; ++t) {
            const int st = t % kDec8Stages;
            const uint32_t parity = (t / kDec8Stages) & 1;
            const int valid = min(kDecTile, k_end - (k_begin + t * kDecTile)) - key_w;  // valid keys of this warp's 32
            ok = mbar_wait(smem_u32(&bars[st]), parity, &abort_flag, 20);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            float sc[kDec8KeysPerWarp / 8][4];
            if (valid > 0) {
                // ---- S = Q K^T for this warp's four blocks of 8 keys
                const uint32_t kt = sK + st * kDec8TileBytes;
#pragma unroll
                for (int nb = 0; nb < kDec8KeysPerWarp / 8; ++nb) {
                    sc[nb][0] = sc[nb][1] = sc[nb][2] = sc[nb][3] = 0.f;
                    const int key = key_w + nb * 8 + (lane & 7);
#pragma unroll
                    for (int hf = 0; hf < 2; ++hf) {  // 4 chunks of 16 bytes per ldmatrix.x4 = four k-steps
                        const int chunk = hf * 4 + (lane >> 3);
                        const uint32_t addr = kt + key * 128 + ((chunk ^ (key & 7)) << 4);
                        uint32_t w[4];
                        ldsm_x4(addr, w[0], w[1], w[2], w[3]);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint32_t b0, b1;   // d = 4 t4, 4 t4 + 1 and 4 t4 + 2, 4 t4 + 3 of the chunk, as fp16 pairs
                            e4m3x4_to_f16x2x2(w[j], b0, b1);
                            mma_16816(sc[nb], qa[hf * 4 + j], b0, b1);
                        }
                    }
                }
                // ---- mask, running max, probabilities
                float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
                for (int nb = 0; nb < kDec8KeysPerWarp / 8; ++nb) {
                    const int k0 = nb * 8 + 2 * t4;
                    if (k0 >= valid) sc[nb][0] = sc[nb][2] = -INFINITY;
                    if (k0 + 1 >= valid) sc[nb][1] = sc[nb][3] = -INFINITY;
                    mx_lo = fmaxf(mx_lo, fmaxf(sc[nb][0], sc[nb][1]));
                    mx_hi = fmaxf(mx_hi, fmaxf(sc[nb][2], sc[nb][3]));
                }
                mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
                mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
                mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
                mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
                const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);  // finite: key 0 of the warp is valid
                const float a_lo = (m_lo == -INFINITY) ? 0.f : fast_exp2((m_lo - mn_lo) * p.scale_log2);
                const float a_hi = (m_hi == -INFINITY) ? 0.f : fast_exp2((m_hi - mn_hi) * p.scale_log2);
                m_lo = mn_lo;
                m_hi = mn_hi;
                const float nm_lo = -mn_lo * p.scale_log2, nm_hi = -mn_hi * p.scale_log2;
                float s_lo = 0.f, s_hi = 0.f;
#pragma unroll
                for (int nb = 0; nb < kDec8KeysPerWarp / 8; ++nb) {
                    const int k0 = nb * 8 + 2 * t4;
                    sc[nb][0] = (k0 < valid) ? fast_exp2(fmaf(sc[nb][0], p.scale_log2, nm_lo)) : 0.f;
                    sc[nb][1] = (k0 + 1 < valid) ? fast_exp2(fmaf(sc[nb][1], p.scale_log2, nm_lo)) : 0.f;
                    sc[nb][2] = (k0 < valid) ? fast_exp2(fmaf(sc[nb][2], p.scale_log2, nm_hi)) : 0.f;
                    sc[nb][3] = (k0 + 1 < valid) ? fast_exp2(fmaf(sc[nb][3], p.scale_log2, nm_hi)) : 0.f;
                    s_lo += sc[nb][0] + sc[nb][1];
                    s_hi += sc[nb][2] + sc[nb][3];
                }
                l_lo = l_lo * a_lo + s_lo;  // per-thread partial of the row sum (the quad is summed at the end)
                l_hi = l_hi * a_hi + s_hi;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    o[i][0] *= a_lo;
                    o[i][1] *= a_lo;
                    o[i][2] *= a_hi;
                    o[i][3] *= a_hi;
                }
            }
            ok = mbar_wait(smem_u32(&bars[kDec8Stages + st]), parity, &abort_flag, 21);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (valid > 0) {
                const uint32_t vt = sV + st * kDec8TileBytes;
                if (valid < kDec8KeysPerWarp) {
                    // rows past the sequence may hold NaN bits: zero them (0 * NaN would poison O)
                    for (int i = lane; i < (kDec8KeysPerWarp - valid) * 8; i += 32) {
                        const int key = key_w + valid + (i >> 3), ch = i & 7;
                        const uint32_t addr = vt + key * 128 + ((ch ^ (key & 7)) << 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0u) : "memory");
                    }
                    __syncwarp();
                }
                // ---- O += P V: two k-steps of 16 keys, sixteen blocks of 8 output columns
#pragma unroll
                for (int k2 = 0; k2 < kDec8KeysPerWarp / 16; ++k2) {
                    uint32_t pa[4];
                    {
                        __half2 h0 = __floats2half2_rn(sc[2 * k2][0], sc[2 * k2][1]);
                        __half2 h1 = __floats2half2_rn(sc[2 * k2][2], sc[2 * k2][3]);
                        __half2 h2 = __floats2half2_rn(sc[2 * k2 + 1][0], sc[2 * k2 + 1][1]);
                        __half2 h3 = __floats2half2_rn(sc[2 * k2 + 1][2], sc[2 * k2 + 1][3]);
                        pa[0] = *reinterpret_cast<uint32_t*>(&h0);
                        pa[1] = *reinterpret_cast<uint32_t*>(&h1);
                        pa[2] = *reinterpret_cast<uint32_t*>(&h2);
                        pa[3] = *reinterpret_cast<uint32_t*>(&h3);
                    }
                    const int key = key_w + k2 * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {  // two 16-byte chunks (32 output columns) per ldmatrix.x4.trans
                        const int ch = q4 * 2 + (lane >> 4);
                        const uint32_t addr = vt + key * 128 + ((ch ^ (key & 7)) << 4);
                        // matrices: (keys 0-7, chunk 2 q4), (keys 8-15, chunk 2 q4), (keys 0-7, chunk 2 q4 + 1), (keys 8-15, ...)
                        uint32_t w[4];
                        ldsm_x4_trans(addr, w[0], w[1], w[2], w[3]);
                        // a transposed 16-bit element is the byte pair (2g, 2g + 1) of one key; the register
                        // holds it for keys 2 t4 and 2 t4 + 1.  Regrouped by byte: the even column of both
                        // keys, then the odd column of both keys, each converted to an fp16 pair.
                        uint32_t ev[4], od[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            uint32_t t;
                            asm("prmt.b32 %0, %1, %1, 0x3120;" : "=r"(t) : "r"(w[j]));
                            e4m3x4_to_f16x2x2(t, ev[j], od[j]);
                        }
                        // accumulator block 2c + parity holds output columns 16c + 2n + parity, n = the MMA's column
                        mma_16816(o[4 * q4], pa, ev[0], ev[1]);
                        mma_16816(o[4 * q4 + 1], pa, od[0], od[1]);
                        mma_16816(o[4 * q4 + 2], pa, ev[2], ev[3]);
                        mma_16816(o[4 * q4 + 3], pa, od[2], od[3]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bars[2 * kDec8Stages + st]));
        }

        // ---- merge the four warps' states and write this chunk's partial result
        // (all tiles this CTA requested have been consumed by every warp before the barrier below,
        // so the ring can be reused as the merge buffer)
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
        float* mo = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));  // [4 warps][16 rows][128]
        float* ml = mo + kDec8Warps * 16 * 128;                                                       // [4][16][2]: m, l
        asm volatile("bar.sync 1, %0;" ::"n"(kDec8Warps * 32) : "memory");
        if (ok) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                // block i = 2c + parity: MMA columns 2 t4 and 2 t4 + 1 are output columns 16c + 4 t4 + parity and + 2
                const int col = (i >> 1) * 16 + 4 * t4 + (i & 1);
                mo[(warp * 16 + g) * 128 + col] = o[i][0];
                mo[(warp * 16 + g) * 128 + col + 2] = o[i][1];
                mo[(warp * 16 + g + 8) * 128 + col] = o[i][2];
                mo[(warp * 16 + g + 8) * 128 + col + 2] = o[i][3];
            }
            if (t4 == 0) {
                ml[(warp * 16 + g) * 2] = m_lo;
                ml[(warp * 16 + g) * 2 + 1] = l_lo;
                ml[(warp * 16 + g + 8) * 2] = m_hi;
                ml[(warp * 16 + g + 8) * 2 + 1] = l_hi;
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kDec8Warps * 32) : "memory");
        if (ok) {
            const int col = tid & 127;   // a thread owns one output column of every second (or fourth ...) row
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
                const long long slot = ((long long)b * p.Hq + h0 + r) * p.n_chunks + c;
                p.o_part[slot * 128 + col] = acc / l * p.v_scale;
                if (col == 0) p.lse_part[slot] = (M * p.scale_log2 + log2f(l)) * 0.6931471805599453f;
            }
        }
    }
}

}  // namespace fa
