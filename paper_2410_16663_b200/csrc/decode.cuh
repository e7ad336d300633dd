// Decode-stage attention (one query row per sequence over the cached K and V), split along
// the cache: each CTA streams one chunk of one (sequence, kv head) through a TMA-fed
// shared-memory ring and keeps running (rowmax, rowsum, O) for the G query heads that share
// the kv head; a second kernel merges the per-chunk partial results.  The work is a single
// pass over the cache, so the kernel is written for HBM bandwidth: arithmetic is plain fp32
// FMA, every cache byte is read exactly once and nothing but the partials is written.
#pragma once

#include "sm100_ptx.cuh"

namespace fa {

constexpr int kDecTile = 128;                 // keys per shared-memory tile
constexpr int kDecStages = 3;                 // ring depth (K and V tiles each 32 KiB)
constexpr int kDecTileBytes = 32768;
constexpr int kDecHalfBytes = 16384;
constexpr int kDecThreads = 128;

struct DecodeParams {
    const void* q;        // [B,1,Hq,128] 16-bit
    const int* seqlens;   // [B] device
    float* o_part;        // [B,Hq,NC,128]
    float* lse_part;      // [B,Hq,NC]
    int B, Hq, Hkv, Smax;
    int chunk;            // keys per chunk (multiple of kDecTile)
    int n_chunks;         // ceil(Smax / chunk)
    int heads_per_item;   // G when query heads of a group are processed together, else 1
    float scale_log2;
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(addr));
    return v;
}

template <typename T>
__device__ __forceinline__ float2 unpack2(uint32_t w);
template <>
__device__ __forceinline__ float2 unpack2<__half>(uint32_t w) {
    return __half22float2(*reinterpret_cast<__half2*>(&w));
}
template <>
__device__ __forceinline__ float2 unpack2<__nv_bfloat16>(uint32_t w) {
    return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

// grid: (n_chunks, items_per_batch, B) where items_per_batch = Hkv (grouped) or Hq (G == 1 fallback)
template <typename T, int G>
__global__ void __launch_bounds__(kDecThreads, 1)
fa_decode_split_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                       const DecodeParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sK = smem_base;                                   // kDecStages tiles
    const uint32_t sV = smem_base + kDecStages * kDecTileBytes;      // kDecStages tiles
    __shared__ __align__(16) float q_s[G][128];
    __shared__ __align__(16) float p_s[G][kDecTile];
    __shared__ float red_s[G][4];
    __shared__ __align__(8) uint64_t bars[2 * kDecStages];
    __shared__ volatile uint32_t abort_flag;

    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int c = blockIdx.x;
    const int item = blockIdx.y;
    const int b = blockIdx.z;
    const int g_all = p.Hq / p.Hkv;
    const int h0 = (p.heads_per_item == 1) ? item : item * G;   // first query head of this item
    const int hk = h0 / g_all;

    int len = p.seqlens[b];
    len = max(0, min(len, p.Smax));
    const int k_begin = c * p.chunk;
    const int k_end = min(len, k_begin + p.chunk);
    if (k_begin >= k_end) return;  // uniform for the CTA: nothing allocated, nothing pending
    const int n_tiles = (k_end - k_begin + kDecTile - 1) / kDecTile;

    if (tid == 0) {
        for (int i = 0; i < 2 * kDecStages; ++i) mbar_init(smem_u32(&bars[i]), 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    // q -> fp32 in shared memory
    for (int i = tid; i < G * 64; i += kDecThreads) {
        const int g = i >> 6, t2 = i & 63;
        const uint32_t w = reinterpret_cast<const uint32_t*>(
            static_cast<const T*>(p.q) + ((long long)b * p.Hq + h0 + g) * 128)[t2];
        const float2 f = unpack2<T>(w);
        q_s[g][2 * t2] = f.x;
        q_s[g][2 * t2 + 1] = f.y;
    }
    __syncthreads();

    auto issue_tile = [&](int t) {
        const int st = t % kDecStages;
        const uint32_t bk = smem_u32(&bars[st]), bv = smem_u32(&bars[kDecStages + st]);
        const int row0 = k_begin + t * kDecTile;
        mbar_expect_tx(bk, kDecTileBytes);
        tma_load_4d(sK + st * kDecTileBytes, &tm_k, bk, 0, hk, row0, b);
        tma_load_4d(sK + st * kDecTileBytes + kDecHalfBytes, &tm_k, bk, 64, hk, row0, b);
        mbar_expect_tx(bv, kDecTileBytes);
        tma_load_4d(sV + st * kDecTileBytes, &tm_v, bv, 0, hk, row0, b);
        tma_load_4d(sV + st * kDecTileBytes + kDecHalfBytes, &tm_v, bv, 64, hk, row0, b);
    };
    int issued = 0;
    if (tid == 0) {
        for (; issued < kDecStages - 1 && issued < n_tiles; ++issued) issue_tile(issued);
    }

    float m_run[G], l_loc[G], o_acc[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m_run[g] = -INFINITY;
        l_loc[g] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) o_acc[g][i] = 0.f;
    }
    const int kg = tid >> 4, dc = tid & 15;  // P V phase: key group (key & 7 == kg) and 8-wide slice of d
    bool ok = true;

    for (int t = 0; t < n_tiles; ++t) {
        const int st = t % kDecStages;
        const uint32_t parity = (t / kDecStages) & 1;
        const int valid = min(kDecTile, k_end - (k_begin + t * kDecTile));  // keys of this tile in range
        if (!mbar_wait(smem_u32(&bars[st]), parity, &abort_flag, 20)) { ok = false; break; }
        // ---- scores: thread `tid` owns key `tid` of the tile
        float s[G];
        {
            float sa[G], sb[G];  // two partial sums per head keep the FMA chains short
#pragma unroll
            for (int g = 0; g < G; ++g) sa[g] = sb[g] = 0.f;
            const uint32_t krow = sK + st * kDecTileBytes + tid * 128;
#pragma unroll
            for (int c16 = 0; c16 < 16; ++c16) {
                const uint4 kw = lds128(krow + (c16 >> 3) * kDecHalfBytes + (((c16 & 7) ^ (tid & 7)) << 4));
                const float2 k0 = unpack2<T>(kw.x), k1 = unpack2<T>(kw.y), k2 = unpack2<T>(kw.z),
                             k3 = unpack2<T>(kw.w);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float4 qa = *reinterpret_cast<const float4*>(&q_s[g][c16 * 8]);
                    const float4 qb = *reinterpret_cast<const float4*>(&q_s[g][c16 * 8 + 4]);
                    sa[g] = fmaf(qa.x, k0.x, sa[g]);
                    sb[g] = fmaf(qb.x, k2.x, sb[g]);
                    sa[g] = fmaf(qa.y, k0.y, sa[g]);
                    sb[g] = fmaf(qb.y, k2.y, sb[g]);
                    sa[g] = fmaf(qa.z, k1.x, sa[g]);
                    sb[g] = fmaf(qb.z, k3.x, sb[g]);
                    sa[g] = fmaf(qa.w, k1.y, sa[g]);
                    sb[g] = fmaf(qb.w, k3.y, sb[g]);
                }
            }
#pragma unroll
            for (int g = 0; g < G; ++g) s[g] = sa[g] + sb[g];
        }
        const bool live = tid < valid;  // keys past the sequence hold arbitrary bits
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float wm = warp_max(live ? s[g] : -INFINITY);
            if (lane == 0) red_s[g][warp] = wm;
        }
        __syncthreads();  // (A) all warps are also past the P V of the previous tile
        if (tid == 0 && issued < n_tiles) {
            issue_tile(issued);  // refills the slot the previous tile used
            ++issued;
        }
        float alpha[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float tm = fmaxf(fmaxf(red_s[g][0], red_s[g][1]), fmaxf(red_s[g][2], red_s[g][3]));
            const float m_new = fmaxf(m_run[g], tm);  // finite: every tile holds at least one key in range
            alpha[g] = (m_run[g] == -INFINITY) ? 0.f : fast_exp2((m_run[g] - m_new) * p.scale_log2);
            const float pv = live ? fast_exp2((s[g] - m_new) * p.scale_log2) : 0.f;
            p_s[g][tid] = pv;
            l_loc[g] = l_loc[g] * alpha[g] + pv;
            m_run[g] = m_new;
#pragma unroll
            for (int i = 0; i < 8; ++i) o_acc[g][i] *= alpha[g];
        }
        __syncthreads();  // (B) probabilities visible
        if (!mbar_wait(smem_u32(&bars[kDecStages + st]), parity, &abort_flag, 21)) { ok = false; break; }
        // ---- O += P V: this thread adds keys kg, kg+8, ... for its 8 output dims
        {
            const uint32_t vbase = sV + st * kDecTileBytes + (dc >> 3) * kDecHalfBytes + (((dc & 7) ^ kg) << 4);
#pragma unroll 4
            for (int i = 0; i < 16; ++i) {
                const int key = kg + 8 * i;
                if (key < valid) {  // never touch rows past the sequence (0 * NaN)
                    const uint4 vw = lds128(vbase + key * 128);
                    const float2 v0 = unpack2<T>(vw.x), v1 = unpack2<T>(vw.y), v2 = unpack2<T>(vw.z),
                                 v3 = unpack2<T>(vw.w);
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float pg = p_s[g][key];
                        o_acc[g][0] = fmaf(pg, v0.x, o_acc[g][0]);
                        o_acc[g][1] = fmaf(pg, v0.y, o_acc[g][1]);
                        o_acc[g][2] = fmaf(pg, v1.x, o_acc[g][2]);
                        o_acc[g][3] = fmaf(pg, v1.y, o_acc[g][3]);
                        o_acc[g][4] = fmaf(pg, v2.x, o_acc[g][4]);
                        o_acc[g][5] = fmaf(pg, v2.y, o_acc[g][5]);
                        o_acc[g][6] = fmaf(pg, v3.x, o_acc[g][6]);
                        o_acc[g][7] = fmaf(pg, v3.y, o_acc[g][7]);
                    }
                }
            }
        }
    }

    // ---- reduce over threads and write this chunk's partial result
    __syncthreads();
    if (ok) {
        // every tile that was requested has been consumed, so the ring is free: reuse its
        // first bytes as the [8 key groups][G][128] reduction buffer
        float* o_red = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float ws = warp_sum(l_loc[g]);
            if (lane == 0) red_s[g][warp] = ws;
#pragma unroll
            for (int i = 0; i < 8; ++i) o_red[(kg * G + g) * 128 + dc * 8 + i] = o_acc[g][i];
        }
        __syncthreads();
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float l = red_s[g][0] + red_s[g][1] + red_s[g][2] + red_s[g][3];
            float acc = 0.f;
#pragma unroll
            for (int r = 0; r < 8; ++r) acc += o_red[(r * G + g) * 128 + tid];
            const long long slot = ((long long)b * p.Hq + h0 + g) * p.n_chunks + c;
            p.o_part[slot * 128 + tid] = acc / l;
            if (tid == 0)
                p.lse_part[slot] = (m_run[g] * p.scale_log2 + log2f(l)) * 0.6931471805599453f;
        }
    } else if (tid == 0) {
        // gave up on a wait: wait (bounded) for copies still in flight before the CTA's
        // shared memory is released
        for (int t = 0; t < issued; ++t) {
            const int st = t % kDecStages;
            const uint32_t parity = (t / kDecStages) & 1;
            const unsigned long long t0 = globaltimer_ns();
            while (!mbar_try_wait(smem_u32(&bars[st]), parity) && globaltimer_ns() - t0 < 100000000ull) {}
            while (!mbar_try_wait(smem_u32(&bars[kDecStages + st]), parity) &&
                   globaltimer_ns() - t0 < 200000000ull) {}
        }
    }
}

// Merge of the per-chunk partials (rowmax/rowsum recurrence applied across chunks):
//   M = max_c LSE_c, w_c = exp(LSE_c - M), O = sum_c w_c O_c / sum_c w_c, LSE = M + ln sum_c w_c.
// grid: B * Hq blocks of 128 threads, thread t owns output dim t.
template <typename T>
__global__ void __launch_bounds__(128)
fa_decode_combine_kernel(const DecodeParams p, T* o, float* lse) {
    const int bh = blockIdx.x;
    const int b = bh / p.Hq;
    const int tid = threadIdx.x;
    int len = p.seqlens[b];
    len = max(0, min(len, p.Smax));
    const int nc = (len + p.chunk - 1) / p.chunk;
    const float* lp = p.lse_part + (long long)bh * p.n_chunks;
    const float* op = p.o_part + (long long)bh * p.n_chunks * 128;
    if (nc == 0) {
        o[(long long)bh * 128 + tid] = T(0.f);
        if (lse && tid == 0) lse[bh] = -INFINITY;
        return;
    }
    float M = -INFINITY;
    for (int c = 0; c < nc; ++c) M = fmaxf(M, lp[c]);
    float wsum = 0.f, acc = 0.f;
    for (int c = 0; c < nc; ++c) {
        const float w = __expf(lp[c] - M);
        wsum += w;
        acc = fmaf(w, op[(long long)c * 128 + tid], acc);
    }
    o[(long long)bh * 128 + tid] = T(acc / wsum);
    if (lse && tid == 0) lse[bh] = M + logf(wsum);
}

}  // namespace fa
