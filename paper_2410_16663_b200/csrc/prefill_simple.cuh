// Prefill forward, straightforward variant: one CTA of 128 threads per (batch, head, 128-row
// query tile), one thread per query row.  Thread 0 additionally issues the TMA loads and the
// tcgen05 MMAs.  K/V tiles go through a two-slot shared-memory ring; S = Q K^T and O += P V
// both accumulate in tensor memory; P is handed to the second MMA either through tensor
// memory (packed 16-bit, over the columns S occupied) or through a swizzled shared-memory
// tile.  Every step of the four-stage block loop (Q*K^T, Exp, Exp*V, rowmax/rowsum update)
// runs strictly one after the other, so this kernel is the reference point the pipelined
// kernel is measured against, and the one kept for A/B checks.
#pragma once

#include <type_traits>

#include "sm100_ptx.cuh"

namespace fa {

// Division of a non-negative 32-bit integer by a divisor fixed at launch time, as a multiply and
// a shift: the persistent kernels turn a work item's index into (batch, head, tile) with it.
// With s = ceil(log2 d) and M = floor(2^(31+s) / d) + 1, floor(n * M / 2^(31+s)) = floor(n / d)
// for every 0 <= n < 2^31 (the excess of M over 2^(31+s)/d adds less than 1/d to the quotient).
struct FastDiv {
    uint32_t mul, shift, d;
    __host__ void set(int divisor) {
        d = static_cast<uint32_t>(divisor);
        uint32_t s = 0;
        while ((1ull << s) < d) ++s;
        shift = 31 + s;
        mul = static_cast<uint32_t>((1ull << shift) / d + 1);
    }
    __host__ __device__ __forceinline__ int div(int n) const {
        return static_cast<int>((static_cast<unsigned long long>(static_cast<uint32_t>(n)) * mul) >> shift);
    }
    __host__ __device__ __forceinline__ void divmod(int n, int& q, int& r) const {
        q = div(n);
        r = n - q * static_cast<int>(d);
    }
};

struct FwdParams {
    void* o;
    float* lse;
    int B, Hq, Hkv, Sq, Skv;
    int causal;
    float scale_log2;  // scale * log2(e)
    long long o_sb, o_ss, o_sh;  // element strides of o
    int o_fp32;
    int n_qtiles;
    int o_align32;  // o and its strides are 32-byte aligned: rows can be written with 256-bit stores
    FastDiv by_bh, by_hq, by_group, by_qtiles, by_qpairs;  // B*Hq, Hq, Hq/Hkv, n_qtiles, ceil(n_qtiles/2)
    // item order of the ping-pong kernel (see pp_decode_item): query tiles come in classes of
    // 2^cls_log2 consecutive tiles; by_class divides by the items of a full class, by_lastcls by
    // the size of the last (possibly smaller) class
    int cls_log2;
    FastDiv by_class, by_lastcls;
    // head-by-head order of the ping-pong kernel for very long sequences (see PpItems::next):
    // every head takes rounds_per_head whole rounds of the grid; 0 = the class order above
    int rounds_per_head;
    FastDiv by_rph;
    // packed variable-length batch (ping-pong kernel only; nullptr otherwise): sequence b owns
    // rows [cu_q[b], cu_q[b+1]) of q and o and rows [cu_k[b], cu_k[b+1]) of k and v; Sq and Skv
    // above are then the longest sequence's, and lse is [Hq, total_q]
    const int* cu_q;
    const int* cu_k;
    int total_q;
    // packed batch over a paged K/V cache (block_table != nullptr; cu_k unused): sequence b has
    // seqlens_k[b] keys, key j in row j % page_size of page block_table[b * table_stride + j / page_size];
    // page_size is a multiple of the 128-key tile and the K/V tensor maps run over the pages
    const int* block_table;
    const int* seqlens_k;
    int table_stride, page_size;
    FastDiv by_tiles_per_page;  // page_size / 128: kv tile j lies in table entry j / that, at tile j % that of the page
    int d;  // head dimension: 128, or 64 (its own kernel)
    float out_scale;  // factor on O (FP8 operands: the factor of V; 1 otherwise)
};

constexpr int kTile = 128;          // query rows per tile == kv rows per tile == head dim
constexpr int kHalfBytes = 16384;   // one 128-row x 64-element 16-bit box
constexpr int kTileBytes = 32768;   // a 128 x 128 16-bit tile = two boxes

// Loads one 128x128 16-bit tile (rows s0.., all of d) as two 64-column swizzled boxes.
__device__ __forceinline__ void load_tile(uint32_t dst, const CUtensorMap* tm, uint32_t bar,
                                          int h, int s0, int b) {
    tma_load_4d(dst, tm, bar, 0, h, s0, b);
    tma_load_4d(dst + kHalfBytes, tm, bar, 64, h, s0, b);
}

#ifndef FA_L2_HINTS
#define FA_L2_HINTS 1
#endif
// The persistent kernels' loads carry an L2 eviction policy: Q is read once (evict first), K and V
// of a head are read again by every later query tile of that head (evict last).
__device__ __forceinline__ void load_tile_hint(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int h, int s0, int b,
                                               uint64_t policy) {
#if FA_L2_HINTS
    tma_load_4d_hint(dst, tm, bar, 0, h, s0, b, policy);
    tma_load_4d_hint(dst + kHalfBytes, tm, bar, 64, h, s0, b, policy);
#else
    load_tile(dst, tm, bar, h, s0, b);
#endif
}

// Host side, once per kernel and device: the opt-in to more than 48 KB of dynamic shared memory
// is a per-device attribute of each kernel function, so a process that launches on several GPUs
// needs it on each, for each kernel.  Returns 0 and the device's SM count, or the CUDA error
// code.  The table of what has been done is keyed by kernel address and device; concurrent first
// calls at worst repeat the same idempotent set-up.
inline int prepare_big_smem_kernel(const void* kern, int smem_bytes, int* sm_count) {
    constexpr int kMaxDev = 64, kMaxKernels = 16;
    struct Entry {
        const void* kern;
        int sms[kMaxDev];
    };
    static Entry table[kMaxKernels] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    Entry* ent = nullptr;
    for (int i = 0; i < kMaxKernels && !ent; ++i) {
        const void* k = __atomic_load_n(&table[i].kern, __ATOMIC_ACQUIRE);
        if (k == kern) ent = &table[i];
        else if (k == nullptr) {
            const void* expected = nullptr;
            if (__atomic_compare_exchange_n(&table[i].kern, &expected, kern, false, __ATOMIC_ACQ_REL, __ATOMIC_ACQUIRE) ||
                expected == kern)
                ent = &table[i];
        }
    }
    const bool cached = ent && dev >= 0 && dev < kMaxDev;
    if (cached) {
        const int n = __atomic_load_n(&ent->sms[dev], __ATOMIC_ACQUIRE);
        if (n > 0) {
            *sm_count = n;
            return 0;
        }
    }
    int n = 0;
    if ((e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return (int)e;
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes)) != cudaSuccess)
        return (int)e;
    if (cached) __atomic_store_n(&ent->sms[dev], n, __ATOMIC_RELEASE);
    *sm_count = n;
    return 0;
}

// Stores 32 consecutive rows of a 16-bit output tile, one row of 128 elements (64 packed words
// w) per lane, so that every store instruction writes whole 128-byte lines.  A lane's own row is
// eight 32-byte sectors; written directly, one instruction would touch 32 different lines with one
// sector each.  Two butterfly exchanges inside each group of four lanes (with the lanes at
// distance 1, then 2) leave lane a of the group with sectors a and 4 + a of all four rows of the
// group, and the four lanes then write the four sectors of one line together.
// row_ptr: this lane's own row (32-byte aligned); row_stride: elements between consecutive rows
// (the rows of lanes l and l + 1); rows_live: how many of the warp's 32 rows exist (lane < rows_live).
template <typename T>
__device__ __forceinline__ void store_rows_coalesced(T* row_ptr, long long row_stride, int rows_live,
                                                     uint32_t (&w)[64]) {
    const int lane = threadIdx.x & 31;
    const bool b0 = lane & 1, b1 = lane & 2;
#if FA_L2_HINTS
    const uint64_t out_policy = l2_policy_evict_first();  // the output is not read again
#endif
    // exchange with the lane at distance 1: keep the sectors whose index has bit 0 == b0
    uint32_t a[4][2][8];  // [q][row slot: own pair member / the other][word]; sector index 2q + b0
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t lo = w[(2 * q) * 8 + i], hi = w[(2 * q + 1) * 8 + i];
            const uint32_t send = b0 ? lo : hi;
            a[q][0][i] = b0 ? hi : lo;
            a[q][1][i] = __shfl_xor_sync(0xffffffffu, send, 1);
        }
    // exchange with the lane at distance 2: keep the sectors whose index has bit 1 == b1
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            uint32_t keep[8], got[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t lo = a[2 * h][r][i], hi = a[2 * h + 1][r][i];
                const uint32_t send = b1 ? lo : hi;
                keep[i] = b1 ? hi : lo;
                got[i] = __shfl_xor_sync(0xffffffffu, send, 2);
            }
            // this lane now holds sector 4h + (lane & 3) of the rows of lanes lane^r and lane^r^2
            const int sector = 4 * h + (lane & 3);
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int src_lane = lane ^ r ^ (2 * t);
                if (src_lane < rows_live) {
                    T* dst = row_ptr + (long long)(src_lane - lane) * row_stride + sector * 16;
                    const uint32_t(&v)[8] = t ? got : keep;
#if FA_L2_HINTS
                    st_global_v8_hint(dst, v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7], out_policy);
#else
                    st_global_v8(dst, v[0], v[1], v[2], v[3], v[4], v[5], v[6], v[7]);
#endif
                }
            }
        }
}

// Number of kv tiles a query tile starting at row q0 has to visit.
__device__ __forceinline__ int kv_tiles_for(int q0, int q_rows, int Sq, int Skv, int causal) {
    int n = (Skv + kTile - 1) / kTile;
    if (causal) {
        int last_row = min(q0 + q_rows, Sq) - 1;
        int last_key = last_row + (Skv - Sq);  // >= 0 because Sq <= Skv
        n = min(n, last_key / kTile + 1);
    }
    return n;
}

template <typename T, bool kPInTmem>
__global__ void __launch_bounds__(128, 1)
fa_fwd_simple_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment for the 128-byte swizzle
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = smem_base;
    const uint32_t sK = sQ + kTileBytes;           // 2 slots
    const uint32_t sV = sK + 2 * kTileBytes;       // 2 slots
    const uint32_t sP = sV + 2 * kTileBytes;       // 1 tile (only when !kPInTmem)
    __shared__ __align__(8) uint64_t bars[8];
    __shared__ uint32_t tmem_holder;
    __shared__ volatile uint32_t abort_flag;

    const uint32_t bar_q = smem_u32(&bars[0]);
    const uint32_t bar_k0 = smem_u32(&bars[1]);  // +8 for slot 1
    const uint32_t bar_v0 = smem_u32(&bars[3]);
    const uint32_t bar_s = smem_u32(&bars[5]);
    const uint32_t bar_o = smem_u32(&bars[6]);

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
        for (int i = 0; i < 7; ++i) mbar_init(smem_u32(&bars[i]), 1);
        abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
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
    const uint32_t lane_sel = static_cast<uint32_t>(warp * 32) << 16;
    const uint32_t tS = tmem_base + lane_sel;        // columns [0,128): S, then P packed in [0,64)
    const uint32_t tO = tmem_base + lane_sel + 128;  // columns [128,256): O

    constexpr uint32_t idesc_qk = instr_desc_f16(std::is_same<T, __nv_bfloat16>::value, 128, 128, false, false);
    constexpr uint32_t idesc_pv = instr_desc_f16(std::is_same<T, __nv_bfloat16>::value, 128, 128, false, true);

    if (tid == 0) {
        mbar_expect_tx(bar_q, kTileBytes);
        load_tile(sQ, &tm_q, bar_q, h, q0, b);
        for (int j = 0; j < 2 && j < n_tiles; ++j) {
            mbar_expect_tx(bar_k0 + 8 * j, kTileBytes);
            load_tile(sK + j * kTileBytes, &tm_k, bar_k0 + 8 * j, hk, j * kTile, b);
            mbar_expect_tx(bar_v0 + 8 * j, kTileBytes);
            load_tile(sV + j * kTileBytes, &tm_v, bar_v0 + 8 * j, hk, j * kTile, b);
        }
    }
    __syncwarp();

    const int row = q0 + tid;          // this thread's query row
    float m_run = -INFINITY;           // running row max, in raw score units
    float l_run = 0.f;                 // running row sum
    bool ok = true;

    for (int j = 0; j < n_tiles && ok; ++j) {
        const int slot = j & 1;
        const uint32_t ring_parity = (j >> 1) & 1;
        // ---- S = Q K_j^T
        if (tid == 0) {
            if (j == 0) ok = mbar_wait(bar_q, 0, &abort_flag, 1);
            ok = ok && mbar_wait(bar_k0 + 8 * slot, ring_parity, &abort_flag, 2);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t koff = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                    mma_ss(tmem_base, smem_desc_sw128(sQ + koff, 16, 1024),
                           smem_desc_sw128(sK + slot * kTileBytes + koff, 16, 1024), idesc_qk,
                           ks > 0);
                }
                mma_commit(bar_s);
            }
        }
        __syncwarp();
        if (!mbar_wait(bar_s, j & 1, &abort_flag, 3)) { ok = false; break; }
        tc_fence_after();

        // ---- load this row of S
        float s[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld_x32(tS + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) s[c * 32 + i] = __uint_as_float(r[i]);
        }
        // ---- mask: only tiles the diagonal or the end of the keys cross
        const int kv0 = j * kTile;
        const bool need_mask = (p.causal && kv0 + kTile - 1 > q0 + off) || (kv0 + kTile > p.Skv);
        if (need_mask) {
            int lim = p.Skv - kv0;                                // columns >= lim are past the keys
            if (p.causal) lim = min(lim, row + off - kv0 + 1);    // columns >= lim are above the diagonal
#pragma unroll
            for (int i = 0; i < 128; ++i)
                if (i >= lim) s[i] = -INFINITY;
        }
        // ---- online softmax update (Appendix A: rowmax / rowsum)
        float m_tile = s[0];
#pragma unroll
        for (int i = 1; i < 128; ++i) m_tile = fmaxf(m_tile, s[i]);
        const float m_new = fmaxf(m_run, m_tile);
        // rows past Sq in a ragged last tile may see nothing; keep them finite
        const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = (m_run == -INFINITY) ? 0.f : fast_exp2((m_run - m_use) * p.scale_log2);
        const float neg_ms = -m_use * p.scale_log2;
        float l_tile = 0.f;
        if (need_mask) {
            // masked entries become exact zeros whatever the scale (0 * -inf would be NaN)
            int lim = p.Skv - kv0;
            if (p.causal) lim = min(lim, row + off - kv0 + 1);
#pragma unroll
            for (int i = 0; i < 128; ++i) {
                s[i] = (i < lim) ? fast_exp2(fmaf(s[i], p.scale_log2, neg_ms)) : 0.f;
                l_tile += s[i];
            }
        } else {
#pragma unroll
            for (int i = 0; i < 128; ++i) {
                s[i] = fast_exp2(fmaf(s[i], p.scale_log2, neg_ms));
                l_tile += s[i];
            }
        }
        l_run = l_run * alpha + l_tile;
        m_run = m_new;

        // ---- O <- alpha * O once the previous P V has landed; refill the slot it freed
        if (j > 0) {
            if (!mbar_wait(bar_o, (j - 1) & 1, &abort_flag, 4)) { ok = false; break; }
            tc_fence_after();
            if (tid == 0 && j + 1 < n_tiles) {
                const int ns = (j + 1) & 1;
                mbar_expect_tx(bar_k0 + 8 * ns, kTileBytes);
                load_tile(sK + ns * kTileBytes, &tm_k, bar_k0 + 8 * ns, hk, (j + 1) * kTile, b);
                mbar_expect_tx(bar_v0 + 8 * ns, kTileBytes);
                load_tile(sV + ns * kTileBytes, &tm_v, bar_v0 + 8 * ns, hk, (j + 1) * kTile, b);
            }
            __syncwarp();
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
        // ---- hand P to the second MMA
        if constexpr (kPInTmem) {
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t r[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = pack2<T>(s[c * 64 + 2 * i], s[c * 64 + 2 * i + 1]);
                tmem_st_x32(tS + c * 32, r);
            }
        } else {
            // row `tid` of the swizzled tile: 16-byte chunk c of a 128-byte row sits at c ^ (row & 7)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const uint32_t row_base = sP + half * kHalfBytes + tid * 128;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const int e = half * 64 + c * 8;
                    uint32_t w0 = pack2<T>(s[e], s[e + 1]), w1 = pack2<T>(s[e + 2], s[e + 3]);
                    uint32_t w2 = pack2<T>(s[e + 4], s[e + 5]), w3 = pack2<T>(s[e + 6], s[e + 7]);
                    const uint32_t addr = row_base + ((c ^ (tid & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(w0),
                                 "r"(w1), "r"(w2), "r"(w3)
                                 : "memory");
                }
            }
            fence_proxy_async_smem();
        }
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();
        // ---- O += P V_j
        if (tid == 0) {
            ok = mbar_wait(bar_v0 + 8 * slot, ring_parity, &abort_flag, 5);
            if (ok) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    // 16 kv rows per step: 2048 bytes down the swizzled V tile (MN-major B)
                    const uint64_t bdesc =
                        smem_desc_sw128(sV + slot * kTileBytes + ks * 2048, kHalfBytes, 1024);
                    if constexpr (kPInTmem) {
                        mma_ts(tmem_base + 128, tmem_base + ks * 8, bdesc, idesc_pv, (j > 0) || (ks > 0));
                    } else {
                        const uint32_t koff = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                        mma_ss(tmem_base + 128, smem_desc_sw128(sP + koff, 16, 1024), bdesc, idesc_pv,
                               (j > 0) || (ks > 0));
                    }
                }
                mma_commit(bar_o);
            }
        }
        __syncwarp();
    }

    // ---- epilogue: O / l, LSE = m*scale + ln l
    if (ok && n_tiles > 0) ok = mbar_wait(bar_o, (n_tiles - 1) & 1, &abort_flag, 6);
    if (ok && n_tiles > 0) {
        tc_fence_after();
        const float inv_l = (l_run > 0.f) ? 1.f / l_run : 0.f;
        const bool live = row < p.Sq;
        const long long obase = (long long)b * p.o_sb + (long long)row * p.o_ss + (long long)h * p.o_sh;
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
            const float lse = (l_run > 0.f) ? (m_run * p.scale_log2 + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
            p.lse[((long long)b * p.Hq + h) * p.Sq + row] = lse;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, 256);
    }
}

// O = 0, LSE = -inf for a problem without keys.
template <typename T>
__global__ void fa_fill_empty_kernel(const FwdParams p) {
    const long long n = (long long)p.B * p.Sq * p.Hq;
    for (long long r = blockIdx.x * (long long)blockDim.x + threadIdx.x; r < n;
         r += (long long)gridDim.x * blockDim.x) {
        const int h = r % p.Hq;
        const long long bi = r / p.Hq;
        const int i = bi % p.Sq;
        const int b = bi / p.Sq;
        const long long obase = (long long)b * p.o_sb + (long long)i * p.o_ss + (long long)h * p.o_sh;
        for (int t = 0; t < p.d; ++t) {
            if (p.o_fp32) static_cast<float*>(p.o)[obase + t] = 0.f;
            else static_cast<T*>(p.o)[obase + t] = T(0.f);
        }
        if (p.lse) p.lse[((long long)b * p.Hq + h) * p.Sq + i] = -INFINITY;
    }
}

}  // namespace fa
