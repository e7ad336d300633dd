// Output projection out = O * W_O on the tensor cores, as the second phase of the fused
// attention + Linear operator (Section 4.2 fuses the attention kernel with the Linear that
// follows it; on one GPU there is no collective to hide, so what the fusion buys here is that the
// projection starts on query blocks whose heads are all done while other blocks are still being
// attended to, in one launch, with O still in L2).
//
// O is the attention output [B, Sq, Hq*128] (16-bit, K = Hq*128 contiguous), W_O is [Hq*128, N]
// row-major (N contiguous), out is [B, Sq, N].  A work item is one 128-row block of one batch
// entry times 256 columns.  The phase runs on the ping-pong kernel's 384-thread layout and in its
// shared and tensor memory:
//   warp 9  (one thread): TMA loads into a ring of four stages; a stage is a 128 x 64 block of O
//                         (K-major, one swizzled box) and a 64 x 256 block of W_O (N-major, four
//                         boxes of 64 columns) -- 48 KiB;
//   warp 8  (one thread): per stage four tcgen05.mma 128 x 256 x 16 into one of two 256-column
//                         accumulators in tensor memory;
//   warps 0-7           : warpgroup a drains accumulator a: one thread per row, 32 columns at a
//                         time, rounded to 16 bits and stored.
// In the fused launch a row block may be loaded only after every head's attention output for it
// has reached global memory: the attention epilogue counts its completed TMA stores per row block
// in `done`, and the loading thread waits (bounded) for the count before the block's first load.
#pragma once

#include "prefill_pingpong.cuh"

namespace fa {

struct ProjParams {
    void* out;                 // [B, Sq, N], the operands' 16-bit type
    int B, Sq, Hq, N;          // K = Hq * 128
    int n_qtiles, n_cblocks;   // row blocks per batch entry, column blocks of 256
    unsigned int* done;        // [B * n_qtiles] completed-store counts, or nullptr (O is final already)
    unsigned int done_target;  // 4 * Hq: one count per epilogue warp and head
};

constexpr int kProjStages = 4;
constexpr int kProjABytes = 128 * 64 * 2;          // 16 KiB
constexpr int kProjWBoxBytes = 64 * 64 * 2;        // 8 KiB: 64 k-rows x 64 columns
constexpr int kProjStageBytes = kProjABytes + 4 * kProjWBoxBytes;   // 48 KiB
static_assert(kProjStages * kProjStageBytes <= (kPpQBufs + kPpNK + kPpNV) * kTileBytes, "the ring fits the kernel's tiles");

namespace prb {   // barrier indices of the projection phase
constexpr int full = 0;                       // [stages] TMA -> MMA thread
constexpr int empty = full + kProjStages;     // [stages] MMA thread (commit) -> loader
constexpr int acc_full = empty + kProjStages; // [2] MMA thread (commit) -> warpgroup a
constexpr int acc_empty = acc_full + 2;       // [2] warpgroup a (128 arrivals) -> MMA thread
constexpr int count = acc_empty + 2;
}  // namespace prb

// Work item t of the CTA's list -> (batch, query tile, column block).  Row blocks go in the order
// the attention phase finishes them (longest query tiles first), all column blocks of a row block
// next to each other so that the CTAs working at one time share a few row blocks of O.
__device__ __forceinline__ void proj_item(const ProjParams& pp, int t, int& b, int& qt, int& cb) {
    const int rb = t / pp.n_cblocks;
    cb = t - rb * pp.n_cblocks;
    const int qi = rb / pp.B;
    b = rb - qi * pp.B;
    qt = pp.n_qtiles - 1 - qi;
}

// bar0: shared address of prb::count barriers (initialised by the caller: full/empty/acc_full
// count 1, acc_empty count 128); smem: 1024-aligned base of the stage ring; tmem: 512 columns.
template <typename T>
__device__ __forceinline__ void proj_phase(const CUtensorMap* tm_a, const CUtensorMap* tm_w, const ProjParams& pp,
                                           uint32_t bar0, uint32_t smem, uint32_t tmem, volatile uint32_t* abort_flag) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int total = pp.B * pp.n_qtiles * pp.n_cblocks;
    const int n_kb = pp.Hq * 2;   // k-blocks of 64
    if (warp == 9) {
        if (lane == 0) {
            // ------------------------------------------------------------ loads
            tma_prefetch_desc(tm_a);
            tma_prefetch_desc(tm_w);
            const uint64_t pol = l2_policy_evict_last();   // both operands are read again by other CTAs
            PpRing<kProjStages> ring;
            int last_rb = -1;
            for (int t = blockIdx.x; t < total; t += gridDim.x) {
                int b, qt, cb;
                proj_item(pp, t, b, qt, cb);
                const int rb = b * pp.n_qtiles + qt;
                if (pp.done != nullptr && rb != last_rb) {
                    // every head's O for this row block has landed (bounded wait, like every other)
                    const unsigned long long t0 = globaltimer_ns();
                    while (ld_acquire_gpu(pp.done + rb) < pp.done_target) {
                        if (*abort_flag) return;
                        if (globaltimer_ns() - t0 > kWaitLimitNs) {
                            *abort_flag = 1u;
                            record_timeout(170);
                            return;
                        }
                        __nanosleep(200);
                    }
                    // the TMA loads below read what other SMs' TMA stores wrote
                    asm volatile("fence.proxy.async;" ::: "memory");
                    last_rb = rb;
                }
                for (int kb = 0; kb < n_kb; ++kb, ring.next()) {
                    if (!mbar_wait(pp_bar(bar0, prb::empty + ring.slot), ring.par ^ 1, abort_flag, 171)) return;
                    const uint32_t fb = pp_bar(bar0, prb::full + ring.slot);
                    const uint32_t dst = smem + ring.slot * kProjStageBytes;
                    mbar_expect_tx(fb, kProjStageBytes);
                    // O block: 64 elements of K (head kb / 2, half kb & 1) x 128 rows
                    tma_load_4d_hint(dst, tm_a, fb, (kb & 1) * 64, kb >> 1, qt * kTile, b, pol);
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        tma_load_4d_hint(dst + kProjABytes + i * kProjWBoxBytes, tm_w, fb, cb * 256 + i * 64, kb * 64, 0, 0, pol);
                }
            }
        }
        __syncwarp();
    } else if (warp == 8) {
        if (lane == 0) {
            // ------------------------------------------------------------ MMA issue
            constexpr bool kBf16 = std::is_same<T, __nv_bfloat16>::value;
            constexpr uint32_t idesc = instr_desc_f16(kBf16, 128, 256, false, true);
            PpRing<kProjStages> ring;
            uint32_t n = 0;   // items of this CTA so far
            for (int t = blockIdx.x; t < total; t += gridDim.x, ++n) {
                const uint32_t acc = n & 1;
                // the warpgroup has read the accumulator's previous item out (passes at once the first time)
                if (!mbar_wait(pp_bar(bar0, prb::acc_empty + acc), ((n >> 1) & 1) ^ 1, abort_flag, 172)) return;
                tc_fence_after();
                for (int kb = 0; kb < n_kb; ++kb, ring.next()) {
                    if (!mbar_wait(pp_bar(bar0, prb::full + ring.slot), ring.par, abort_flag, 173)) return;
                    tc_fence_after();
                    const uint32_t sa = smem + ring.slot * kProjStageBytes;
                    const uint32_t a_lo = desc_lo(sa, 16);
                    // W_O is the N-major operand: 64-column blocks 8 KiB apart, 16 k-rows (2048 bytes) per MMA
                    const uint32_t b_lo = desc_lo(sa + kProjABytes, kProjWBoxBytes);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        mma_ss_lo(tmem + 256 * acc, a_lo + ((ks * 32) >> 4), b_lo + ks * (2048 >> 4), idesc,
                                  (kb > 0 || ks > 0) ? 1u : 0u);
                    mma_commit(pp_bar(bar0, prb::empty + ring.slot));
                }
                mma_commit(pp_bar(bar0, prb::acc_full + acc));
            }
        }
        __syncwarp();
    } else if (warp < 8) {
        // ---------------------------------------------------------------- epilogue
        const int a = warp >> 2;                     // this warpgroup drains accumulator a
        const int r = tid & 127;
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        uint32_t n = 0, mine = 0;
        for (int t = blockIdx.x; t < total; t += gridDim.x, ++n) {
            if ((int)(n & 1) != a) continue;
            int b, qt, cb;
            proj_item(pp, t, b, qt, cb);
            if (!pp_warp_wait(pp_bar(bar0, prb::acc_full + a), mine & 1, abort_flag, 174 + a)) return;
            ++mine;
            tc_fence_after();
            const int row = qt * kTile + r;
            T* row_ptr = static_cast<T*>(pp.out) + ((long long)b * pp.Sq + row) * pp.N + (long long)cb * 256;
            // 32 columns at a time: few registers, and a thread's eight stores of a chunk fill
            // whole 64-byte pieces of its row (the lines are completed in L2 before they go to HBM)
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t acc[32];
                tmem_ld_x32(tmem + lane_sel + 256 * a + 32 * c, acc);
                tmem_wait_ld();
                if (c == 7) {
                    // the whole accumulator has been read: the next item may overwrite it
                    tc_fence_before();
                    mbar_arrive(pp_bar(bar0, prb::acc_empty + a));
                }
                if (row < pp.Sq) {
                    uint4* dst = reinterpret_cast<uint4*>(row_ptr + 32 * c);
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        dst[i] = make_uint4(pack2<T>(__uint_as_float(acc[8 * i]), __uint_as_float(acc[8 * i + 1])),
                                            pack2<T>(__uint_as_float(acc[8 * i + 2]), __uint_as_float(acc[8 * i + 3])),
                                            pack2<T>(__uint_as_float(acc[8 * i + 4]), __uint_as_float(acc[8 * i + 5])),
                                            pack2<T>(__uint_as_float(acc[8 * i + 6]), __uint_as_float(acc[8 * i + 7])));
                }
            }
        }
    }
}

// The projection alone: O is final in global memory (the second launch of the two-launch form).
template <typename T>
__global__ void __launch_bounds__(kPipeThreads, 1)
fa_proj_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w, const ProjParams pp) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[prb::count];
    __shared__ uint32_t tmem_holder;
    __shared__ uint32_t abort_word;
    const uint32_t smem_base = smem_u32(smem_raw);
    const uint32_t bar0 = smem_u32(&bars[0]);
    const int tid = threadIdx.x, warp = tid >> 5;
    if (smem_base & 1023u) {
        if (tid == 0) record_timeout(901);
        return;
    }
    if (tid == 0) {
        for (int i = 0; i < prb::count; ++i) mbar_init(pp_bar(bar0, i), i >= prb::acc_empty ? 128 : 1);
        abort_word = 0;
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
    proj_phase<T>(&tm_a, &tm_w, pp, bar0, smem_base, tmem_base, &abort_word);
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

// Attention and projection in one launch: the ping-pong kernel, then the projection phase in the
// same shared and tensor memory.  A CTA starts projecting when its own attention items are done;
// row blocks whose heads other CTAs are still working on are waited for through `done`.  The
// grid must be resident as a whole (the host uses a cooperative launch): a CTA that waits for a
// row block relies on the CTAs that own its heads making progress.
template <typename T, bool kSingle>
__global__ void __launch_bounds__(kPipeThreads, 1)
fa_fwd_pingpong_proj_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                            const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                            const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
                            const FwdParams p, const int total_items, const ProjParams pp) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(1024) PpStatic ss;
    const uint32_t smem_base = smem_u32(smem_raw);
    if (!pp_attention<T, true, kSingle, false, false, true>(tm_q, tm_k, tm_v, tm_o, p, total_items, ss, smem_base, pp.done))
        return;
    // every role has left its loops and every store of this CTA has landed; the tiles are about
    // to be overwritten by TMA loads, the exchange arrays become the phase's barriers
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    static_assert(prb::count * 8 <= sizeof(ss.m_xch), "the phase's barriers fit the exchange array");
    const uint32_t bar0 = smem_u32(&ss.m_xch[0][0]);
    if (threadIdx.x == 0) {
        for (int i = 0; i < prb::count; ++i) mbar_init(pp_bar(bar0, i), i >= prb::acc_empty ? 128 : 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (ss.abort_flag == 0) proj_phase<T>(&tm_a, &tm_w, pp, bar0, smem_base, ss.tmem_holder, &ss.abort_flag);
    tc_fence_before();
    __syncthreads();
    if ((threadIdx.x >> 5) == 8) {
        __syncwarp();
        tmem_dealloc(ss.tmem_holder, 512);
    }
}

// fused != 0: one cooperative launch (pp.done must point at zeroed counters); otherwise the
// projection alone, on an O that is final.  Returns 0, -3 (unsupported) or -7 with the CUDA error.
template <typename T>
int launch_proj(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                const CUtensorMap& ta, const CUtensorMap& tw, const FwdParams& fp, const ProjParams& pp, int fused,
                cudaStream_t st, int* cuda_err) {
    constexpr int smem = (kPpQBufs + kPpNK + kPpNV) * kTileBytes;
    int sm_count = 0;
    cudaError_t e;
    if (!fused) {
        auto kern = fa_proj_kernel<T>;
        if (int ce = prepare_big_smem_kernel(reinterpret_cast<const void*>(kern), kProjStages * kProjStageBytes, &sm_count)) { *cuda_err = ce; return -7; }
        const long long total = (long long)pp.B * pp.n_qtiles * pp.n_cblocks;
        const int grid = (int)(total < sm_count ? total : sm_count);
        kern<<<grid, kPipeThreads, kProjStages * kProjStageBytes, st>>>(ta, tw, pp);
        e = cudaGetLastError();
        if (e != cudaSuccess) { *cuda_err = (int)e; return -7; }
        return 0;
    }
    const bool single = fp.Skv <= 32 * kTile;
    auto kern = single ? fa_fwd_pingpong_proj_kernel<T, true> : fa_fwd_pingpong_proj_kernel<T, false>;
    if (int ce = prepare_big_smem_kernel(reinterpret_cast<const void*>(kern), smem, &sm_count)) { *cuda_err = ce; return -7; }
    const long long total = (long long)fp.n_qtiles * fp.B * fp.Hq;
    if (total > 0x7fffffffll) return -3;
    const int grid = (int)(total < sm_count ? total : sm_count);
    FwdParams fpc = pp_plan_items(fp, grid, 512.0);
    int total_i = (int)total;
    ProjParams ppc = pp;
    void* args[] = {(void*)&tq, (void*)&tk, (void*)&tv, (void*)&to, (void*)&ta, (void*)&tw, (void*)&fpc, (void*)&total_i, (void*)&ppc};
    e = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(kern), dim3(grid), dim3(kPipeThreads), args, smem, st);
    if (e != cudaSuccess) { *cuda_err = (int)e; return -7; }
    return 0;
}

}  // namespace fa
