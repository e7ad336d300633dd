// Host side of the C ABI declared in include/fa.h: argument validation, TMA tensor-map
// encoding, launch configuration.  No device memory is allocated here; every buffer is the
// caller's.  All kernels live in the headers included below (one translation unit).
#include "../../include/fa.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <mutex>

#include "decode.cuh"
#include "prefill_pingpong.cuh"
#include "proj_gemm.cuh"
#include "prefill_d64.cuh"
#include "prefill_d64_stream.cuh"
#include "prefill_d256.cuh"
#include "decode_fp8.cuh"
#include "prefill_pipelined.cuh"
#include "prefill_simple.cuh"

namespace {

thread_local int t_last_cuda_error = 0;

int cuda_fail(cudaError_t e) {
    t_last_cuda_error = static_cast<int>(e);
    return FA_ERR_CUDA;
}

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup, so that the library
// loads (and can report FA_ERR_DEVICE) on machines without a driver.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// Tensor map over a [B, S, H, d] 16-bit tensor (d = 128 or 64) with element strides (sb, ss, sh);
// a box is box_rows sequence positions x 64 elements of d for one (batch, head), 128-byte swizzled.
int encode_map(CUtensorMap* tm, const void* base, int B, int S, int H, int64_t sb, int64_t ss, int64_t sh,
               int box_rows, bool bf16, int d = 128) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return FA_ERR_DEVICE;
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)H, (cuuint64_t)S, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)sh * 2, (cuuint64_t)ss * 2, (cuuint64_t)sb * 2};
    // a dimension of extent 1 never advances; give it a harmless legal stride
    if (H == 1) strides[0] = (cuuint64_t)d * 2;
    if (S == 1) strides[1] = strides[0] * (cuuint64_t)H;
    if (B == 1) strides[2] = strides[1] * (cuuint64_t)S;
    cuuint32_t box[4] = {64, 1, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(tm, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4,
                    const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        t_last_cuda_error = static_cast<int>(r);
        return FA_ERR_CUDA;
    }
    return FA_OK;
}

// Tensor map over a [B, S, H, 128] one-byte tensor, contiguous: a box is box_rows sequence
// positions x 128 bytes for one (batch, head), 128-byte swizzled.
int encode_map_u8(CUtensorMap* tm, const void* base, int B, int S, int H, int box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return FA_ERR_DEVICE;
    cuuint64_t dims[4] = {128, (cuuint64_t)H, (cuuint64_t)S, (cuuint64_t)B};
    cuuint64_t strides[3] = {128, (cuuint64_t)H * 128, (cuuint64_t)S * H * 128};
    cuuint32_t box[4] = {128, 1, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        t_last_cuda_error = static_cast<int>(r);
        return FA_ERR_CUDA;
    }
    return FA_OK;
}

// Tensor map over a row-major [rows, cols] 16-bit matrix: a box is 64 rows x 64 columns, 128-byte
// swizzled (the projection weight, an N-major MMA operand).  Encoded with four dimensions so that
// the kernels' one load wrapper serves it; the outer two have extent 1.
int encode_map_matrix(CUtensorMap* tm, const void* base, int rows, int cols, bool bf16) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return FA_ERR_DEVICE;
    cuuint64_t dims[4] = {(cuuint64_t)cols, (cuuint64_t)rows, 1, 1};
    cuuint64_t strides[3] = {(cuuint64_t)cols * 2, (cuuint64_t)cols * 2 * rows, (cuuint64_t)cols * 2 * rows};
    cuuint32_t box[4] = {64, 64, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(tm, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4,
                    const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        t_last_cuda_error = static_cast<int>(r);
        return FA_ERR_CUDA;
    }
    return FA_OK;
}

// a page holds a multiple of the 128-key tile, or 16, 32 or 64 keys (several pages per tile)
bool page_size_ok(int ps) { return ps > 0 && (ps % fa::kDecTile == 0 || ps == 16 || ps == 32 || ps == 64); }

int check_device() {
    static thread_local int cached_dev = -1, cached_rc = FA_OK;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev == cached_dev) return cached_rc;
    int major = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return cuda_fail(e);
    cached_dev = dev;
    cached_rc = (major == 10) ? FA_OK : FA_ERR_DEVICE;
    return cached_rc;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

void default_strides(int64_t s[3], int S, int H, int d = 128) {
    if (s[0] == 0 && s[1] == 0 && s[2] == 0) {
        s[2] = d;
        s[1] = (int64_t)H * d;
        s[0] = (int64_t)S * H * d;
    }
}

bool strides_ok(const int64_t s[3], int B, int S, int H, int d = 128) {
    for (int i = 0; i < 3; ++i) {
        if (s[i] < 0 || (s[i] & 7)) return false;
        if (s[i] >= (1ll << 38)) return false;
    }
    if (H > 1 && s[2] < d) return false;
    if (S > 1 && s[1] < d) return false;
    if (B > 1 && s[0] < d) return false;
    return true;
}

template <typename K>
int set_smem(K kernel, int bytes) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return e == cudaSuccess ? FA_OK : cuda_fail(e);
}

constexpr int kSimpleSmem = 1024 + 6 * fa::kTileBytes;

template <typename T, bool kPInTmem>
int launch_simple(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const fa::FwdParams& fp,
                  cudaStream_t st) {
    auto kern = fa::fa_fwd_simple_kernel<T, kPInTmem>;
    int rc = set_smem(kern, kSimpleSmem);
    if (rc) return rc;
    dim3 grid(fp.n_qtiles, fp.Hq, fp.B);
    kern<<<grid, 128, kSimpleSmem, st>>>(tq, tk, tv, fp);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FA_OK : cuda_fail(e);
}

// Kernel parameters of a dense (not packed, not paged) forward from validated arguments whose
// strides have been filled in.
fa::FwdParams dense_fwd_params(const fa_params& p) {
    fa::FwdParams fp;
    fp.o = p.o;
    fp.lse = p.lse;
    fp.B = p.B; fp.Hq = p.Hq; fp.Hkv = p.Hkv; fp.Sq = p.Sq; fp.Skv = p.Skv;
    fp.causal = p.causal ? 1 : 0;
    // strictly positive, so that a hidden score (-inf) times the scale is -inf and never NaN;
    // for scale == 0 the substitute is far below anything fp32 scores could resolve
    fp.scale_log2 = fmaxf(p.scale * 1.4426950408889634f, 1e-30f);
    fp.o_sb = p.o_stride[0]; fp.o_ss = p.o_stride[1]; fp.o_sh = p.o_stride[2];
    fp.o_fp32 = (p.o_dtype == FA_DTYPE_FP32) ? 1 : 0;
    fp.n_qtiles = (p.Sq + fa::kTile - 1) / fa::kTile;
    fp.by_bh.set(p.B * p.Hq);
    fp.by_hq.set(p.Hq);
    fp.by_group.set(p.Hq / p.Hkv);
    fp.by_qtiles.set(fp.n_qtiles > 0 ? fp.n_qtiles : 1);
    fp.by_qpairs.set(fp.n_qtiles > 0 ? (fp.n_qtiles + 1) / 2 : 1);
    fp.cls_log2 = 0;  // set by the ping-pong launcher
    fp.by_class.set(1);
    fp.by_lastcls.set(1);
    fp.rounds_per_head = 0;
    fp.by_rph.set(1);
    fp.out_scale = 1.f;
    fp.cu_q = nullptr;
    fp.cu_k = nullptr;
    fp.total_q = 0;
    fp.block_table = nullptr;
    fp.seqlens_k = nullptr;
    fp.table_stride = 0;
    fp.page_size = 1;
    fp.by_tiles_per_page.set(1);
    fp.d = p.d;
    fp.o_align32 = ((reinterpret_cast<uintptr_t>(p.o) & 31u) == 0 && (p.o_stride[0] & 15) == 0 &&
                    (p.o_stride[1] & 15) == 0 && (p.o_stride[2] & 15) == 0) ? 1 : 0;
    return fp;
}

// Head dimension 64: keys from which the ping-pong kernel is used (128 < Skv <= 256 has the
// short-sequence pipeline of its own; up to 128 keys the kernel with four small CTAs per SM, which
// the ping-pong kernel ties there and beats by 3 to 37 % from 300 keys on).
#ifndef FA_D64_PINGPONG_FROM
#define FA_D64_PINGPONG_FROM 257
#endif
constexpr int kD64PingPongFrom = FA_D64_PINGPONG_FROM;

int forward_impl(const fa_params& in, cudaStream_t st) {
    fa_params p = in;
    // ---- validation (no CUDA call before it passes)
    if (p.B < 0 || p.Hq <= 0 || p.Hkv <= 0 || p.Sq < 0 || p.Skv < 0 || p.d <= 0) return FA_ERR_SHAPE;
    if (p.Hq % p.Hkv) return FA_ERR_SHAPE;
    if (p.d != 128 && p.d != 64 && p.d != 256) return FA_ERR_UNSUPPORTED;
    // d = 64 and d = 256 have kernels of their own (d = 64 also takes variant 3, the ping-pong kernel)
    if (p.d != 128 && p.variant != 0 && !(p.d == 64 && p.variant == 3)) return FA_ERR_UNSUPPORTED;
    if (p.dtype != FA_DTYPE_FP16 && p.dtype != FA_DTYPE_BF16) return FA_ERR_UNSUPPORTED;
    if (p.o_dtype != p.dtype && p.o_dtype != FA_DTYPE_FP32) return FA_ERR_UNSUPPORTED;
    if (!(p.scale >= 0.f) || isinf(p.scale)) return FA_ERR_UNSUPPORTED;
    if (p.causal && p.Sq > p.Skv) return FA_ERR_UNSUPPORTED;
    if (p.Hq > 65535 || p.B > 65535) return FA_ERR_UNSUPPORTED;
    if (p.B == 0 || p.Sq == 0) return FA_OK;
    if (!p.q || !p.o) return FA_ERR_NULL;
    if (p.Skv > 0 && (!p.k || !p.v)) return FA_ERR_NULL;
    default_strides(p.q_stride, p.Sq, p.Hq, p.d);
    default_strides(p.k_stride, p.Skv, p.Hkv, p.d);
    default_strides(p.v_stride, p.Skv, p.Hkv, p.d);
    default_strides(p.o_stride, p.Sq, p.Hq, p.d);
    if (!strides_ok(p.q_stride, p.B, p.Sq, p.Hq, p.d) || !strides_ok(p.k_stride, p.B, p.Skv, p.Hkv, p.d) ||
        !strides_ok(p.v_stride, p.B, p.Skv, p.Hkv, p.d) || !strides_ok(p.o_stride, p.B, p.Sq, p.Hq, p.d))
        return FA_ERR_SHAPE;
    if (!aligned16(p.q) || !aligned16(p.k) || !aligned16(p.v) || !aligned16(p.o)) return FA_ERR_ALIGN;
    if (p.lse && (reinterpret_cast<uintptr_t>(p.lse) & 3u)) return FA_ERR_ALIGN;

    int rc = check_device();
    if (rc) return rc;

    fa::FwdParams fp = dense_fwd_params(p);
    const bool bf16 = p.dtype == FA_DTYPE_BF16;

    if (p.Skv == 0) {
        const long long rows = (long long)p.B * p.Sq * p.Hq;
        const int blocks = (int)((rows + 127) / 128 < 4096 ? (rows + 127) / 128 : 4096);
        if (bf16) fa::fa_fill_empty_kernel<__nv_bfloat16><<<blocks, 128, 0, st>>>(fp);
        else fa::fa_fill_empty_kernel<__half><<<blocks, 128, 0, st>>>(fp);
        cudaError_t e = cudaGetLastError();
        return e == cudaSuccess ? FA_OK : cuda_fail(e);
    }

    CUtensorMap tq, tk, tv;
    rc = encode_map(&tq, p.q, p.B, p.Sq, p.Hq, p.q_stride[0], p.q_stride[1], p.q_stride[2], 128, bf16, p.d);
    if (rc) return rc;
    rc = encode_map(&tk, p.k, p.B, p.Skv, p.Hkv, p.k_stride[0], p.k_stride[1], p.k_stride[2], 128, bf16, p.d);
    if (rc) return rc;
    rc = encode_map(&tv, p.v, p.B, p.Skv, p.Hkv, p.v_stride[0], p.v_stride[1], p.v_stride[2], 128, bf16, p.d);
    if (rc) return rc;

    if (p.d == 64 && (p.variant == 3 || (p.variant == 0 && p.Skv >= kD64PingPongFrom))) {
        // long sequences: the ping-pong kernel with tiles of one 64-element box (see PpOperands)
        CUtensorMap to = tq;
        if (!fp.o_fp32) {  // the output leaves through TMA stores of 32 rows x 64 columns
            rc = encode_map(&to, p.o, p.B, p.Sq, p.Hq, p.o_stride[0], p.o_stride[1], p.o_stride[2], 32, bf16, 64);
            if (rc) return rc;
        }
        return bf16 ? fa::launch_pingpong<__nv_bfloat16, false, 64>(tq, tk, tv, to, fp, st, &t_last_cuda_error)
                    : fa::launch_pingpong<__half, false, 64>(tq, tk, tv, to, fp, st, &t_last_cuda_error);
    }
    if (p.d == 64 && p.Skv > 128 && p.Skv <= 256) {   // (unless the ping-pong kernel was asked for)
        // short sequences: all keys are one tile; a persistent pipeline over (batch, head, two query tiles)
        return bf16 ? fa::launch_d64_stream<__nv_bfloat16>(tq, tk, tv, fp, st, &t_last_cuda_error)
                    : fa::launch_d64_stream<__half>(tq, tk, tv, fp, st, &t_last_cuda_error);
    }
    if (p.d == 64) {  // one CTA per (batch, head, query tile), four CTAs per SM
        auto kern = bf16 ? fa::fa_fwd_d64_slim_kernel<__nv_bfloat16> : fa::fa_fwd_d64_slim_kernel<__half>;
        int sm_count = 0;
        if (int ce = fa::prepare_big_smem_kernel(reinterpret_cast<const void*>(kern), fa::kD64SlimSmem, &sm_count))
            return cuda_fail(static_cast<cudaError_t>(ce));
        dim3 grid(fp.n_qtiles, fp.Hq, fp.B);
        kern<<<grid, 128, fa::kD64SlimSmem, st>>>(tq, tk, tv, fp);
        cudaError_t e = cudaGetLastError();
        return e == cudaSuccess ? FA_OK : cuda_fail(e);
    }

    if (p.d == 256) {  // one CTA per (batch, head, query tile), one CTA per SM
        auto kern = bf16 ? fa::fa_fwd_d256_kernel<__nv_bfloat16> : fa::fa_fwd_d256_kernel<__half>;
        int sm_count = 0;
        if (int ce = fa::prepare_big_smem_kernel(reinterpret_cast<const void*>(kern), fa::kD256Smem, &sm_count))
            return cuda_fail(static_cast<cudaError_t>(ce));
        CUtensorMap tvh;   // V in boxes of 64 keys: the kernel's V slots hold half a tile
        rc = encode_map(&tvh, p.v, p.B, p.Skv, p.Hkv, p.v_stride[0], p.v_stride[1], p.v_stride[2], 64, bf16, p.d);
        if (rc) return rc;
        dim3 grid(fp.n_qtiles, fp.Hq, fp.B);
        kern<<<grid, fa::kD256Threads, fa::kD256Smem, st>>>(tq, tk, tvh, fp);
        cudaError_t e = cudaGetLastError();
        return e == cudaSuccess ? FA_OK : cuda_fail(e);
    }

    // Default choice, from timings of both kernels on B200: the ping-pong kernel (one query tile
    // per CTA, Q K^T running ahead of the softmax) wins from 1024 keys on; the paired-tile kernel
    // keeps an edge on shorter sequences, where items change every few steps.
    int variant = p.variant;
    if (variant == 0) variant = (p.Skv >= 1024) ? 3 : 4;
    switch (variant) {
        case 4:  // pipelined kernel, two query tiles per CTA
            return bf16 ? fa::launch_pipelined<__nv_bfloat16>(tq, tk, tv, fp, st, &t_last_cuda_error)
                        : fa::launch_pipelined<__half>(tq, tk, tv, fp, st, &t_last_cuda_error);
        case 1:  // simple kernel, P handed over through tensor memory
            return bf16 ? launch_simple<__nv_bfloat16, true>(tq, tk, tv, fp, st)
                        : launch_simple<__half, true>(tq, tk, tv, fp, st);
        case 2:  // simple kernel, P handed over through shared memory
            return bf16 ? launch_simple<__nv_bfloat16, false>(tq, tk, tv, fp, st)
                        : launch_simple<__half, false>(tq, tk, tv, fp, st);
        case 3: {  // ping-pong kernel: one query tile per CTA, two softmax warpgroups alternate over kv steps
            CUtensorMap to = tq;
            if (!fp.o_fp32) {  // the output leaves through TMA stores of 32 rows x 64 columns
                rc = encode_map(&to, p.o, p.B, p.Sq, p.Hq, p.o_stride[0], p.o_stride[1], p.o_stride[2], 32, bf16);
                if (rc) return rc;
            }
            return bf16 ? fa::launch_pingpong<__nv_bfloat16>(tq, tk, tv, to, fp, st, &t_last_cuda_error)
                        : fa::launch_pingpong<__half>(tq, tk, tv, to, fp, st, &t_last_cuda_error);
        }
        default:
            return FA_ERR_UNSUPPORTED;
    }
}

// Streams and events of fa_forward_host, made once per device and kept for the life of the
// process (host-side objects; no device memory).
constexpr int kHostParts = 4;
struct HostPipe {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t start = nullptr, finish = nullptr, in_done[kHostParts] = {}, fwd_done[kHostParts] = {};
    bool ready = false;
    // held by fa_forward_host from its first event record to its last wait: the events are shared
    // by every call on the device, so two host threads must not interleave their enqueue sequences
    std::mutex enqueue;
};
HostPipe* host_pipe() {
    constexpr int kMaxDev = 64;
    static HostPipe pipes[kMaxDev];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    HostPipe& hp = pipes[dev];
    if (!hp.ready) {
        bool ok = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.finish, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < kHostParts; ++i)
            ok = cudaEventCreateWithFlags(&hp.in_done[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.fwd_done[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            t_last_cuda_error = static_cast<int>(cudaGetLastError());
            return nullptr;
        }
        hp.ready = true;
    }
    return &hp;
}

int forward_plain(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv,
                  int Sq, int Skv, int d, int causal, float scale, int dtype, void* stream) {
    fa_params p;
    memset(&p, 0, sizeof p);
    p.q = q; p.k = k; p.v = v; p.o = o; p.lse = lse;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Sq = Sq; p.Skv = Skv; p.d = d;
    p.causal = causal; p.scale = scale; p.dtype = dtype; p.o_dtype = dtype;
    return forward_impl(p, static_cast<cudaStream_t>(stream));
}

// ---- decode helpers
// long_ok: the 16-bit kernels; the FP8 kernel measured 1 % slower with 4096-key chunks and keeps
// 2048.  The workspace functions size for the shorter chunks, which covers both.
int decode_chunk(int B, int Hkv, int Smax, bool long_ok = false) {
    // Keys per work item (multiples of the tile).  A CTA costs a few microseconds on top of its
    // tiles (launch, the first loads' latency, the merge), so chunks are as long as the number of
    // work items allows: 4096 keys when that still gives eight waves on 148 SMs, 2048 keys when
    // that gives four (sequences of different lengths then balance well; 4096 against 2048 keys
    // on 64 sequences of 1K to 32K keys: 2.38 against 2.43 ms with 32 kv heads, 0.606 against
    // 0.615 ms with 8; 8192 keys are level with 2048, 1024 slower); otherwise the longest chunk, up to 4096 keys, that
    // keeps about one work item per SM (timed on one to sixteen sequences of 4K to 128K keys: e.g.
    // one sequence of 32K keys with 8 kv heads takes 32 us with 2048-key chunks against 61 us with
    // 256-key chunks); 256 keys when even that leaves SMs without work.
    auto items = [&](int chunk) { return (long long)B * Hkv * ((Smax + chunk - 1) / chunk); };
    if (long_ok && items(4096) >= 8ll * 148) return 4096;
    if (items(2048) >= 4ll * 148) return 2048;
    for (int chunk = 4096; chunk > 256; chunk >>= 1)
        if (items(chunk) >= 120) return chunk;
    return 256;
}

}  // namespace

extern "C" {

int fa_forward(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv, int Sq,
               int Skv, int d, int causal, float scale, void* stream) {
    return forward_plain(q, k, v, o, lse, B, Hq, Hkv, Sq, Skv, d, causal, scale, FA_DTYPE_FP16, stream);
}

int fa_forward_bf16(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv,
                    int Sq, int Skv, int d, int causal, float scale, void* stream) {
    return forward_plain(q, k, v, o, lse, B, Hq, Hkv, Sq, Skv, d, causal, scale, FA_DTYPE_BF16, stream);
}

int fa_forward_fp8(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq, int Hkv, int Sq,
                   int Skv, int d, int causal, float scale, float q_scale, float k_scale, float v_scale, int o_dtype,
                   void* stream) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || Sq < 0 || Skv < 0 || d <= 0) return FA_ERR_SHAPE;
    if (Hq % Hkv) return FA_ERR_SHAPE;
    if (d != 128) return FA_ERR_UNSUPPORTED;
    if (o_dtype != FA_DTYPE_FP16 && o_dtype != FA_DTYPE_BF16) return FA_ERR_UNSUPPORTED;
    if (!(scale >= 0.f) || isinf(scale)) return FA_ERR_UNSUPPORTED;
    if (!(q_scale > 0.f) || isinf(q_scale) || !(k_scale > 0.f) || isinf(k_scale) || !(v_scale > 0.f) || isinf(v_scale))
        return FA_ERR_UNSUPPORTED;
    if (causal && Sq > Skv) return FA_ERR_UNSUPPORTED;
    if (Hq > 65535 || B > 65535) return FA_ERR_UNSUPPORTED;
    if (B == 0 || Sq == 0) return FA_OK;
    if (!q || !o) return FA_ERR_NULL;
    if (Skv > 0 && (!k || !v)) return FA_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return FA_ERR_ALIGN;
    if (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) return FA_ERR_ALIGN;
    int rc = check_device();
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool bf16 = o_dtype == FA_DTYPE_BF16;

    fa::FwdParams fp;
    fp.o = o;
    fp.lse = lse;
    fp.B = B; fp.Hq = Hq; fp.Hkv = Hkv; fp.Sq = Sq; fp.Skv = Skv;
    fp.causal = causal ? 1 : 0;
    // the scores are products of the stored 8-bit values: both factors go into the softmax scale
    fp.scale_log2 = fmaxf(scale * q_scale * k_scale * 1.4426950408889634f, 1e-30f);
    fp.o_sb = (long long)Sq * Hq * 128; fp.o_ss = (long long)Hq * 128; fp.o_sh = 128;
    fp.o_fp32 = 0;
    fp.o_align32 = 0;
    fp.n_qtiles = (Sq + fa::kTile - 1) / fa::kTile;
    fp.by_bh.set(B * Hq);
    fp.by_hq.set(Hq);
    fp.by_group.set(Hq / Hkv);
    fp.by_qtiles.set(fp.n_qtiles);
    fp.by_qpairs.set((fp.n_qtiles + 1) / 2);
    fp.cls_log2 = 0;
    fp.by_class.set(1);
    fp.by_lastcls.set(1);
    fp.rounds_per_head = 0;
    fp.by_rph.set(1);
    fp.out_scale = v_scale;
    fp.cu_q = nullptr;
    fp.cu_k = nullptr;
    fp.total_q = 0;
    fp.block_table = nullptr;
    fp.seqlens_k = nullptr;
    fp.table_stride = 0;
    fp.page_size = 1;
    fp.by_tiles_per_page.set(1);
    fp.d = 128;
    if (Skv == 0) {
        const long long rows = (long long)B * Sq * Hq;
        const int blocks = (int)((rows + 127) / 128 < 4096 ? (rows + 127) / 128 : 4096);
        if (bf16) fa::fa_fill_empty_kernel<__nv_bfloat16><<<blocks, 128, 0, st>>>(fp);
        else fa::fa_fill_empty_kernel<__half><<<blocks, 128, 0, st>>>(fp);
        cudaError_t e = cudaGetLastError();
        return e == cudaSuccess ? FA_OK : cuda_fail(e);
    }
    CUtensorMap tq, tk, tv, to;
    rc = encode_map_u8(&tq, q, B, Sq, Hq, 128);
    if (rc) return rc;
    rc = encode_map_u8(&tk, k, B, Skv, Hkv, 128);
    if (rc) return rc;
    rc = encode_map_u8(&tv, v, B, Skv, Hkv, 128);
    if (rc) return rc;
    rc = encode_map(&to, o, B, Sq, Hq, (int64_t)Sq * Hq * 128, (int64_t)Hq * 128, 128, 32, bf16);
    if (rc) return rc;
    return bf16 ? fa::launch_pingpong<__nv_bfloat16, true>(tq, tk, tv, to, fp, st, &t_last_cuda_error)
                : fa::launch_pingpong<__half, true>(tq, tk, tv, to, fp, st, &t_last_cuda_error);
}

size_t fa_forward_proj_workspace_bytes(int B, int Sq) {
    if (B <= 0 || Sq <= 0) return 0;
    return (size_t)B * ((Sq + fa::kTile - 1) / fa::kTile) * sizeof(unsigned int);
}

int fa_forward_proj(const void* q, const void* k, const void* v, const void* w_o, void* o, float* lse, void* out,
                    int B, int Hq, int Hkv, int Sq, int Skv, int d, int d_model, int causal, float scale, int dtype,
                    int fused, void* workspace, size_t workspace_bytes, void* stream) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || Sq < 0 || Skv < 0 || d <= 0 || d_model <= 0) return FA_ERR_SHAPE;
    if (Hq % Hkv) return FA_ERR_SHAPE;
    if (d != 128 || d_model % 256) return FA_ERR_UNSUPPORTED;
    if (dtype != FA_DTYPE_FP16 && dtype != FA_DTYPE_BF16) return FA_ERR_UNSUPPORTED;
    if (!(scale >= 0.f) || isinf(scale)) return FA_ERR_UNSUPPORTED;
    if (causal && Sq > Skv) return FA_ERR_UNSUPPORTED;
    if (Hq > 16383 || B > 65535) return FA_ERR_UNSUPPORTED;
    if ((long long)B * ((Sq + fa::kTile - 1) / fa::kTile) * (d_model / 256) > 0x7fffffffll) return FA_ERR_UNSUPPORTED;
    if (B == 0 || Sq == 0) return FA_OK;
    if (!q || !o || !out || !w_o) return FA_ERR_NULL;
    if (Skv > 0 && (!k || !v)) return FA_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(w_o)) return FA_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(out) & 31u) return FA_ERR_ALIGN;
    if (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) return FA_ERR_ALIGN;
    if (fused) {
        if (reinterpret_cast<uintptr_t>(workspace) & 3u) return FA_ERR_ALIGN;
        if (!workspace || workspace_bytes < fa_forward_proj_workspace_bytes(B, Sq)) return FA_ERR_WORKSPACE;
    }
    int rc = check_device();
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool bf16 = dtype == FA_DTYPE_BF16;
    cudaError_t e;

    fa_params ap;
    memset(&ap, 0, sizeof ap);
    ap.q = q; ap.k = k; ap.v = v; ap.o = o; ap.lse = lse;
    ap.B = B; ap.Hq = Hq; ap.Hkv = Hkv; ap.Sq = Sq; ap.Skv = Skv; ap.d = d;
    ap.causal = causal; ap.scale = scale; ap.dtype = dtype; ap.o_dtype = dtype;
    ap.variant = 3;   // the ping-pong kernel in both forms, so that they compute the same O
    default_strides(ap.q_stride, Sq, Hq);
    default_strides(ap.k_stride, Skv, Hkv);
    default_strides(ap.v_stride, Skv, Hkv);
    default_strides(ap.o_stride, Sq, Hq);

    fa::ProjParams pp;
    pp.out = out;
    pp.B = B; pp.Sq = Sq; pp.Hq = Hq; pp.N = d_model;
    pp.n_qtiles = (Sq + fa::kTile - 1) / fa::kTile;
    pp.n_cblocks = d_model / 256;
    pp.done = nullptr;
    pp.done_target = 4u * (unsigned int)Hq;

    CUtensorMap tq, tk, tv, to, ta, tw;
    // O as the projection's K-major operand: the attention output read back in 128 x 64 boxes
    rc = encode_map(&ta, o, B, Sq, Hq, (int64_t)Sq * Hq * 128, (int64_t)Hq * 128, 128, 128, bf16);
    if (rc) return rc;
    rc = encode_map_matrix(&tw, w_o, Hq * 128, d_model, bf16);
    if (rc) return rc;

    if (!fused || Skv == 0) {
        // two launches: the attention kernel (or, without keys, the fill that writes O = 0), then the projection
        rc = forward_impl(ap, st);
        if (rc) return rc;
        rc = bf16 ? fa::launch_proj<__nv_bfloat16>(ta, tw, ta, ta, ta, tw, dense_fwd_params(ap), pp, 0, st, &t_last_cuda_error)
                  : fa::launch_proj<__half>(ta, tw, ta, ta, ta, tw, dense_fwd_params(ap), pp, 0, st, &t_last_cuda_error);
        return rc;
    }
    e = cudaMemsetAsync(workspace, 0, fa_forward_proj_workspace_bytes(B, Sq), st);
    if (e != cudaSuccess) return cuda_fail(e);
    pp.done = static_cast<unsigned int*>(workspace);
    rc = encode_map(&tq, q, B, Sq, Hq, ap.q_stride[0], ap.q_stride[1], ap.q_stride[2], 128, bf16);
    if (rc) return rc;
    rc = encode_map(&tk, k, B, Skv, Hkv, ap.k_stride[0], ap.k_stride[1], ap.k_stride[2], 128, bf16);
    if (rc) return rc;
    rc = encode_map(&tv, v, B, Skv, Hkv, ap.v_stride[0], ap.v_stride[1], ap.v_stride[2], 128, bf16);
    if (rc) return rc;
    rc = encode_map(&to, o, B, Sq, Hq, ap.o_stride[0], ap.o_stride[1], ap.o_stride[2], 32, bf16);
    if (rc) return rc;
    const fa::FwdParams fp = dense_fwd_params(ap);
    return bf16 ? fa::launch_proj<__nv_bfloat16>(tq, tk, tv, to, ta, tw, fp, pp, 1, st, &t_last_cuda_error)
                : fa::launch_proj<__half>(tq, tk, tv, to, ta, tw, fp, pp, 1, st, &t_last_cuda_error);
}

int fa_forward_ex(const fa_params* p, void* stream) {
    if (!p) return FA_ERR_NULL;
    return forward_impl(*p, static_cast<cudaStream_t>(stream));
}

// Packed batch; K and V packed too (block_table == nullptr: k, v [total_k,Hkv,d], cu_seqlens_k) or in
// pages (k, v [num_pages,page_size,Hkv,d], seqlens_k and the block table; total_k = num_pages * page_size).
static int varlen_impl(const void* q, const void* k, const void* v, void* o, float* lse, const int* cu_seqlens_q,
                       const int* cu_seqlens_k, int B, int Hq, int Hkv, int total_q, int total_k, int max_seqlen_q,
                       int max_seqlen_k, int d, int causal, float scale, int dtype, void* stream,
                       const int* block_table, int num_pages, int page_size, int table_stride) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || total_q < 0 || total_k < 0 || max_seqlen_q < 0 || max_seqlen_k < 0 || d <= 0)
        return FA_ERR_SHAPE;
    if (Hq % Hkv) return FA_ERR_SHAPE;
    if (max_seqlen_q > total_q || (!block_table && max_seqlen_k > total_k)) return FA_ERR_SHAPE;
    if (d != 128 && d != 64) return FA_ERR_UNSUPPORTED;
    if (dtype != FA_DTYPE_FP16 && dtype != FA_DTYPE_BF16) return FA_ERR_UNSUPPORTED;
    if (!(scale >= 0.f) || isinf(scale)) return FA_ERR_UNSUPPORTED;
    if (Hq > 65535 || B > 65535) return FA_ERR_UNSUPPORTED;
    if (B == 0 || total_q == 0 || max_seqlen_q == 0) return FA_OK;
    if (!q || !o || !cu_seqlens_q || !cu_seqlens_k) return FA_ERR_NULL;
    if (total_k > 0 && (!k || !v)) return FA_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return FA_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(cu_seqlens_q) | reinterpret_cast<uintptr_t>(cu_seqlens_k) |
         reinterpret_cast<uintptr_t>(lse)) & 3u)
        return FA_ERR_ALIGN;
    int rc = check_device();
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool bf16 = dtype == FA_DTYPE_BF16;

    fa::FwdParams fp;
    fp.o = o;
    fp.lse = lse;
    fp.B = B; fp.Hq = Hq; fp.Hkv = Hkv; fp.Sq = max_seqlen_q; fp.Skv = max_seqlen_k;
    fp.causal = causal ? 1 : 0;
    fp.scale_log2 = fmaxf(scale * 1.4426950408889634f, 1e-30f);
    fp.o_sb = 0; fp.o_ss = (long long)Hq * d; fp.o_sh = d;
    fp.o_fp32 = 0;
    fp.o_align32 = 0;
    fp.n_qtiles = (max_seqlen_q + fa::kTile - 1) / fa::kTile;
    fp.by_bh.set(B * Hq);
    fp.by_hq.set(Hq);
    fp.by_group.set(Hq / Hkv);
    fp.by_qtiles.set(fp.n_qtiles);
    fp.by_qpairs.set((fp.n_qtiles + 1) / 2);
    fp.cls_log2 = 0;
    fp.by_class.set(1);
    fp.by_lastcls.set(1);
    fp.rounds_per_head = 0;
    fp.by_rph.set(1);
    fp.out_scale = 1.f;
    fp.cu_q = cu_seqlens_q;
    fp.cu_k = cu_seqlens_k;
    fp.total_q = total_q;
    fp.d = d;
    fp.block_table = block_table;
    fp.seqlens_k = block_table ? cu_seqlens_k : nullptr;   // per-sequence key counts in the paged form
    fp.table_stride = table_stride;
    fp.page_size = block_table ? page_size : 1;
    fp.by_tiles_per_page.set(block_table ? page_size / fa::kTile : 1);

    if (total_k == 0 || max_seqlen_k == 0) {
        // no keys anywhere: O = 0, LSE = -inf over the packed rows, seen as one sequence
        fa::FwdParams fe = fp;
        fe.B = 1; fe.Sq = total_q;
        const long long rows = (long long)total_q * Hq;
        const int blocks = (int)((rows + 127) / 128 < 4096 ? (rows + 127) / 128 : 4096);
        if (bf16) fa::fa_fill_empty_kernel<__nv_bfloat16><<<blocks, 128, 0, st>>>(fe);
        else fa::fa_fill_empty_kernel<__half><<<blocks, 128, 0, st>>>(fe);
        cudaError_t e = cudaGetLastError();
        return e == cudaSuccess ? FA_OK : cuda_fail(e);
    }
    // the packed tensors as one batch entry; a sequence's rows are reached through the prefix sums
    CUtensorMap tq, tk, tv, to;
    rc = encode_map(&tq, q, 1, total_q, Hq, (int64_t)total_q * Hq * d, (int64_t)Hq * d, d, 128, bf16, d);
    if (rc) return rc;
    // K and V: one batch entry with every sequence back to back, or one entry per page
    const int slabs = block_table ? num_pages : 1, slab_rows = block_table ? page_size : total_k;
    rc = encode_map(&tk, k, slabs, slab_rows, Hkv, (int64_t)slab_rows * Hkv * d, (int64_t)Hkv * d, d, 128, bf16, d);
    if (rc) return rc;
    rc = encode_map(&tv, v, slabs, slab_rows, Hkv, (int64_t)slab_rows * Hkv * d, (int64_t)Hkv * d, d, 128, bf16, d);
    if (rc) return rc;
    rc = encode_map(&to, o, 1, total_q, Hq, (int64_t)total_q * Hq * d, (int64_t)Hq * d, d, 32, bf16, d);
    if (rc) return rc;
    if (d == 64)
        return bf16 ? fa::launch_pingpong<__nv_bfloat16, false, 64>(tq, tk, tv, to, fp, st, &t_last_cuda_error)
                    : fa::launch_pingpong<__half, false, 64>(tq, tk, tv, to, fp, st, &t_last_cuda_error);
    return bf16 ? fa::launch_pingpong<__nv_bfloat16>(tq, tk, tv, to, fp, st, &t_last_cuda_error)
                : fa::launch_pingpong<__half>(tq, tk, tv, to, fp, st, &t_last_cuda_error);
}

int fa_forward_varlen(const void* q, const void* k, const void* v, void* o, float* lse, const int* cu_seqlens_q,
                      const int* cu_seqlens_k, int B, int Hq, int Hkv, int total_q, int total_k, int max_seqlen_q,
                      int max_seqlen_k, int d, int causal, float scale, int dtype, void* stream) {
    return varlen_impl(q, k, v, o, lse, cu_seqlens_q, cu_seqlens_k, B, Hq, Hkv, total_q, total_k, max_seqlen_q,
                       max_seqlen_k, d, causal, scale, dtype, stream, nullptr, 0, 0, 0);
}

int fa_forward_varlen_paged(const void* q, const void* k_pages, const void* v_pages, const int* block_table, void* o,
                            float* lse, const int* cu_seqlens_q, const int* seqlens_k, int B, int Hq, int Hkv,
                            int total_q, int num_pages, int page_size, int max_pages, int table_stride,
                            int max_seqlen_q, int max_seqlen_k, int d, int causal, float scale, int dtype, void* stream) {
    if (num_pages < 0 || max_pages < 0 || page_size <= 0 || page_size % fa::kTile) return FA_ERR_SHAPE;
    if (table_stride < max_pages) return FA_ERR_SHAPE;
    if ((long long)num_pages * page_size > 0x7fffffffll) return FA_ERR_SHAPE;
    if (max_seqlen_k > (long long)max_pages * page_size) return FA_ERR_SHAPE;
    if (B > 0 && max_pages > 0 && !block_table) return FA_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(block_table) & 3u) return FA_ERR_ALIGN;
    if (num_pages == 0) max_seqlen_k = 0;
    return varlen_impl(q, k_pages, v_pages, o, lse, cu_seqlens_q, seqlens_k, B, Hq, Hkv, total_q, num_pages * page_size,
                       max_seqlen_q, max_seqlen_k, d, causal, scale, dtype, stream, block_table, num_pages, page_size,
                       table_stride);
}

size_t fa_decode_workspace_bytes(int B, int Hq, int Hkv, int Skv_max, int d) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Skv_max <= 0 || (d != 128 && d != 64)) return 0;
    const int chunk = decode_chunk(B, Hkv, Skv_max);
    const size_t nc = (size_t)((Skv_max + chunk - 1) / chunk);
    return (size_t)B * Hq * nc * ((size_t)d + 1) * sizeof(float);
}

size_t fa_decode_append_workspace_bytes(int B, int Sq, int Hq, int Hkv, int Skv_max, int d) {
    if (Sq <= 0) return 0;
    return (size_t)Sq * fa_decode_workspace_bytes(B, Hq, Hkv, Skv_max, d);
}

}  // extern "C"

namespace {
// The argument checks every 16-bit decode entry point shares, in the order the header documents
// (shape, unsupported, NULL, alignment); no CUDA call.  B == 0 passes: the caller returns FA_OK.
int decode_check_args(const void* q, const void* k_cache, const void* v_cache, const void* o, const int* seqlens_k,
                      int B, int Hq, int Hkv, int Skv_max, int d, float scale, int Sq) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || Skv_max < 0 || d <= 0 || Sq < 1) return FA_ERR_SHAPE;
    if (Sq > 64 || Sq > Skv_max) return FA_ERR_UNSUPPORTED;   // several query rows are the LAST rows of the cache
    if (Hq % Hkv) return FA_ERR_SHAPE;
    if (d != 128 && d != 64) return FA_ERR_UNSUPPORTED;
    if (!(scale >= 0.f) || isinf(scale)) return FA_ERR_UNSUPPORTED;
    if (B > 65535 || Hq > 65535) return FA_ERR_UNSUPPORTED;
    if (B == 0) return FA_OK;
    if (!q || !o || !seqlens_k) return FA_ERR_NULL;
    if (Skv_max > 0 && (!k_cache || !v_cache)) return FA_ERR_NULL;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o)) return FA_ERR_ALIGN;
    return FA_OK;
}

// Launch of the merge kernel as a programmatic dependent of the split kernel before it in the
// stream: its launch is processed while the split kernel still runs, and its blocks start (they
// wait in griddepcontrol.wait) when the last block of the split kernel has finished and its
// writes are visible.
template <typename T, int D>
cudaError_t launch_combine(const fa::DecodeParams& dp, int blocks, void* o, float* lse, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(D);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fa::fa_decode_combine_kernel<T, D>, dp, static_cast<T*>(o), lse);
}

// Launch of the split kernel and of the merge for one head dimension.
template <int D>
int decode_launch(const CUtensorMap& tk, const CUtensorMap& tv, const fa::DecodeParams& dp, void* o, float* lse, int g,
                  bool bf16, bool direct, bool have_keys, cudaStream_t st) {
    const int B = dp.B, Sq = dp.Sq, Hq = dp.Hq, Hkv = dp.Hkv;
    if (have_keys) {
        constexpr int smem = fa::DecShape<D>::kSmem;
        int sm_count = 0;
        // at most 8 (token, head) rows per kv head: the keys-as-rows form of the consumers
        const bool key_rows = g * Sq <= 8;
        auto kern = bf16 ? ((Sq > 1) ? (key_rows ? fa::fa_decode_split_mma_kernel<true, __nv_bfloat16, D, true>
                                                 : fa::fa_decode_split_mma_kernel<true, __nv_bfloat16, D>)
                                     : (key_rows ? fa::fa_decode_split_mma_kernel<false, __nv_bfloat16, D, true>
                                                 : fa::fa_decode_split_mma_kernel<false, __nv_bfloat16, D>))
                         : ((Sq > 1) ? (key_rows ? fa::fa_decode_split_mma_kernel<true, __half, D, true>
                                                 : fa::fa_decode_split_mma_kernel<true, __half, D>)
                                     : (key_rows ? fa::fa_decode_split_mma_kernel<false, __half, D, true>
                                                 : fa::fa_decode_split_mma_kernel<false, __half, D>));
        if (int ce = fa::prepare_big_smem_kernel(reinterpret_cast<const void*>(kern), smem, &sm_count))
            return cuda_fail(static_cast<cudaError_t>(ce));
        dim3 grid(Hkv * ((g * Sq + 15) / 16), dp.n_chunks, B);   // 16 (token, head) rows per CTA
        kern<<<grid, fa::kDecMmaThreads, smem, st>>>(tk, tv, dp);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(e);
    }
    if (direct) return FA_OK;
    cudaError_t e = bf16 ? launch_combine<__nv_bfloat16, D>(dp, B * Sq * Hq, o, lse, st)
                         : launch_combine<__half, D>(dp, B * Sq * Hq, o, lse, st);
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? FA_OK : cuda_fail(e);
}

// Decode over a contiguous cache (block_table == nullptr; k_cache, v_cache [B,Skv_max,Hkv,d])
// or over pages (k_cache, v_cache [num_pages,page_size,Hkv,d]; Skv_max = max_pages * page_size).
int decode_impl(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse, const int* seqlens_k,
                int B, int Hq, int Hkv, int Skv_max, int d, float scale, void* workspace, size_t workspace_bytes,
                void* stream, const int* block_table, int num_pages, int page_size, int table_stride, int Sq = 1,
                bool bf16 = false) {
    int rc = decode_check_args(q, k_cache, v_cache, o, seqlens_k, B, Hq, Hkv, Skv_max, d, scale, Sq);
    if (rc) return rc;
    if (B == 0) return FA_OK;
    if (!aligned16(workspace)) return FA_ERR_ALIGN;
    const size_t need = fa_decode_append_workspace_bytes(B, Sq, Hq, Hkv, Skv_max, d);
    if (need > 0 && (!workspace || workspace_bytes < need)) return FA_ERR_WORKSPACE;
    rc = check_device();
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    fa::DecodeParams dp;
    dp.q = q;
    dp.seqlens = seqlens_k;
    dp.B = B; dp.Hq = Hq; dp.Hkv = Hkv; dp.Smax = Skv_max;
    dp.Sq = Sq;
    dp.chunk = Skv_max > 0 ? decode_chunk(B, Hkv, Skv_max, true) : 256;
    dp.n_chunks = Skv_max > 0 ? (Skv_max + dp.chunk - 1) / dp.chunk : 1;
    if (dp.n_chunks > 65535) return FA_ERR_UNSUPPORTED;   // the chunks are the grid's second dimension
    dp.o_part = static_cast<float*>(workspace);
    dp.lse_part = dp.o_part + (size_t)B * Sq * Hq * dp.n_chunks * d;
    dp.scale_log2 = scale * 1.4426950408889634f;
    dp.block_table = block_table;
    dp.page_size = block_table ? page_size : 1;
    dp.table_stride = table_stride;
    dp.v_scale = 1.f;
    // one chunk per sequence: the split kernel writes the result itself, no merge kernel
    const bool direct = Skv_max > 0 && dp.n_chunks == 1;
    dp.o_final = direct ? o : nullptr;
    dp.lse_final = direct ? lse : nullptr;
    const int g = Hq / Hkv;

    CUtensorMap tk, tv;
    if (Skv_max > 0) {
        // the outermost dimension of the maps is the sequence, or the page
        const int slabs = block_table ? num_pages : B;
        const int slab_rows = block_table ? page_size : Skv_max;
        const int box_rows = (block_table && page_size < fa::kDecTile) ? page_size : fa::kDecTile;
        rc = encode_map(&tk, k_cache, slabs, slab_rows, Hkv, (int64_t)slab_rows * Hkv * d, (int64_t)Hkv * d, d,
                        box_rows, bf16, d);
        if (rc) return rc;
        rc = encode_map(&tv, v_cache, slabs, slab_rows, Hkv, (int64_t)slab_rows * Hkv * d, (int64_t)Hkv * d, d,
                        box_rows, bf16, d);
        if (rc) return rc;
    }
    return d == 64 ? decode_launch<64>(tk, tv, dp, o, lse, g, bf16, direct, Skv_max > 0, st)
                   : decode_launch<128>(tk, tv, dp, o, lse, g, bf16, direct, Skv_max > 0, st);
}
}  // namespace

extern "C" {

int fa_decode(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse, const int* seqlens_k,
              int B, int Hq, int Hkv, int Skv_max, int d, float scale, void* workspace, size_t workspace_bytes,
              void* stream) {
    return decode_impl(q, k_cache, v_cache, o, lse, seqlens_k, B, Hq, Hkv, Skv_max, d, scale, workspace,
                       workspace_bytes, stream, nullptr, 0, 0, 0);
}

// FP8 cache, contiguous (block_table == nullptr) or in pages (Skv_max = max_pages * page_size).
static int decode_fp8_impl(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                           const int* seqlens_k, int B, int Hq, int Hkv, int Skv_max, int d, float scale, float k_scale,
                           float v_scale, void* workspace, size_t workspace_bytes, void* stream, const int* block_table,
                           int num_pages, int page_size, int table_stride, bool bf16 = false) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || Skv_max < 0 || d <= 0) return FA_ERR_SHAPE;
    if (Hq % Hkv) return FA_ERR_SHAPE;
    if (d != 128) return FA_ERR_UNSUPPORTED;
    if (!(scale >= 0.f) || isinf(scale)) return FA_ERR_UNSUPPORTED;
    if (!(k_scale > 0.f) || isinf(k_scale) || !(v_scale > 0.f) || isinf(v_scale)) return FA_ERR_UNSUPPORTED;
    if (B > 65535 || Hq > 65535) return FA_ERR_UNSUPPORTED;
    if (B == 0) return FA_OK;
    if (!q || !o || !seqlens_k) return FA_ERR_NULL;
    if (Skv_max > 0 && (!k_cache || !v_cache)) return FA_ERR_NULL;
    if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(o) || !aligned16(workspace))
        return FA_ERR_ALIGN;
    const size_t need = fa_decode_workspace_bytes(B, Hq, Hkv, Skv_max, d);
    if (need > 0 && (!workspace || workspace_bytes < need)) return FA_ERR_WORKSPACE;
    int rc = check_device();
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    fa::DecodeParams dp;
    dp.q = q;
    dp.seqlens = seqlens_k;
    dp.B = B; dp.Hq = Hq; dp.Hkv = Hkv; dp.Smax = Skv_max;
    dp.chunk = Skv_max > 0 ? decode_chunk(B, Hkv, Skv_max) : 256;
    dp.n_chunks = Skv_max > 0 ? (Skv_max + dp.chunk - 1) / dp.chunk : 1;
    if (dp.n_chunks > 65535) return FA_ERR_UNSUPPORTED;   // the chunks are the grid's second dimension
    dp.o_part = static_cast<float*>(workspace);
    dp.lse_part = dp.o_part + (size_t)B * Hq * dp.n_chunks * 128;
    dp.scale_log2 = scale * k_scale * 1.4426950408889634f;   // the scores are q . (k_scale * k8)
    dp.block_table = block_table;
    dp.page_size = block_table ? page_size : 1;
    dp.table_stride = table_stride;
    dp.v_scale = v_scale;
    dp.Sq = 1;
    dp.bf16_io = bf16 ? 1 : 0;
    // one chunk per sequence: the split kernel writes O and LSE itself and no merge is launched
    const bool direct = Skv_max > 0 && dp.n_chunks == 1;
    dp.o_final = direct ? o : nullptr;
    dp.lse_final = direct ? lse : nullptr;
    const int g = Hq / Hkv;
    if (Skv_max > 0) {
        CUtensorMap tk, tv;
        const int slabs = block_table ? num_pages : B;          // outermost dimension: the sequence, or the page
        const int slab_rows = block_table ? page_size : Skv_max;
        const int box_rows = (block_table && page_size < fa::kDecTile) ? page_size : fa::kDecTile;
        rc = encode_map_u8(&tk, k_cache, slabs, slab_rows, Hkv, box_rows);
        if (rc) return rc;
        rc = encode_map_u8(&tv, v_cache, slabs, slab_rows, Hkv, box_rows);
        if (rc) return rc;
        constexpr int smem = 1024 + 2 * fa::kDec8Stages * fa::kDec8TileBytes;
        int sm_count = 0;
        // keys as the MMA's rows and up to 8 query heads as its columns (two column blocks for 9..16 heads)
        auto kern = (g > 8) ? fa::fa_decode_split_fp8_kernel<2> : fa::fa_decode_split_fp8_kernel<1>;
        if (int ce = fa::prepare_big_smem_kernel(reinterpret_cast<const void*>(kern), smem, &sm_count))
            return cuda_fail(static_cast<cudaError_t>(ce));
        dim3 grid(Hkv * ((g + 15) / 16), dp.n_chunks, B);
        kern<<<grid, fa::kDec8Threads, smem, st>>>(tk, tv, dp);
        cudaError_t e = cudaGetLastError();
        rc = e == cudaSuccess ? FA_OK : cuda_fail(e);
        if (rc) return rc;
    }
    if (direct) return FA_OK;
    cudaError_t e = bf16 ? launch_combine<__nv_bfloat16, 128>(dp, B * Hq, o, lse, st)
                         : launch_combine<__half, 128>(dp, B * Hq, o, lse, st);
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? FA_OK : cuda_fail(e);
}

int fa_decode_ex(const fa_decode_params* p, void* stream) {
    if (!p) return FA_ERR_NULL;
    if (p->dtype != FA_DTYPE_FP16 && p->dtype != FA_DTYPE_BF16) return FA_ERR_UNSUPPORTED;
    const int Sq = p->Sq > 0 ? p->Sq : 1;
    if (p->block_table) {
        if (p->num_pages < 0 || p->max_pages < 0 || !page_size_ok(p->page_size)) return FA_ERR_SHAPE;
        if (p->table_stride < p->max_pages) return FA_ERR_SHAPE;
        if ((long long)p->max_pages * p->page_size > 0x7fffffffll) return FA_ERR_SHAPE;
        if (p->max_pages > 0 && p->num_pages == 0) return FA_ERR_SHAPE;
        if (reinterpret_cast<uintptr_t>(p->block_table) & 3u) return FA_ERR_ALIGN;
        return decode_impl(p->q, p->k, p->v, p->o, p->lse, p->seqlens_k, p->B, p->Hq, p->Hkv, p->max_pages * p->page_size,
                           p->d, p->scale, p->workspace, p->workspace_bytes, stream, p->block_table, p->num_pages,
                           p->page_size, p->table_stride, Sq, p->dtype == FA_DTYPE_BF16);
    }
    return decode_impl(p->q, p->k, p->v, p->o, p->lse, p->seqlens_k, p->B, p->Hq, p->Hkv, p->Skv_max, p->d, p->scale,
                       p->workspace, p->workspace_bytes, stream, nullptr, 0, 0, 0, Sq, p->dtype == FA_DTYPE_BF16);
}

int fa_decode_append(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                     const int* seqlens_k, int B, int Sq, int Hq, int Hkv, int Skv_max, int d, float scale,
                     void* workspace, size_t workspace_bytes, void* stream) {
    return decode_impl(q, k_cache, v_cache, o, lse, seqlens_k, B, Hq, Hkv, Skv_max, d, scale, workspace,
                       workspace_bytes, stream, nullptr, 0, 0, 0, Sq);
}

int fa_decode_fp8(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse, const int* seqlens_k,
                  int B, int Hq, int Hkv, int Skv_max, int d, float scale, float k_scale, float v_scale,
                  void* workspace, size_t workspace_bytes, void* stream) {
    return decode_fp8_impl(q, k_cache, v_cache, o, lse, seqlens_k, B, Hq, Hkv, Skv_max, d, scale, k_scale, v_scale,
                           workspace, workspace_bytes, stream, nullptr, 0, 0, 0);
}

int fa_decode_fp8_bf16(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                       const int* seqlens_k, int B, int Hq, int Hkv, int Skv_max, int d, float scale, float k_scale,
                       float v_scale, void* workspace, size_t workspace_bytes, void* stream) {
    return decode_fp8_impl(q, k_cache, v_cache, o, lse, seqlens_k, B, Hq, Hkv, Skv_max, d, scale, k_scale, v_scale,
                           workspace, workspace_bytes, stream, nullptr, 0, 0, 0, true);
}

static int decode_fp8_paged_checked(bool bf16, const void* q, const void* k_pages, const void* v_pages, const int* block_table, void* o,
                        float* lse, const int* seqlens_k, int B, int Hq, int Hkv, int num_pages, int page_size,
                        int max_pages, int table_stride, int d, float scale, float k_scale, float v_scale,
                        void* workspace, size_t workspace_bytes, void* stream) {
    if (num_pages < 0 || max_pages < 0 || !page_size_ok(page_size)) return FA_ERR_SHAPE;
    if (table_stride < max_pages) return FA_ERR_SHAPE;
    if ((long long)max_pages * page_size > 0x7fffffffll) return FA_ERR_SHAPE;
    if (B > 0 && max_pages > 0 && !block_table) return FA_ERR_NULL;
    if (max_pages > 0 && num_pages == 0) return FA_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(block_table) & 3u) return FA_ERR_ALIGN;
    return decode_fp8_impl(q, k_pages, v_pages, o, lse, seqlens_k, B, Hq, Hkv, max_pages * page_size, d, scale, k_scale,
                           v_scale, workspace, workspace_bytes, stream, block_table, num_pages, page_size, table_stride, bf16);
}

int fa_decode_fp8_paged(const void* q, const void* k_pages, const void* v_pages, const int* block_table, void* o,
                        float* lse, const int* seqlens_k, int B, int Hq, int Hkv, int num_pages, int page_size,
                        int max_pages, int table_stride, int d, float scale, float k_scale, float v_scale,
                        void* workspace, size_t workspace_bytes, void* stream) {
    return decode_fp8_paged_checked(false, q, k_pages, v_pages, block_table, o, lse, seqlens_k, B, Hq, Hkv, num_pages,
                                    page_size, max_pages, table_stride, d, scale, k_scale, v_scale, workspace,
                                    workspace_bytes, stream);
}

int fa_decode_fp8_paged_bf16(const void* q, const void* k_pages, const void* v_pages, const int* block_table, void* o,
                             float* lse, const int* seqlens_k, int B, int Hq, int Hkv, int num_pages, int page_size,
                             int max_pages, int table_stride, int d, float scale, float k_scale, float v_scale,
                             void* workspace, size_t workspace_bytes, void* stream) {
    return decode_fp8_paged_checked(true, q, k_pages, v_pages, block_table, o, lse, seqlens_k, B, Hq, Hkv, num_pages,
                                    page_size, max_pages, table_stride, d, scale, k_scale, v_scale, workspace,
                                    workspace_bytes, stream);
}

int fa_decode_paged(const void* q, const void* k_pages, const void* v_pages, const int* block_table, void* o,
                    float* lse, const int* seqlens_k, int B, int Hq, int Hkv, int num_pages, int page_size,
                    int max_pages, int table_stride, int d, float scale, void* workspace, size_t workspace_bytes,
                    void* stream) {
    if (num_pages < 0 || max_pages < 0 || !page_size_ok(page_size)) return FA_ERR_SHAPE;
    if (table_stride < max_pages) return FA_ERR_SHAPE;
    if ((long long)max_pages * page_size > 0x7fffffffll) return FA_ERR_SHAPE;
    if (B > 0 && max_pages > 0 && !block_table) return FA_ERR_NULL;
    if (max_pages > 0 && num_pages == 0) return FA_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(block_table) & 3u) return FA_ERR_ALIGN;
    return decode_impl(q, k_pages, v_pages, o, lse, seqlens_k, B, Hq, Hkv, max_pages * page_size, d, scale, workspace,
                       workspace_bytes, stream, block_table, num_pages, page_size, table_stride);
}

// ---- decode without a caller workspace -------------------------------------------------------
// Scratch for the per-chunk partials of fa_decode_noalloc.  It is part of the device image, so
// every GPU that loads the library holds it until exit.  In host code the name below is only a
// host-side stand-in for the device array; the device address is looked up once per device.
static __device__ __align__(256) unsigned char g_decode_scratch[FA_DECODE_NOALLOC_BYTES];

int fa_decode_noalloc(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                      const int* seqlens_k, int B, int Hq, int Hkv, int Skv_max, int d, float scale,
                      void* stream) {
    // every argument check of fa_decode first, with the same codes in the same order, then the size
    // limit of the fixed scratch: nothing CUDA-related happens for a call that is going to be refused
    int rc = decode_check_args(q, k_cache, v_cache, o, seqlens_k, B, Hq, Hkv, Skv_max, d, scale, 1);
    if (rc) return rc;
    if (B == 0) return FA_OK;
    if (fa_decode_workspace_bytes(B, Hq, Hkv, Skv_max, d) > (size_t)FA_DECODE_NOALLOC_BYTES)
        return FA_ERR_WORKSPACE;
    rc = check_device();   // a GPU this library has no code for is FA_ERR_DEVICE, not a failed symbol lookup
    if (rc) return rc;
    constexpr int kMaxDevices = 64;
    static void* scratch_of_device[kMaxDevices] = {nullptr};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return FA_ERR_DEVICE;
    void* scratch = __atomic_load_n(&scratch_of_device[dev], __ATOMIC_ACQUIRE);
    if (!scratch) {
        // set-up, once per device, with that device current (it is: we just asked which one)
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_decode_scratch);
        if (e != cudaSuccess) return cuda_fail(e);
        if (!ptr) return FA_ERR_DEVICE;
        __atomic_store_n(&scratch_of_device[dev], ptr, __ATOMIC_RELEASE);  // same value from any thread
        scratch = ptr;
    }
    return fa_decode(q, k_cache, v_cache, o, lse, seqlens_k, B, Hq, Hkv, Skv_max, d, scale, scratch,
                     (size_t)FA_DECODE_NOALLOC_BYTES, stream);
}

size_t fa_forward_host_staging_bytes(int B, int Hq, int Hkv, int Sq, int Skv, int d) {
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Skv < 0 || (d != 64 && d != 128 && d != 256)) return 0;
    auto up = [](size_t x) { return (x + 1023) & ~(size_t)1023; };
    const size_t qo = up((size_t)B * Sq * Hq * d * 2);
    const size_t kv = up((size_t)B * Skv * Hkv * d * 2);
    const size_t l = up((size_t)B * Hq * Sq * 4);
    return 2 * qo + 2 * kv + l;
}

int fa_forward_host(const void* q_host, const void* k_host, const void* v_host, void* o_host, float* lse_host,
                    int B, int Hq, int Hkv, int Sq, int Skv, int d, int causal, float scale, int dtype,
                    void* staging, size_t staging_bytes, void* stream) {
    if (B < 0 || Hq <= 0 || Hkv <= 0 || Sq < 0 || Skv < 0 || d <= 0) return FA_ERR_SHAPE;
    if (d != 64 && d != 128 && d != 256) return FA_ERR_UNSUPPORTED;   // the head dimensions fa_forward takes
    if (dtype != FA_DTYPE_FP16 && dtype != FA_DTYPE_BF16) return FA_ERR_UNSUPPORTED;
    if (B == 0 || Sq == 0) return FA_OK;
    if (!q_host || !o_host || (Skv > 0 && (!k_host || !v_host))) return FA_ERR_NULL;
    const size_t need = fa_forward_host_staging_bytes(B, Hq, Hkv, Sq, Skv, d);
    if (!staging || staging_bytes < need) return FA_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(staging) & 1023u) return FA_ERR_ALIGN;
    auto up = [](size_t x) { return (x + 1023) & ~(size_t)1023; };
    const size_t qo_b = (size_t)B * Sq * Hq * d * 2, kv_b = (size_t)B * Skv * Hkv * d * 2;
    char* base = static_cast<char*>(staging);
    char* dq = base;
    char* dk = dq + up(qo_b);
    char* dv = dk + up(kv_b);
    char* dout = dv + up(kv_b);
    char* dl = dout + up(qo_b);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    // The batch is cut into up to four parts, and the three stages of a part -- copy in, forward,
    // copy out -- run on three streams (the caller's for the forward, two of the library's own for
    // the copies), chained by events: the copy engines of both directions and the SMs then work
    // at the same time on different parts.  Everything is ordered after the work already on
    // `stream`, and `stream` waits for the last copy out.
    HostPipe* hp = host_pipe();
    if (!hp) return FA_ERR_CUDA;
    std::lock_guard<std::mutex> enqueue_lock(hp->enqueue);
    const int parts = B < kHostParts ? B : kHostParts;
    if ((e = cudaEventRecord(hp->start, st)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamWaitEvent(hp->in, hp->start, 0)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamWaitEvent(hp->out, hp->start, 0)) != cudaSuccess) return cuda_fail(e);
    const size_t q1 = (size_t)Sq * Hq * d * 2, kv1 = (size_t)Skv * Hkv * d * 2, l1 = (size_t)Hq * Sq * 4;
    for (int c = 0; c < parts; ++c) {
        const int b0 = (int)((long long)B * c / parts), b1 = (int)((long long)B * (c + 1) / parts);
        const size_t nb = (size_t)(b1 - b0);
        if ((e = cudaMemcpyAsync(dq + b0 * q1, static_cast<const char*>(q_host) + b0 * q1, nb * q1,
                                 cudaMemcpyHostToDevice, hp->in)) != cudaSuccess) return cuda_fail(e);
        if (kv1) {
            if ((e = cudaMemcpyAsync(dk + b0 * kv1, static_cast<const char*>(k_host) + b0 * kv1, nb * kv1,
                                     cudaMemcpyHostToDevice, hp->in)) != cudaSuccess) return cuda_fail(e);
            if ((e = cudaMemcpyAsync(dv + b0 * kv1, static_cast<const char*>(v_host) + b0 * kv1, nb * kv1,
                                     cudaMemcpyHostToDevice, hp->in)) != cudaSuccess) return cuda_fail(e);
        }
        if ((e = cudaEventRecord(hp->in_done[c], hp->in)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(st, hp->in_done[c], 0)) != cudaSuccess) return cuda_fail(e);
        int rc = forward_plain(dq + b0 * q1, dk + b0 * kv1, dv + b0 * kv1, dout + b0 * q1,
                               reinterpret_cast<float*>(dl + b0 * l1), (int)nb, Hq, Hkv, Sq, Skv, d, causal, scale,
                               dtype, stream);
        if (rc) return rc;
        if ((e = cudaEventRecord(hp->fwd_done[c], st)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaStreamWaitEvent(hp->out, hp->fwd_done[c], 0)) != cudaSuccess) return cuda_fail(e);
        if ((e = cudaMemcpyAsync(static_cast<char*>(o_host) + b0 * q1, dout + b0 * q1, nb * q1, cudaMemcpyDeviceToHost,
                                 hp->out)) != cudaSuccess) return cuda_fail(e);
        if (lse_host)
            if ((e = cudaMemcpyAsync(reinterpret_cast<char*>(lse_host) + b0 * l1, dl + b0 * l1, nb * l1,
                                     cudaMemcpyDeviceToHost, hp->out)) != cudaSuccess) return cuda_fail(e);
    }
    if ((e = cudaEventRecord(hp->finish, hp->out)) != cudaSuccess) return cuda_fail(e);
    if ((e = cudaStreamWaitEvent(st, hp->finish, 0)) != cudaSuccess) return cuda_fail(e);
    return FA_OK;
}

int fa_device_status(unsigned int detail[2]) {
    unsigned int h[4] = {0, 0, 0, 0};
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e);
    e = cudaMemcpyFromSymbol(h, fa::g_status, sizeof h);
    if (e != cudaSuccess) return cuda_fail(e);
    if (h[0] == 0) return FA_OK;
    if (detail) {
        detail[0] = h[1];
        detail[1] = h[2];
    }
    unsigned int z[4] = {0, 0, 0, 0};
    e = cudaMemcpyToSymbol(fa::g_status, z, sizeof z);
    if (e != cudaSuccess) return cuda_fail(e);
    return FA_ERR_TIMEOUT;
}

int fa_selftest_wait(unsigned int limit_us, unsigned int* gave_up, void* stream) {
    if (!gave_up) return FA_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(gave_up) & 3u) return FA_ERR_ALIGN;
    if (limit_us == 0 || limit_us > 100000u) return FA_ERR_UNSUPPORTED;   // at most a tenth of a second
    int rc = check_device();
    if (rc) return rc;
    fa::fa_selftest_wait_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(1000ull * limit_us, gave_up);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? FA_OK : cuda_fail(e);
}

const char* fa_strerror(int code) {
    switch (code) {
        case FA_OK: return "ok";
        case FA_ERR_NULL: return "a required pointer is NULL";
        case FA_ERR_SHAPE: return "invalid shape or stride";
        case FA_ERR_UNSUPPORTED: return "unsupported configuration";
        case FA_ERR_ALIGN: return "pointer not sufficiently aligned";
        case FA_ERR_WORKSPACE: return "workspace missing or too small";
        case FA_ERR_DEVICE: return "device is not compute capability 10.x or no driver";
        case FA_ERR_CUDA: return "CUDA call failed (see fa_last_cuda_error)";
        case FA_ERR_TIMEOUT: return "a bounded device-side wait expired";
        default: return "unknown error code";
    }
}

int fa_version(void) { return 100; }

int fa_last_cuda_error(void) { return t_last_cuda_error; }

}  // extern "C"
