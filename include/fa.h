/*
 * fa.h -- C ABI of the B200 (sm_100a) fused attention forward library.
 *
 * The library computes, for every batch b, query head h and query row i,
 *
 *     O[b,i,h,:] = sum_j softmax_j( scale * <Q[b,i,h,:], K[b,j,hk,:]> + mask(i,j) ) * V[b,j,hk,:]
 *     LSE[b,h,i] = ln sum_j exp( scale * <Q[b,i,h,:], K[b,j,hk,:]> + mask(i,j) )
 *
 * i.e. the paper's attention operator Softmax(Q K^T / sqrt(d)) V (Section 5.1), evaluated
 * with the FlashAttention2-style fused, blocked, online-softmax method the paper builds on
 * (Section 4.1; Appendix A: per block Q*K^T, Exp, Exp*V, update of rowmax/rowsum), so that
 * neither the score matrix nor the attention_mask is ever stored (Section 4.1, tiling-mask:
 * the mask is lower triangular; fully masked blocks are skipped, fully visible blocks are
 * not masked).  The decode entry point evaluates the decode-stage form of Appendix C
 * (one query row per sequence over the cached keys and values).
 *
 * Conventions shared by every entry point
 *   - All q/k/v/o/lse/seqlens/workspace pointers are DEVICE pointers owned by the caller,
 *     unless an argument is explicitly named *_host.  The library never allocates or frees
 *     device memory and never keeps a pointer after the call returns.
 *   - Layout: q and o are [B, Sq, Hq, d], k and v are [B, Skv, Hkv, d], d contiguous
 *     (the paper's B*S*N*D layout, Section 4.2).  lse is [B, Hq, Sq] float, natural log.
 *   - Head mapping: query head h reads kv head h / (Hq / Hkv); Hq % Hkv must be 0.
 *   - causal != 0 applies the lower-triangular mask aligned to the last key:
 *     row i sees key j iff j <= i + (Skv - Sq).
 *   - scale is used as given (callers pass 1/sqrt(d)).
 *   - stream is a cudaStream_t passed as void*.  Calls only enqueue work on it; they do
 *     not synchronise.  Two calls that write the same buffers must be ordered by the caller.
 *   - Return value: FA_OK or a negative FA_ERR_* code.  Arguments are validated before any
 *     CUDA call; on a validation error nothing has been enqueued.  No entry point throws,
 *     aborts or traps.
 *   - Device-side waits are bounded.  If one ever expires the kernel records it in a status
 *     word, drains and returns; fa_device_status() reports it after the stream is idle.
 */
#ifndef FA_H_
#define FA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FA_OK 0
#define FA_ERR_NULL (-1)        /* a required pointer is NULL                                 */
#define FA_ERR_SHAPE (-2)       /* negative dims, Hq % Hkv != 0, bad stride                  */
#define FA_ERR_UNSUPPORTED (-3) /* head dimension, causal with Sq > Skv, unknown dtype        */
#define FA_ERR_ALIGN (-4)       /* a pointer or stride is not 16-byte aligned                */
#define FA_ERR_WORKSPACE (-5)   /* workspace missing or too small                            */
#define FA_ERR_DEVICE (-6)      /* current device is not compute capability 10.x             */
#define FA_ERR_CUDA (-7)        /* a CUDA call failed; see fa_last_cuda_error()              */
#define FA_ERR_TIMEOUT (-8)     /* a bounded device-side wait expired (fa_device_status)     */

#define FA_DTYPE_FP16 0
#define FA_DTYPE_BF16 1
#define FA_DTYPE_FP32 2 /* only as fa_params.o_dtype */

/*
 * Prefill / general forward, fp16 inputs and output (Section 5.1 operator; Section 4.1 method).
 *   q [B,Sq,Hq,d], k,v [B,Skv,Hkv,d], o [B,Sq,Hq,d] fp16, contiguous; lse [B,Hq,Sq] float or NULL.
 *   d must be 128, 64 (the short vision workload of the evaluation section) or 256; 64 and 256
 *   have kernels of their own and are taken by fa_forward, fa_forward_bf16, fa_forward_host and
 *   fa_forward_ex (variant 0; d = 64 also variant 3).  The packed-batch and the 16-bit decode
 *   entry points take 128 and 64; the 8-bit and projection entry points want 128.
 *   B == 0 or Sq == 0 is a successful no-op.  Skv == 0 gives O = 0, LSE = -inf.
 *   o and lse must not alias the inputs.
 */
int fa_forward(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq,
               int Hkv, int Sq, int Skv, int d, int causal, float scale, void* stream);

/* Same operation with bfloat16 inputs and output. */
int fa_forward_bf16(const void* q, const void* k, const void* v, void* o, float* lse, int B,
                    int Hq, int Hkv, int Sq, int Skv, int d, int causal, float scale,
                    void* stream);

/*
 * Extended form: explicit element strides (batch, sequence, head; d is contiguous) so that
 * [B,H,S,d] storage can be passed too, and a choice of output type (the input type, or
 * FA_DTYPE_FP32 to read the fp32 accumulator without the final 16-bit rounding).
 * A stride of 0 means "contiguous [B,S,H,d]".  Strides must be multiples of 8 elements.
 */
typedef struct fa_params {
    const void* q;
    const void* k;
    const void* v;
    void* o;
    float* lse; /* may be NULL */
    int B, Hq, Hkv, Sq, Skv, d;
    int causal;
    float scale;
    int dtype;   /* FA_DTYPE_FP16 or FA_DTYPE_BF16: type of q, k, v */
    int o_dtype; /* same as dtype, or FA_DTYPE_FP32 */
    int64_t q_stride[3]; /* batch, sequence, head -- in elements */
    int64_t k_stride[3];
    int64_t v_stride[3];
    int64_t o_stride[3];
    int variant; /* 0 = default: the ping-pong kernel when Skv >= 1024, else the paired-tile pipelined
                    kernel.  Others force one kernel, for A/B timing and tests: 1, 2 = simple kernels
                    (P through tensor / shared memory), 3 = ping-pong, 4 = paired-tile pipelined. */
} fa_params;

int fa_forward_ex(const fa_params* p, void* stream);

/*
 * Forward with 8-bit operands (Appendix D.2 evaluates the operator with 8-bit operands; the paper
 * names no format, scales or granularity, so this is the reading taken here): the computation of
 * fa_forward with Q = q_scale * q, K = k_scale * k, V = v_scale * v, where q [B,Sq,Hq,d] and
 * k, v [B,Skv,Hkv,d] hold FP8 e4m3 bit patterns (1 sign, 4 exponent, 3 mantissa bits, bias 7, no
 * infinities; one byte per element, contiguous, 16-byte aligned) and the three factors are
 * positive and finite, one per tensor.  Both products run on the tensor cores with 8-bit
 * operands and fp32 accumulation; for the second one the probabilities are rounded to e4m3 as
 * well (after a fixed power-of-two factor that is divided out again), which is the one place
 * where this entry point is less accurate than the 16-bit ones: a probability carries a relative
 * rounding of up to 2^-4, so O_i moves by up to 2^-4 * sum_j P_ij |V_j| (plus a much smaller
 * absolute term from probabilities below the format's normal range).  LSE is computed from the
 * unrounded probabilities and is as accurate as fa_forward's.
 *   o [B,Sq,Hq,d] of o_dtype (FA_DTYPE_FP16 or FA_DTYPE_BF16), lse [B,Hq,Sq] float or NULL;
 *   d must be 128.  Everything else (mask, head mapping, no-ops, aliasing) as for fa_forward.
 *   No NaN pattern (0x7f, 0xff) may occur in q, k, v.
 * Errors: as fa_forward; FA_ERR_UNSUPPORTED also for a factor that is not positive and finite
 * and for an o_dtype other than the two 16-bit types.
 */
int fa_forward_fp8(const void* q, const void* k, const void* v, void* o, float* lse, int B, int Hq,
                   int Hkv, int Sq, int Skv, int d, int causal, float scale, float q_scale,
                   float k_scale, float v_scale, int o_dtype, void* stream);

/*
 * Attention followed by the output projection (Section 4.2 fuses the attention kernel with the
 * Linear that follows it; Appendix C writes the projection as the decoder layer's last step of
 * attention).  On one GPU there is no collective behind the Linear, so this is that fused kernel
 * without its AllReduce:
 *     O   = fa_forward(q, k, v)                       [B, Sq, Hq, d], also returned
 *     out = O viewed as [B, Sq, Hq * d]  times  w_o   [B, Sq, d_model]
 * with w_o [Hq * d, d_model] row-major (d_model contiguous), all in the 16-bit type `dtype`, fp32
 * accumulation in both products, O rounded to 16 bits between them.
 *   fused != 0: ONE launch.  The attention phase is the ping-pong kernel of fa_forward; a CTA that
 *   has finished its attention items goes on to 128 x 256 blocks of the projection, each as soon as
 *   the attention output of every head for its 128 query rows has reached global memory (a counter
 *   per row block in `workspace`, which the call zeroes; the wait on it is bounded like every
 *   other).  The launch is cooperative: it fails with FA_ERR_CUDA rather than start if the GPU
 *   cannot hold the whole grid at once.
 *   fused == 0: the same two kernels as two launches on `stream` (no workspace needed).
 *   d must be 128, d_model a multiple of 256; out 32-byte aligned; workspace of at least
 *   fa_forward_proj_workspace_bytes(B, Sq) bytes, 4-byte aligned.  lse may be NULL.
 * Errors: as fa_forward; FA_ERR_UNSUPPORTED also for other d_model, FA_ERR_WORKSPACE for a missing
 * or short workspace with fused != 0.
 */
int fa_forward_proj(const void* q, const void* k, const void* v, const void* w_o, void* o, float* lse,
                    void* out, int B, int Hq, int Hkv, int Sq, int Skv, int d, int d_model, int causal,
                    float scale, int dtype, int fused, void* workspace, size_t workspace_bytes,
                    void* stream);

size_t fa_forward_proj_workspace_bytes(int B, int Sq);

/*
 * Forward over a packed batch of sequences of different lengths (the batched serving runs of the
 * evaluation section process requests of unequal length together): the same computation as
 * fa_forward, sequence by sequence.  Sequence b owns rows [cu_seqlens_q[b], cu_seqlens_q[b+1])
 * of q and o and rows [cu_seqlens_k[b], cu_seqlens_k[b+1]) of k and v; with the causal mask its
 * diagonal is aligned bottom-right, as in fa_forward, sequence by sequence.
 *   q, o [total_q, Hq, d]; k, v [total_k, Hkv, d], d = 128 or 64, contiguous, 16-byte aligned,
 *   dtype as given (FA_DTYPE_FP16 or FA_DTYPE_BF16; o has the same type); lse [Hq, total_q] float or NULL;
 *   cu_seqlens_q, cu_seqlens_k: int32 [B + 1] on the DEVICE, non-decreasing, first entry 0, last
 *   entry total_q / total_k; max_seqlen_q / max_seqlen_k: upper bounds of the sequence lengths
 *   (they size the launch: a longer sequence would be cut off at the bound).
 *   A sequence without keys, and under the causal mask every row that sees no key (a sequence
 *   with more queries than keys), gives O = 0 and LSE = -inf.  The prefix sums are read by the
 *   kernel only and are not validated.  K and V rows of the NEXT sequence may be loaded, but they
 *   never reach a result (their scores are masked and their V rows are cleared on chip).
 * Errors: as fa_forward; FA_ERR_SHAPE also for max_seqlen_q > total_q or max_seqlen_k > total_k.
 */
int fa_forward_varlen(const void* q, const void* k, const void* v, void* o, float* lse,
                      const int* cu_seqlens_q, const int* cu_seqlens_k, int B, int Hq, int Hkv, int total_q,
                      int total_k, int max_seqlen_q, int max_seqlen_k, int d, int causal, float scale,
                      int dtype, void* stream);

/*
 * Decode stage (Appendix C): one query row per sequence over that sequence's cached keys
 * and values, split along the cache into chunks whose partial results (fp32 O and LSE) are
 * merged by a second kernel with the same rowmax/rowsum recurrence (Appendix A) applied
 * across chunks.
 *   q [B,1,Hq,d] fp16, k_cache,v_cache [B,Skv_max,Hkv,d] fp16, o [B,1,Hq,d] fp16,
 *   lse [B,Hq] float or NULL, seqlens_k [B] int32 on the DEVICE: only the first
 *   seqlens_k[b] cache rows of sequence b are read; rows beyond may hold anything (NaN too).
 *   A sequence with seqlens_k[b] == 0 gives O = 0 and LSE = -inf.  Values of seqlens_k
 *   outside [0, Skv_max] are clamped.
 *   workspace: at least fa_decode_workspace_bytes(...) bytes, 16-byte aligned, contents
 *   need no initialisation and are overwritten.
 *   d is 128 or 64 (FA_ERR_UNSUPPORTED otherwise; fa_decode_workspace_bytes then returns 0); the
 *   same holds for fa_decode_paged, fa_decode_append, fa_decode_ex and fa_decode_noalloc, which
 *   run the same kernel.  The 8-bit cache forms (fa_decode_fp8...) take d = 128 only.
 *   Skv_max may not exceed 65535 chunks of the cache split (chunks are 256 to 4096 keys long, so
 *   16 million keys always fit; FA_ERR_UNSUPPORTED beyond).
 */
int fa_decode(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
              const int* seqlens_k, int B, int Hq, int Hkv, int Skv_max, int d, float scale,
              void* workspace, size_t workspace_bytes, void* stream);

size_t fa_decode_workspace_bytes(int B, int Hq, int Hkv, int Skv_max, int d);

/*
 * fa_forward_varlen over a paged K/V cache (chunked prefill of a batch of requests whose
 * earlier keys already sit in a serving system's page pool): q, o, lse, cu_seqlens_q as for
 * fa_forward_varlen; sequence b has seqlens_k[b] keys (int32 [B] on the DEVICE), key j in row
 * j mod page_size of page block_table[b * table_stride + j / page_size] of the pools k_pages,
 * v_pages [num_pages, page_size, Hkv, d]; page_size a positive multiple of 128; max_seqlen_k an
 * upper bound of seqlens_k, at most max_pages * page_size.  The causal mask is aligned
 * bottom-right per sequence (the queries are the sequence's LAST rows).  Only the table entries
 * that cover keys [0, seqlens_k[b]) are used; the first entry of every sequence's row is always
 * read (it exists: table_stride >= 1) and ignored when the sequence has no keys.  Rows of a page
 * past the end of its sequence, and unused pages, may hold anything (NaN too).
 * Errors: as fa_forward_varlen; FA_ERR_SHAPE also for a page_size that is not a multiple of 128,
 * table_stride < max_pages or max_seqlen_k > max_pages * page_size.
 */
int fa_forward_varlen_paged(const void* q, const void* k_pages, const void* v_pages, const int* block_table,
                            void* o, float* lse, const int* cu_seqlens_q, const int* seqlens_k, int B, int Hq,
                            int Hkv, int total_q, int num_pages, int page_size, int max_pages, int table_stride,
                            int max_seqlen_q, int max_seqlen_k, int d, int causal, float scale, int dtype,
                            void* stream);

/*
 * The general form of the 16-bit decode: fp16 or bf16 (q, caches and o share the type), one or
 * several query rows per sequence (Sq <= 0 means 1; see fa_decode_append), contiguous cache
 * (block_table == NULL: k, v [B,Skv_max,Hkv,d]) or paged (k, v [num_pages,page_size,Hkv,d];
 * Skv_max is then ignored and max_pages * page_size takes its place; see fa_decode_paged).
 * workspace: fa_decode_append_workspace_bytes(B, Sq, Hq, Hkv, Skv_max or max_pages * page_size, d).
 * Everything else as documented for fa_decode, fa_decode_append and fa_decode_paged.
 */
typedef struct fa_decode_params {
    const void* q;          /* [B,Sq,Hq,d] */
    const void* k;          /* cache or page pool */
    const void* v;
    void* o;                /* [B,Sq,Hq,d] */
    float* lse;             /* [B,Hq,Sq] or NULL */
    const int* seqlens_k;   /* [B], device */
    const int* block_table; /* NULL, or [B,table_stride] on the device */
    int B, Sq, Hq, Hkv, Skv_max, d;
    int dtype;              /* FA_DTYPE_FP16 or FA_DTYPE_BF16 */
    int num_pages, page_size, max_pages, table_stride;
    float scale;
    void* workspace;
    size_t workspace_bytes;
} fa_decode_params;
int fa_decode_ex(const fa_decode_params* p, void* stream);

/*
 * Decode after several tokens were appended (Appendix C with Sq > 1 new tokens per sequence, as
 * in chunked or speculative decoding): the Sq query rows of sequence b are the LAST Sq positions
 * of its cache, so query t (0 <= t < Sq) sees the keys 0 .. seqlens_k[b] - Sq + t -- the
 * bottom-right aligned causal mask of fa_forward, computed by the split-KV decode kernels
 * instead of the prefill kernel, which for a few query rows over a long cache would leave
 * most of the GPU idle.
 *   q, o [B,Sq,Hq,d] fp16 contiguous, lse [B,Hq,Sq] float or NULL; 1 <= Sq <= 64; caches,
 *   seqlens_k (the lengths INCLUDING the Sq new tokens), scale, stream as for fa_decode.
 *   A query that sees no key (seqlens_k[b] < Sq - t) gives O = 0 and LSE = -inf.
 *   workspace: at least fa_decode_append_workspace_bytes(...) bytes, 16-byte aligned.
 * Errors: as fa_decode; FA_ERR_UNSUPPORTED also for Sq > 64 or Sq > Skv_max.
 */
int fa_decode_append(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                     const int* seqlens_k, int B, int Sq, int Hq, int Hkv, int Skv_max, int d, float scale,
                     void* workspace, size_t workspace_bytes, void* stream);

size_t fa_decode_append_workspace_bytes(int B, int Sq, int Hq, int Hkv, int Skv_max, int d);

/*
 * Decode over an 8-bit cache (Appendix D.2 evaluates the operator with 8-bit operands; in the
 * decode stage the cache dominates the traffic, so here it is the cached K and V that are 8-bit):
 * the computation of fa_decode with K = k_scale * k_cache and V = v_scale * v_cache, where
 * k_cache and v_cache [B,Skv_max,Hkv,d] hold FP8 e4m3 bit patterns (1 sign, 4 exponent, 3
 * mantissa bits, bias 7, no infinities; one byte per element, contiguous, 16-byte aligned) and
 * k_scale, v_scale are positive finite factors for the whole tensor.  q and o are fp16 and the
 * probabilities are rounded to fp16 as in fa_decode; the widened cache values are exact in fp16.
 * Rows beyond seqlens_k[b] may hold anything (the NaN patterns 0x7f / 0xff too).
 * Everything else (lse, seqlens_k, workspace size and alignment, errors) as for fa_decode;
 * FA_ERR_UNSUPPORTED also for a scale that is not positive and finite.
 */
int fa_decode_fp8(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                  const int* seqlens_k, int B, int Hq, int Hkv, int Skv_max, int d, float scale,
                  float k_scale, float v_scale, void* workspace, size_t workspace_bytes, void* stream);

/* fa_decode_fp8 with q and o in bf16 (the models of the evaluation section run in either 16-bit
 * type; the 8-bit cache is the same).  The products still run in fp16, the type the cache bytes
 * widen to exactly: q is converted on load, which is exact for magnitudes in fp16's normal range
 * (6.1e-5 to 65504; larger ones become infinities), the probabilities are rounded to fp16, and o
 * is rounded to bf16 when it is stored.  Everything else as for fa_decode_fp8. */
int fa_decode_fp8_bf16(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                       const int* seqlens_k, int B, int Hq, int Hkv, int Skv_max, int d, float scale,
                       float k_scale, float v_scale, void* workspace, size_t workspace_bytes, void* stream);

/* fa_decode_fp8 over a paged cache: k_pages, v_pages [num_pages, page_size, Hkv, d] of e4m3 bytes;
 * block_table, page_size, max_pages, table_stride as for fa_decode_paged, scales as for fa_decode_fp8. */
int fa_decode_fp8_paged(const void* q, const void* k_pages, const void* v_pages, const int* block_table,
                        void* o, float* lse, const int* seqlens_k, int B, int Hq, int Hkv, int num_pages,
                        int page_size, int max_pages, int table_stride, int d, float scale, float k_scale,
                        float v_scale, void* workspace, size_t workspace_bytes, void* stream);

/* fa_decode_fp8_paged with q and o in bf16 (see fa_decode_fp8_bf16). */
int fa_decode_fp8_paged_bf16(const void* q, const void* k_pages, const void* v_pages, const int* block_table,
                             void* o, float* lse, const int* seqlens_k, int B, int Hq, int Hkv, int num_pages,
                             int page_size, int max_pages, int table_stride, int d, float scale, float k_scale,
                             float v_scale, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Decode over a paged cache: the same computation as fa_decode (Appendix C), with the cached
 * keys and values of a sequence scattered over fixed-size pages of a pool shared by all
 * sequences, as serving systems keep them for batched decoding (the batch 8/16 serving runs of
 * the evaluation section).  Key j of sequence b is row (j mod page_size) of page
 * block_table[b * table_stride + j / page_size].
 *   k_pages, v_pages [num_pages, page_size, Hkv, d] fp16 on the device, 16-byte aligned;
 *   page_size a positive multiple of 128, or 16, 32 or 64 (a 128-key tile is then one box of a
 *   page or several whole pages; other sizes are refused);
 *   block_table int32 on the DEVICE, table_stride >= max_pages entries per sequence; only the
 *   entries that cover keys [0, seqlens_k[b]) are read and they must lie in [0, num_pages)
 *   (a page index outside that range reads as zeros and never faults); rows of a page past the
 *   end of its sequence may hold anything (NaN too);
 *   seqlens_k [B] int32 on the DEVICE, clamped to [0, max_pages * page_size];
 *   q, o, lse, scale, stream as for fa_decode; workspace of at least
 *   fa_decode_workspace_bytes(B, Hq, Hkv, max_pages * page_size, d) bytes.
 * Errors: FA_ERR_SHAPE for a page_size other than those or table_stride < max_pages;
 * otherwise as fa_decode.
 */
int fa_decode_paged(const void* q, const void* k_pages, const void* v_pages, const int* block_table,
                    void* o, float* lse, const int* seqlens_k, int B, int Hq, int Hkv, int num_pages,
                    int page_size, int max_pages, int table_stride, int d, float scale, void* workspace,
                    size_t workspace_bytes, void* stream);

/*
 * Decode for callers that cannot allocate device memory (the paper has no counterpart; this is a
 * convenience of this library).  Some hosts of this code may not call cudaMalloc at all: code
 * running inside a framework that owns the memory pool and forbids outside allocations, a
 * real-time serving loop that must not take the allocator's locks or risk an out-of-memory
 * failure mid-request, or a plugin that is handed buffers and nothing else.  They still pass
 * q, the caches, o, lse and seqlens_k exactly as for fa_decode, but no workspace: the per-chunk
 * partial results go to a fixed array that lives inside the library's device image
 * (FA_DECODE_NOALLOC_BYTES bytes, held by every GPU that loads the library until the process
 * exits).
 *   - The call fails with FA_ERR_WORKSPACE, before any CUDA work, when
 *     fa_decode_workspace_bytes(B, Hq, Hkv, Skv_max, d) exceeds FA_DECODE_NOALLOC_BYTES.
 *   - The first call on each device looks the array's device address up (once per device, with
 *     that device current); make that first call before starting any stream capture.
 *   - No entry of the array needs to start at zero: every slot the merge reads is written by
 *     the same call first.  All calls share the one array, so two calls whose kernels may
 *     overlap on the GPU (different streams, no ordering between them) race on it; order them.
 *   - The function itself allocates nothing: no cudaMalloc, cudaFree or allocating library call.
 * Results are bit-identical to fa_decode's for the same arguments, and so are the argument checks
 * and their error codes (they run before the size limit is looked at and before any CUDA call).
 */
#define FA_DECODE_NOALLOC_BYTES (4u << 20)
int fa_decode_noalloc(const void* q, const void* k_cache, const void* v_cache, void* o, float* lse,
                      const int* seqlens_k, int B, int Hq, int Hkv, int Skv_max, int d, float scale,
                      void* stream);

/*
 * Host-buffer form of fa_forward for callers whose tensors live in host memory (pinned memory
 * makes the copies asynchronous): copies q, k, v to the device staging area, runs the forward,
 * copies o and lse back.  dtype is FA_DTYPE_FP16 or FA_DTYPE_BF16; d is 64, 128 or 256, as for
 * fa_forward (FA_ERR_UNSUPPORTED otherwise, and fa_forward_host_staging_bytes then returns 0).
 * staging is a DEVICE buffer of at least fa_forward_host_staging_bytes(...) bytes, 1024-byte
 * aligned, owned by the caller.  The call is ordered after the work already on `stream`, and the
 * results are in o_host / lse_host once `stream` is idle.  Inside, the batch is cut into up to
 * four parts whose copy-in, forward and copy-out stages overlap: the forward runs on `stream`,
 * the copies on two streams the library creates once per device (with a handful of events) and
 * keeps; nothing else is created and no device memory is allocated.  Make the first call on a
 * device outside stream capture.  Calls that share a staging buffer must be issued on the same
 * stream.  Host threads may call concurrently on one device with staging buffers and streams of
 * their own: the enqueue sequence of a call is serialised inside the library.
 */
int fa_forward_host(const void* q_host, const void* k_host, const void* v_host, void* o_host,
                    float* lse_host, int B, int Hq, int Hkv, int Sq, int Skv, int d, int causal,
                    float scale, int dtype, void* staging, size_t staging_bytes, void* stream);

size_t fa_forward_host_staging_bytes(int B, int Hq, int Hkv, int Sq, int Skv, int d);

/*
 * Reads and clears the device-side status word of the current device.  Synchronises the
 * device.  Returns FA_OK, FA_ERR_TIMEOUT if a bounded wait expired since the last call
 * (detail[0] = where, detail[1] = block index, if detail != NULL), or FA_ERR_CUDA.
 */
int fa_device_status(unsigned int detail[2]);

/*
 * Self-test of the bounded waits (no counterpart in the paper): launches one small CTA whose 64
 * threads wait, for at most limit_us microseconds (1 .. 100000), on a barrier that nothing will
 * ever complete.  The wait gives up by construction -- no trap, no fault, no endless loop -- and
 * every thread returns normally.  Afterwards *gave_up (a DEVICE counter the caller zeroed) has
 * been raised by 64 and fa_device_status() reports FA_ERR_TIMEOUT once, with detail[0] == 990,
 * then FA_OK again: the same path a kernel of the library takes if one of its waits ever expired.
 */
int fa_selftest_wait(unsigned int limit_us, unsigned int* gave_up, void* stream);

const char* fa_strerror(int code);
int fa_version(void);         /* major * 10000 + minor * 100 + patch */
int fa_last_cuda_error(void); /* cudaError_t of the last failed CUDA call on this thread */

#ifdef __cplusplus
}
#endif
#endif /* FA_H_ */
