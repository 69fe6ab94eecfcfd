/*
 * sva.h -- C ABI of the block-sparse spatiotemporal attention library (sm_100a).
 *
 * The path follows the sparse-attention description of the paper (Sec. "Sparse
 * Attention": critical key blocks are chosen per query block and "computed
 * exactly"; LTX-2.3 pipeline paragraph: "score-based routing", block-wise
 * sparsity, "FlashAttention dense fallback"):
 *
 *   route   : mean-pool Q and K per block, block scores, per-row top-k or
 *             cumulative-mass cut  ->  CSR list of kept key blocks per query block
 *   attend  : softmax attention of every query over the keys of its kept blocks only
 *   dense   : the same with every block kept
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller.  The structs
 *     and the returned strings live on the host.
 *   - Q, K, V, O are [B, H, N, d] with d contiguous; strides for b, h, n are given in
 *     ELEMENTS.  N counts the valid tokens: tokens >= N do not exist (they are never
 *     read as keys and never written as queries), so buffers need not be padded.
 *   - Row index of the block structure: r = (b*H + h)*Nb + I with Nb = ceil(N/block),
 *     R = B*H*Nb.  CSR entries are key-block indices J in [0, Nb), ascending and
 *     unique inside a row.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*), never
 *     synchronise the device and may be issued back to back on one stream.
 *   - The library allocates no device memory; scratch is the caller's `workspace`
 *     (routing and attention each state their size).  One exception, by design:
 *     sva_block_select_noalloc takes its scratch from a 16 MiB device array that is part of
 *     the library image.  The library keeps no state between calls apart from per-device
 *     caches of constants (SM count, function attributes, that array's address) and the
 *     process-global test switches of sva_debug.h.
 *   - Three things differ from the boundary as first drafted for this path and are deliberate:
 *     (i) the attention calls take `workspace, workspace_bytes` (the tensor-core kernel reads V
 *     from a tiled transposed copy, and the library does not allocate); (ii) faults found on
 *     the device are bits in *device_status (SVA_DEV_*), not return codes: the calls are
 *     asynchronous, so the host cannot know at return time; (iii) "no forced window" is a
 *     NEGATIVE half-width; win_t = win_s = 0 is a window of one block, the diagonal.
 *   - Every call validates its arguments on the host first and returns a non-zero
 *     sva_status_t WITHOUT launching anything when they are bad.  No exception
 *     crosses the ABI.  Non-finite inputs give undefined (but memory-safe) results.
 *   - `device_status` (optional, device int32, zero it before the call): kernels OR
 *     SVA_DEV_* bits into it instead of trapping (a bad CSR entry is never used as an
 *     address, a pipeline wait that ran out gives up and the block exits).
 */
#ifndef SVA_H_
#define SVA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SVA_OK = 0,
  SVA_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, bad enum            */
  SVA_ERR_UNSUPPORTED = 2,   /* shape outside what the kernels are built for          */
  SVA_ERR_WORKSPACE = 3,     /* workspace missing or too small                        */
  SVA_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed (launch, map encode) */
  SVA_ERR_ALIGNMENT = 5,     /* pointer or stride not aligned as required             */
  SVA_ERR_SCRATCH_LIMIT = 6  /* sva_block_select_noalloc: problem needs more than the built-in scratch */
} sva_status_t;

/* bits a kernel may set in *device_status */
#define SVA_DEV_BAD_INDEX 1  /* CSR entry outside [0,Nb) or row_ptr not monotone: never dereferenced (the entry is
                                skipped, replaced by block 0 or its row treated as empty, depending on the kernel);
                                the affected rows' output is not meaningful */
#define SVA_DEV_TIMEOUT   2  /* a bounded pipeline wait expired; output of that block is undefined */

typedef enum { SVA_BF16 = 0, SVA_FP8_E4M3 = 1 } sva_qk_dtype_t;

typedef struct {
  int32_t B, H, N, d;        /* d in {64, 128}                                        */
  int32_t block;             /* tokens per block, 64 or 128; same for queries and keys */
  int64_t q_stride[3];       /* element strides of b, h, n (d has stride 1)           */
  int64_t k_stride[3];
  int64_t v_stride[3];
  int64_t o_stride[3];
  float softmax_scale;       /* <= 0 selects 1/sqrt(d)                                */
  int32_t qk_dtype;          /* SVA_BF16: Q,K bf16.  SVA_FP8_E4M3: Q,K are e4m3 bytes
                                with one fp32 scale per (b,h,block), [B,H,Nb]          */
} sva_problem_t;

typedef struct {
  int32_t mode;              /* 0 = top-k, 1 = cumulative softmax mass >= mass, capped at k */
  int32_t k;                 /* 1 <= k; values above Nb mean Nb                       */
  float mass;                /* tau in (0,1]; mode 1 only                             */
  int32_t win_t, win_s;      /* forced neighbour half-widths on the (frame, strip) block
                                grid; negative = no forced window                     */
  int32_t blocks_per_frame;  /* strips per frame; Nb must be a multiple when a window is set */
} sva_select_t;

/* Size queries for the routing call below (the routing step of the paper's sparse attention; they
 * compute nothing).  Capacity (in entries) that col_idx must have for sva_block_select: R * per-row cap,
 * where the per-row cap is max(min(k,Nb), window size).  0 on bad input, for more than 1024 blocks per
 * head (the routing kernels' limit) and when R * cap would not fit the CSR's int32 offsets. */
int64_t sva_select_max_nnz(const sva_problem_t* p, const sva_select_t* s);

/* Bytes of scratch sva_block_select needs (pooled means, the score matrix, per-row staging). 0 on bad input. */
size_t sva_select_workspace_bytes(const sva_problem_t* p, const sva_select_t* s);

/*
 * Routing (the paper's "score-based routing" of critical blocks).
 *   q, k          : Q and K as described by p (bf16, or e4m3 bytes + q_scale/k_scale)
 *   row_ptr       : out, [R+1] int32, row_ptr[R] = number of kept (row, block) pairs
 *   col_idx       : out, capacity sva_select_max_nnz entries; rows are packed back to back
 *   block_scores  : optional out, [B,H,Nb,Nb] fp32, the scaled pooled scores
 *   workspace     : >= sva_select_workspace_bytes, 256-byte aligned
 * Pooling is a mean over the VALID tokens of a block; score = softmax_scale*<qbar,kbar>;
 * order = forced window first, then score descending, ties to the LOWER block index;
 * mode 0 keeps min(k,Nb) blocks, mode 1 the shortest prefix whose softmax mass (over all
 * Nb blocks of the row) reaches `mass`, at least one block, at most k; the forced window is
 * always kept.  Arithmetic is fp32 with a fixed summation order; the kept mass of mode 1 is summed in
 * units of 2^-31 (order-independent), which can move a decision only where the mass is within ~1e-7 of
 * `mass`.  Results are deterministic.
 */
int sva_block_select(const sva_problem_t* p, const sva_select_t* s, const void* q, const void* k,
                     const float* q_scale, const float* k_scale, int32_t* row_ptr,
                     int32_t* col_idx, float* block_scores, void* workspace,
                     size_t workspace_bytes, void* stream);

/*
 * The pooling step of the routing alone: q_mean, k_mean ([B,H,Nb,d] fp32 contiguous, 16-byte aligned) =
 * the mean over the valid tokens of each block of Q and K as described by p (e4m3 codes are multiplied
 * by their block scale).  Together with sva_block_select_pooled it is sva_block_select in two calls,
 * for callers that want the HBM-bound pooling pass and the latency-bound rest on streams of their own.
 */
int sva_pool_qk(const sva_problem_t* p, const void* q, const void* k, const float* q_scale, const float* k_scale,
                float* q_mean, float* k_mean, void* stream);

/*
 * The same routing from block means the caller already holds (sva_pool_qk or sva_qk_norm_rope_pool writes them): the
 * pooling pass over Q and K is skipped, everything else is sva_block_select.
 *   q_mean, k_mean : [B,H,Nb,d] fp32 contiguous, 16-byte aligned; the mean over the valid tokens of each block
 * workspace as for sva_block_select (the part that held the means stays unused).
 */
int sva_block_select_pooled(const sva_problem_t* p, const sva_select_t* s, const float* q_mean, const float* k_mean,
                            int32_t* row_ptr, int32_t* col_idx, float* block_scores, void* workspace,
                            size_t workspace_bytes, void* stream);

/*
 * Attention prologue in one pass over Q and K (the paper lists the fused QK-norm + RoPE among the
 * lossless fusion flags of its deployments), per token n and head, in fp32:
 *   RMS norm over the head dimension :  u_c = x_c / sqrt(mean_c(x_c^2) + eps) * g_c      (g_q for Q, g_k for K)
 *   rotary embedding, adjacent pairs :  y_2i   = u_2i * cos[n,i] - u_2i+1 * sin[n,i]
 *                                        y_2i+1 = u_2i+1 * cos[n,i] + u_2i * sin[n,i]
 * y is rounded to bf16 and written to q_out / k_out (strides of p; may be q / k themselves).  From the
 * rounded values, in the same pass:
 *   q_mean, k_mean (optional, both or neither): block means for sva_block_select_pooled;
 *   q8, k8, q_scale, k_scale (optional, all or none): what sva_quantize_qk_fp8 would produce from q_out, k_out.
 * g_q, g_k: [d] fp32; cos_table, sin_table: [N, d/2] fp32 (shared by all heads and batch items; any
 * position-to-angle rule, e.g. a 3-D one for video, is the caller's); all 16-byte aligned.  Token rows >= N
 * are neither read nor written.  p->qk_dtype is ignored (the inputs are bf16).
 * Errors: INVALID_ARG (null, eps < 0, half-given optional group), ALIGNMENT, UNSUPPORTED.
 */
int sva_qk_norm_rope_pool(const sva_problem_t* p, const void* q, const void* k, const float* g_q, const float* g_k,
                          const float* cos_table, const float* sin_table, float eps, void* q_out, void* k_out,
                          float* q_mean, float* k_mean, void* q8, void* k8, float* q_scale, float* k_scale,
                          void* stream);

/*
 * Routing for callers that cannot allocate device memory.  (The paper has no counterpart;
 * this is a packaging variant of sva_block_select, same kernels, same results.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin handed only its
 * input and output buffers by a host runtime, a step that executes inside a region where the
 * allocator must not be touched, a process whose memory pool is owned by someone else.  Such
 * a caller has nowhere to get the `workspace` that sva_block_select asks for.
 *
 * Here the scratch lives inside the library: a file-scope device array of
 * SVA_NOALLOC_SCRATCH_BYTES (16 MiB), present on every GPU that loads the library for as long
 * as the process lives.  The call allocates and frees nothing.  Arguments and results are
 * those of sva_block_select minus workspace/workspace_bytes.
 *   - Limit: sva_select_workspace_bytes(p, s) must be <= SVA_NOALLOC_SCRATCH_BYTES, otherwise
 *     SVA_ERR_SCRATCH_LIMIT is returned and nothing is launched (B*H*Nb*d*8 bytes of pooled
 *     means and B*H*Nb*Nb*4 of scores dominate: e.g. 24 heads x 256 blocks x d=128 fits,
 *     64 heads x 372 blocks does not).
 *   - The first call on each device looks up the array's device address (once per device, with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls share the one array and it keeps the previous call's contents; every value
 *     a call reads from it is written by that same call first, so nothing needs clearing.
 *     Two calls that may overlap on the GPU (different streams, no dependency) race on it:
 *     serialise them.
 */
#define SVA_NOALLOC_SCRATCH_BYTES (16u << 20)
int sva_block_select_noalloc(const sva_problem_t* p, const sva_select_t* s, const void* q,
                             const void* k, const float* q_scale, const float* k_scale,
                             int32_t* row_ptr, int32_t* col_idx, float* block_scores,
                             void* stream);

/*
 * Exact attention over the kept blocks ("critical blocks are computed exactly"):
 *   o_i = sum_j softmax_j(scale*<q_i,k_j>) v_j,  j over the valid keys of the kept blocks
 *   lse_i = log sum_j exp(scale*<q_i,k_j>)       (optional, [B,H,N] fp32 contiguous)
 * O is bf16.  A row with an empty list writes zeros and lse = -inf.
 * q, k, v, o must be 16-byte aligned and every stride a multiple of 8 elements
 * (16 for e4m3 Q/K).  One tensor-core kernel (bf16 x bf16 or e4m3 x e4m3 MMA for Q K^T, bf16 for P V,
 * fp32 accumulate) serves every supported shape: d = 128 or 64 (64 is computed as 128 with a zero upper
 * half), bf16 or e4m3 Q/K, 128- or 64-token blocks.
 * workspace: >= sva_attn_one_call_workspace_bytes(p) bytes, 256-byte aligned: the kernel's row counters and, for
 * 64-token blocks, its tile lists (256 bytes to a few MB), rewritten by every call (so two calls that may overlap
 * on the GPU need a workspace each).  These calls read V where it lies.
 * sva_attn_workspace_bytes(p) is what the two-step form below needs: the same plus a tiled, transposed copy of V
 * (2*B*H*Nb*block*128 bytes) that sva_attn_prepare_v writes; it also serves the one-call form.
 * Both are 0 only for an unsupported problem.  sva_block_sparse_attn_fwd_fp4 needs 256 bytes (its row counters).
 */
size_t sva_attn_workspace_bytes(const sva_problem_t* p);
size_t sva_attn_one_call_workspace_bytes(const sva_problem_t* p);
int sva_block_sparse_attn_fwd(const sva_problem_t* p, const void* q, const void* k, const void* v,
                              const float* q_scale, const float* k_scale, const int32_t* row_ptr,
                              const int32_t* col_idx, void* o, float* lse, int32_t* device_status,
                              void* workspace, size_t workspace_bytes, void* stream);

/*
 * Piecewise attention: exact over the kept blocks, approximate remainder for the dropped ones (the paper's
 * sparse-attention section: non-critical blocks "compensated with first-order Taylor approximation"; its
 * LTX-2.3 pipeline runs with the "approximate remainder enabled").  The paper prints no formula; this is the
 * expansion of exp(scale <q_i, k_j>) about the mean key of each dropped block J (n_J keys, mean key kbar_J,
 * mean value vbar_J; a_iJ = scale <q_i, kbar_J>):
 *     Z_i = sum_{j kept} exp(s_ij)     + sum_{J dropped} n_J exp(a_iJ)              (the first-order term cancels)
 *     N_i = sum_{j kept} exp(s_ij) v_j + sum_{J dropped} n_J exp(a_iJ) vbar_J  [+ the first-order term]
 *     o_i = N_i / Z_i,   lse_i = ln Z_i            (exact part and remainder share one online softmax)
 * order 0 stops there: a dropped block acts as n_J copies of its mean key carrying its mean value.  On the
 * device the dropped blocks cost ceil(Nb/128) extra tiles per query block, whose "keys" and "values" are the
 * bf16-rounded block means (written into the workspace by this call), the kept blocks masked out.
 * order 1 adds scale * exp(sbar_IJ) * C_J^T q_i per dropped block, C_J = sum_j (k_j - kbar_J) v_j^T, weighted at
 * the query block's mean query (sbar_IJ is the routing score) so that the dropped blocks collapse into one d x d
 * matrix per query block, A_I = sum_J exp(sbar_IJ) C_J.  On the device: C_J per key block (one tensor-core product
 * K_J^T V_J, centred), the weights from `block_scores` and the CSR, A_I as a [Nb x Nb] x [Nb x d*d] GEMM per head
 * (2*Nb^2*d^2 FLOP), all bf16 in the workspace, and one more tile per row in the attention kernel whose "P" are the
 * scaled query values and whose "V" is A_I (two such tiles per tile row with 64-token blocks).
 *   block_scores : order 1 only: the [B,H,Nb,Nb] fp32 score matrix sva_block_select wrote for this Q, K
 *                  (16-byte aligned); ignored (may be NULL) for order 0
 * Supported: bf16 Q/K, d = 128, 128- or 64-token blocks; otherwise SVA_ERR_UNSUPPORTED.  A query block that
 * drops nothing gets exactly the result of sva_block_sparse_attn_fwd.  workspace: >=
 * sva_attn_remainder_workspace_bytes(p, order), 256-byte aligned, rewritten by every call (order 1 holds two
 * d x d bf16 matrices per block row there: 2 * 32 KB * R).  Everything else as for sva_block_sparse_attn_fwd.
 */
size_t sva_attn_remainder_workspace_bytes(const sva_problem_t* p, int32_t order);
int sva_block_sparse_attn_remainder_fwd(const sva_problem_t* p, const void* q, const void* k, const void* v,
                                        const int32_t* row_ptr, const int32_t* col_idx, const float* block_scores,
                                        void* o, float* lse, int32_t* device_status, int32_t order, void* workspace,
                                        size_t workspace_bytes, void* stream);

/* The dense fallback: every block kept, no CSR read. */
int sva_dense_attn_fwd(const sva_problem_t* p, const void* q, const void* k, const void* v,
                       const float* q_scale, const float* k_scale, void* o, float* lse,
                       int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The tensor-core path in two steps, on a transposed copy of V: the attention kernel then needs about 1 % fewer
 * cycles than the one-call form (both MMAs of one instruction form), at the price of the copy (a pass over V, its
 * workspace) -- worth it where the copy can be made off the critical path, e.g. because the producer of V can be
 * made to write the prepared layout itself; under a power cap the one-call form measured faster.
 * sva_attn_prepare_v writes the tiled transposed copy of V (per (b,h)
 * and key block one contiguous tile [d][block keys], keys >= N zero) and resets the row counter in
 * `workspace`; sva_block_sparse_attn_fwd_prepared then runs the attention kernel alone (row_ptr ==
 * NULL means dense).  A prepared workspace serves any number of attention calls on that V that do
 * not overlap on the GPU (after a call that reported SVA_DEV_TIMEOUT, prepare again); the caller
 * orders prepare and attention (same stream, or an event).  Together they compute what
 * sva_block_sparse_attn_fwd / sva_dense_attn_fwd compute in one call (q_scale, k_scale: as there, NULL for
 * bf16 Q/K; the bytes agree, the P V products being the same sums).  SVA_ERR_UNSUPPORTED for the dense form of bf16 Q/K with 64-token blocks (it runs as
 * 128-token blocks, which a workspace prepared for 64-token blocks does not fit): use the one-call
 * entry point there.
 */
int sva_attn_prepare_v(const sva_problem_t* p, const void* v, void* workspace, size_t workspace_bytes,
                       void* stream);
int sva_block_sparse_attn_fwd_prepared(const sva_problem_t* p, const void* q, const void* k, const float* q_scale,
                                       const float* k_scale, const int32_t* row_ptr, const int32_t* col_idx, void* o,
                                       float* lse, int32_t* device_status, void* workspace, size_t workspace_bytes,
                                       void* stream);

/*
 * Diagnostic twin of sva_block_sparse_attn_fwd: the same contract computed by a plain fp32
 * CUDA-core kernel (no tensor cores, no TMA).  row_ptr == NULL means dense.  Slow; it exists
 * so that the tensor-core kernel can be cross-checked on the device.
 */
int sva_block_sparse_attn_fwd_simt(const sva_problem_t* p, const void* q, const void* k,
                                   const void* v, const float* q_scale, const float* k_scale,
                                   const int32_t* row_ptr, const int32_t* col_idx, void* o,
                                   float* lse, int32_t* device_status, void* stream);

/*
 * FP8 variant's quantiser (the problem statement's "FP8 QK^T variant for the paper's quantization
 * technique"; the paper's Quantization section cites the 8-bit attention line of work for it and prints no
 * formula): per (b,h,block) absmax a over the valid tokens, scale s = a/448
 * (s = 1 when a = 0), y = x/s in fp32, round-to-nearest-even saturating cast to OCP e4m3.
 * q8/k8 use the strides of p (in elements = bytes); scales are [B,H,Nb] fp32.
 */
int sva_quantize_qk_fp8(const sva_problem_t* p, const void* q_bf16, const void* k_bf16, void* q8,
                        void* k8, float* q_scale, float* k_scale, void* stream);

/*
 * Block-scaled 4-bit quantiser for Q and K (NVFP4 is the paper's quantisation format -- its Quantization section
 * and the per-model appendix paragraphs -- and the low-bit attention work it cites quantises Q K^T; the paper
 * prints no formula).  As read here, every scalar step one fp32 operation rounded to nearest:
 *   per (b,h)            g  = amax / (6 * 448) over the existing tokens (1 if amax = 0)
 *   per token, 16 elems  sf = e4m3((amax_block / 6) / g), round-to-nearest-even, saturating at 448
 *   per element          code = e2m1(x / (value(sf) * g)), round-to-nearest-even, saturating at +-6
 *                        (e2m1 magnitudes 0, .5, 1, 1.5, 2, 3, 4, 6; code = sign << 3 | index; all 0 where sf = 0)
 *   x ~= value(code) * value(sf) * g
 * Outputs (device, 16-byte aligned), in the layout the block-scaled tensor-core MMA takes:
 *   q4, k4     : [B*H][Nb*128 tokens][64] bytes, two codes per byte (even element in the low nibble), rows >= N zero
 *   q_sf, k_sf : [B*H][Nb][2][32][4][4] bytes: for 128-token block I and half c of the head dimension, the scale of
 *                token t (within the block) and scale block kb (within the half) is byte (t%32)*16 + (t/32)*4 + kb
 *   q_g, k_g   : [B*H] fp32
 * d = 128 and block = 128 only (SVA_ERR_UNSUPPORTED otherwise).  workspace: >= 8*B*H bytes, 16-byte aligned.
 */
int sva_quantize_qk_fp4(const sva_problem_t* p, const void* q_bf16, const void* k_bf16, void* q4, void* k4,
                        void* q_sf, void* k_sf, float* q_g, float* k_g, void* workspace, size_t workspace_bytes,
                        void* stream);

/*
 * Attention with 4-bit Q and K (the block-scaled low-bit Q K^T of the paper's quantisation direction): q4, k4,
 * q_sf, k_sf, q_g, k_g as sva_quantize_qk_fp4 writes them; V, P V, O and the softmax as in
 * sva_block_sparse_attn_fwd.  S = Q K^T runs as a block-scaled e2m1 x e2m1 tensor-core MMA with fp32 accumulation
 * (the e4m3 scale factors are applied by the MMA, the two fp32 tensor scales are folded into the softmax scale),
 * so the result is attention over the DEQUANTISED Q and K.  row_ptr == NULL means dense.  d = 128, block = 128
 * only; p's q/k strides and qk_dtype are ignored (the code tensors have their own fixed layout).  V is read where
 * it lies (no transposed copy): workspace >= 256 bytes (the row counters), 256-byte aligned.
 */
int sva_block_sparse_attn_fwd_fp4(const sva_problem_t* p, const void* q4, const void* k4, const void* q_sf,
                                  const void* k_sf, const float* q_g, const float* k_g, const void* v,
                                  const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse,
                                  int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same quantiser with K smoothing, the step the 8-bit attention work cited in the paper's related
 * work on quantised attention puts before the cast: per (b,h) the mean key over the N tokens,
 *   k_mean[b,h,:] = (1/N) sum_j k[b,h,j,:]        (fp32; per-block sums in a fixed order, then the blocks in
 *                                                   index order, so the result is reproducible)
 * is subtracted from every key in fp32 (one rounding) and k - k_mean is what gets scaled and cast.  Every
 * logit of query i changes by the same -scale*<q_i, k_mean>, so softmax over keys, O, pooled-score order
 * and kept mass are those of the original problem (up to rounding), while K loses the common offset that
 * would otherwise use up the e4m3 range.  Only the log-sum-exp moves:
 *   lse_original[b,h,i] = lse_of_the_quantised_problem[b,h,i] + lse_shift[b,h,i],
 *   lse_shift[b,h,i] = scale * <q[b,h,i,:], k_mean[b,h,:]>   (from the bf16 q; optional, [B,H,N] fp32).
 * Q is quantised as by sva_quantize_qk_fp8.  k_mean: [B,H,d] fp32, 16-byte aligned, written.  workspace:
 * >= sva_smooth_workspace_bytes(p) = 4*B*H*Nb*d bytes, 16-byte aligned.
 * Errors: as sva_quantize_qk_fp8, plus SVA_ERR_WORKSPACE.
 */
size_t sva_smooth_workspace_bytes(const sva_problem_t* p);
int sva_quantize_qk_fp8_smooth_k(const sva_problem_t* p, const void* q_bf16, const void* k_bf16, void* q8,
                                 void* k8, float* q_scale, float* k_scale, float* k_mean, float* lse_shift,
                                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * Token-subset gather / scatter (the paper's token pruning keeps a subset of the video tokens, about
 * half of them, on some denoising calls; attention then runs over the kept tokens only, and the
 * blocking of the routing applies to the gathered sequence).
 *   gather : dst[b,h,m,:]              = src[b,h,token_idx[b,m],:]   m < M, token_idx[b,m] in [0, n_src)
 *   scatter: dst[b,h,token_idx[b,m],:] = src[b,h,m,:]                token_idx[b,m] in [0, n_dst)
 * src / dst are [B,H,*,d] tensors of elem_bytes-sized elements (1, 2 or 4), d contiguous, strides in
 * elements, 16-byte aligned with d*elem_bytes a multiple of 16; token_idx is [B,M] int32 (the same
 * subset for every head of a batch item; repeated indices make scatter order-dependent).  Rows that
 * scatter does not name keep their contents.  An index out of range is reported in device_status
 * (SVA_DEV_BAD_INDEX) and its row skipped.
 */
int sva_gather_tokens(const void* src, const int64_t src_stride[3], const int32_t* token_idx, int32_t B, int32_t H,
                      int32_t M, int32_t n_src, int32_t d, int32_t elem_bytes, void* dst,
                      const int64_t dst_stride[3], int32_t* device_status, void* stream);
int sva_scatter_tokens(const void* src, const int64_t src_stride[3], const int32_t* token_idx, int32_t B, int32_t H,
                       int32_t M, int32_t n_dst, int32_t d, int32_t elem_bytes, void* dst,
                       const int64_t dst_stride[3], int32_t* device_status, void* stream);

const char* sva_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* SVA_H_ */
