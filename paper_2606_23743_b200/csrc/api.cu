// C ABI entry points: host-side validation, then the kernel launchers.
#include "common.cuh"

namespace sva {

void ts_set_prof_buffer(void* p);
void ts_set_debug_mode(int v);
int ts_set_wait_limit(long long cycles);

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int validate_problem(const sva_problem_t* p) {
  if (!p) return SVA_ERR_INVALID_ARG;
  if (p->B <= 0 || p->H <= 0 || p->N <= 0) return SVA_ERR_INVALID_ARG;
  if (p->qk_dtype != SVA_BF16 && p->qk_dtype != SVA_FP8_E4M3) return SVA_ERR_INVALID_ARG;
  if (p->d != 64 && p->d != 128) return SVA_ERR_UNSUPPORTED;
  if (p->block != 64 && p->block != 128) return SVA_ERR_UNSUPPORTED;
  if ((long long)p->B * p->H * ((p->N + p->block - 1) / p->block) > 0x7fffffffLL / 64) return SVA_ERR_UNSUPPORTED;
  return SVA_OK;
}

static int check_strides(const int64_t s[3], int mult) {
  for (int i = 0; i < 3; ++i) {
    if (s[i] < 0) return SVA_ERR_INVALID_ARG;
    if (s[i] % mult != 0) return SVA_ERR_ALIGNMENT;
  }
  return SVA_OK;
}

// What the routing kernels cannot take: more than 1024 blocks per head (a lane holds at most 32 scores of
// a row), or a CSR whose capacity R * cap would overflow its int32 offsets.
static bool select_fits(const Dims& m, const sva_select_t* s) {
  return m.Nb <= 1024 && (long long)m.R * select_row_cap(m, s) <= 0x7fffffffLL;
}

static int validate_select(const Dims& m, const sva_select_t* s) {
  if (!s) return SVA_ERR_INVALID_ARG;
  if (s->mode != 0 && s->mode != 1) return SVA_ERR_INVALID_ARG;
  if (s->k < 1) return SVA_ERR_INVALID_ARG;
  if (s->mode == 1 && !(s->mass > 0.f && s->mass <= 1.f)) return SVA_ERR_INVALID_ARG;
  if (s->win_t >= 0 && s->win_s >= 0) {
    if (s->blocks_per_frame <= 0 || m.Nb % s->blocks_per_frame != 0) return SVA_ERR_INVALID_ARG;
  }
  if (!select_fits(m, s)) return SVA_ERR_UNSUPPORTED;
  return SVA_OK;
}

static int validate_attn(const sva_problem_t* p, const void* q, const void* k, const void* v,
                         const float* qs, const float* ks, const void* o) {
  int rc = validate_problem(p);
  if (rc) return rc;
  if (!q || !k || !v || !o) return SVA_ERR_INVALID_ARG;
  const bool f8 = p->qk_dtype == SVA_FP8_E4M3;
  if (f8 && (!qs || !ks)) return SVA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return SVA_ERR_ALIGNMENT;
  if ((rc = check_strides(p->q_stride, f8 ? 16 : 8))) return rc;
  if ((rc = check_strides(p->k_stride, f8 ? 16 : 8))) return rc;
  if ((rc = check_strides(p->v_stride, 8))) return rc;
  if ((rc = check_strides(p->o_stride, 8))) return rc;
  if (p->q_stride[2] < p->d || p->k_stride[2] < p->d || p->v_stride[2] < p->d || p->o_stride[2] < p->d)
    return SVA_ERR_INVALID_ARG;
  return SVA_OK;
}

// The tensor-core kernel serves every shape validate_problem lets through except more than 16383 key
// blocks per head (its 64-token-block tile descriptors hold 14-bit block indices); only there do the
// public attention calls run the CUDA-core kernel instead.

}  // namespace sva

using namespace sva;

extern "C" {

int64_t sva_select_max_nnz(const sva_problem_t* p, const sva_select_t* s) {
  if (validate_problem(p) || !s || s->k < 1) return 0;
  Dims m = make_dims(p);
  if (!select_fits(m, s)) return 0;
  return (int64_t)m.R * select_row_cap(m, s);
}

size_t sva_select_workspace_bytes(const sva_problem_t* p, const sva_select_t* s) {
  if (validate_problem(p) || !s || s->k < 1) return 0;
  Dims m = make_dims(p);
  if (!select_fits(m, s)) return 0;
  return select_workspace_bytes(m, s);
}

int sva_block_select(const sva_problem_t* p, const sva_select_t* s, const void* q, const void* k,
                     const float* q_scale, const float* k_scale, int32_t* row_ptr,
                     int32_t* col_idx, float* block_scores, void* workspace,
                     size_t workspace_bytes, void* stream) {
  int rc = validate_problem(p);
  if (rc) return rc;
  Dims m = make_dims(p);
  if ((rc = validate_select(m, s))) return rc;
  if (!q || !k || !row_ptr || !col_idx) return SVA_ERR_INVALID_ARG;
  if (m.fp8 && (!q_scale || !k_scale)) return SVA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k)) return SVA_ERR_ALIGNMENT;
  if ((rc = check_strides(p->q_stride, m.fp8 ? 16 : 8))) return rc;
  if ((rc = check_strides(p->k_stride, m.fp8 ? 16 : 8))) return rc;
  if (!workspace) return SVA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return SVA_ERR_ALIGNMENT;
  return launch_select(m, p, s, q, k, q_scale, k_scale, row_ptr, col_idx, block_scores, workspace,
                       workspace_bytes, (cudaStream_t)stream);
}

int sva_pool_qk(const sva_problem_t* p, const void* q, const void* k, const float* q_scale, const float* k_scale,
                float* q_mean, float* k_mean, void* stream) {
  int rc = validate_problem(p);
  if (rc) return rc;
  Dims m = make_dims(p);
  if (!q || !k || !q_mean || !k_mean) return SVA_ERR_INVALID_ARG;
  if (m.fp8 && (!q_scale || !k_scale)) return SVA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(q_mean) || !aligned16(k_mean)) return SVA_ERR_ALIGNMENT;
  if ((rc = check_strides(p->q_stride, m.fp8 ? 16 : 8))) return rc;
  if ((rc = check_strides(p->k_stride, m.fp8 ? 16 : 8))) return rc;
  return launch_pool(m, p, q, k, q_scale, k_scale, q_mean, k_mean, (cudaStream_t)stream);
}

int sva_block_select_pooled(const sva_problem_t* p, const sva_select_t* s, const float* q_mean, const float* k_mean,
                            int32_t* row_ptr, int32_t* col_idx, float* block_scores, void* workspace,
                            size_t workspace_bytes, void* stream) {
  int rc = validate_problem(p);
  if (rc) return rc;
  Dims m = make_dims(p);
  if ((rc = validate_select(m, s))) return rc;
  if (!q_mean || !k_mean || !row_ptr || !col_idx) return SVA_ERR_INVALID_ARG;
  if (!aligned16(q_mean) || !aligned16(k_mean)) return SVA_ERR_ALIGNMENT;
  if (!workspace) return SVA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return SVA_ERR_ALIGNMENT;
  return launch_select_pooled(m, p, s, q_mean, k_mean, row_ptr, col_idx, block_scores, workspace, workspace_bytes,
                              (cudaStream_t)stream);
}

int sva_qk_norm_rope_pool(const sva_problem_t* p, const void* q, const void* k, const float* g_q, const float* g_k,
                          const float* cos_table, const float* sin_table, float eps, void* q_out, void* k_out,
                          float* q_mean, float* k_mean, void* q8, void* k8, float* q_scale, float* k_scale,
                          void* stream) {
  int rc = validate_problem(p);
  if (rc) return rc;
  if (!q || !k || !g_q || !g_k || !cos_table || !sin_table || !q_out || !k_out) return SVA_ERR_INVALID_ARG;
  if (!(eps >= 0.f)) return SVA_ERR_INVALID_ARG;
  if ((q_mean == nullptr) != (k_mean == nullptr)) return SVA_ERR_INVALID_ARG;
  const int n8 = (q8 != nullptr) + (k8 != nullptr) + (q_scale != nullptr) + (k_scale != nullptr);
  if (n8 != 0 && n8 != 4) return SVA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(q_out) || !aligned16(k_out) || !aligned16(g_q) || !aligned16(g_k) ||
      !aligned16(cos_table) || !aligned16(sin_table) || (q8 && (!aligned16(q8) || !aligned16(k8))))
    return SVA_ERR_ALIGNMENT;
  if ((rc = check_strides(p->q_stride, q8 ? 16 : 8))) return rc;
  if ((rc = check_strides(p->k_stride, q8 ? 16 : 8))) return rc;
  Dims m = make_dims(p);
  return launch_prologue(m, p, q, k, g_q, g_k, cos_table, sin_table, eps, q_out, k_out, q_mean, k_mean, q8, k8,
                         q_scale, k_scale, (cudaStream_t)stream);
}

/* Same routing, scratch taken from the library's built-in device array: no allocation. */
int sva_block_select_noalloc(const sva_problem_t* p, const sva_select_t* s, const void* q,
                             const void* k, const float* q_scale, const float* k_scale,
                             int32_t* row_ptr, int32_t* col_idx, float* block_scores,
                             void* stream) {
  int rc = validate_problem(p);
  if (rc) return rc;
  Dims m = make_dims(p);
  if ((rc = validate_select(m, s))) return rc;
  if (!q || !k || !row_ptr || !col_idx) return SVA_ERR_INVALID_ARG;
  if (m.fp8 && (!q_scale || !k_scale)) return SVA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k)) return SVA_ERR_ALIGNMENT;
  if ((rc = check_strides(p->q_stride, m.fp8 ? 16 : 8))) return rc;
  if ((rc = check_strides(p->k_stride, m.fp8 ? 16 : 8))) return rc;
  return launch_select_noalloc(m, p, s, q, k, q_scale, k_scale, row_ptr, col_idx, block_scores,
                               (cudaStream_t)stream);
}

size_t sva_attn_workspace_bytes(const sva_problem_t* p) {
  if (validate_problem(p)) return 0;
  Dims m = make_dims(p);
  return attn_ts_workspace_bytes(m);
}

size_t sva_attn_one_call_workspace_bytes(const sva_problem_t* p) {
  if (validate_problem(p)) return 0;
  return attn_ts_one_call_workspace_bytes(make_dims(p));
}

int sva_block_sparse_attn_fwd(const sva_problem_t* p, const void* q, const void* k, const void* v,
                              const float* q_scale, const float* k_scale, const int32_t* row_ptr,
                              const int32_t* col_idx, void* o, float* lse, int32_t* device_status,
                              void* workspace, size_t workspace_bytes, void* stream) {
  int rc = validate_attn(p, q, k, v, q_scale, k_scale, o);
  if (rc) return rc;
  if (!row_ptr || !col_idx) return SVA_ERR_INVALID_ARG;
  Dims m = make_dims(p);
  if (attn_ts_serves(m))
    return launch_attn_ts(m, p, q, k, v, q_scale, k_scale, row_ptr, col_idx, o, lse, device_status, workspace, workspace_bytes,
                          (cudaStream_t)stream);
  return launch_attn_simt(m, p, q, k, v, q_scale, k_scale, row_ptr, col_idx, o, lse, device_status,
                          (cudaStream_t)stream);
}

size_t sva_attn_remainder_workspace_bytes(const sva_problem_t* p, int32_t order) {
  if (validate_problem(p) || (order != 0 && order != 1)) return 0;
  return attn_ts_remainder_workspace_bytes(make_dims(p), order);
}

int sva_block_sparse_attn_remainder_fwd(const sva_problem_t* p, const void* q, const void* k, const void* v,
                                        const int32_t* row_ptr, const int32_t* col_idx, const float* block_scores,
                                        void* o, float* lse, int32_t* device_status, int32_t order, void* workspace,
                                        size_t workspace_bytes, void* stream) {
  int rc = validate_attn(p, q, k, v, nullptr, nullptr, o);
  if (rc) return rc;
  if (!row_ptr || !col_idx) return SVA_ERR_INVALID_ARG;
  if (order != 0 && order != 1) return SVA_ERR_INVALID_ARG;
  Dims m = make_dims(p);
  if (!attn_ts_remainder_serves(m)) return SVA_ERR_UNSUPPORTED;
  if (order == 1 && (!block_scores || !aligned16(block_scores))) return SVA_ERR_INVALID_ARG;
  return launch_attn_ts(m, p, q, k, v, nullptr, nullptr, row_ptr, col_idx, o, lse, device_status, workspace,
                        workspace_bytes, (cudaStream_t)stream, order, block_scores);
}

int sva_block_sparse_attn_fwd_fp4(const sva_problem_t* p, const void* q4, const void* k4, const void* q_sf,
                                  const void* k_sf, const float* q_g, const float* k_g, const void* v,
                                  const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse,
                                  int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = validate_problem(p);
  if (rc) return rc;
  if (!q4 || !k4 || !q_sf || !k_sf || !q_g || !k_g || !v || !o) return SVA_ERR_INVALID_ARG;
  if (row_ptr && !col_idx) return SVA_ERR_INVALID_ARG;
  if (!aligned16(q4) || !aligned16(k4) || !aligned16(q_sf) || !aligned16(k_sf) || !aligned16(v) || !aligned16(o))
    return SVA_ERR_ALIGNMENT;
  if ((rc = check_strides(p->v_stride, 8))) return rc;
  if ((rc = check_strides(p->o_stride, 8))) return rc;
  if (p->v_stride[2] < p->d || p->o_stride[2] < p->d) return SVA_ERR_INVALID_ARG;
  Dims m = make_dims(p);
  m.fp8 = false;
  return launch_attn_ts_fp4(m, p, q4, k4, q_sf, k_sf, q_g, k_g, v, row_ptr, col_idx, o, lse, device_status, workspace,
                            workspace_bytes, (cudaStream_t)stream);
}

int sva_dense_attn_fwd(const sva_problem_t* p, const void* q, const void* k, const void* v,
                       const float* q_scale, const float* k_scale, void* o, float* lse,
                       int32_t* device_status, void* workspace, size_t workspace_bytes, void* stream) {
  int rc = validate_attn(p, q, k, v, q_scale, k_scale, o);
  if (rc) return rc;
  Dims m = make_dims(p);
  if (attn_ts_serves(m))
    return launch_attn_ts(m, p, q, k, v, q_scale, k_scale, nullptr, nullptr, o, lse, device_status, workspace, workspace_bytes,
                          (cudaStream_t)stream);
  return launch_attn_simt(m, p, q, k, v, q_scale, k_scale, nullptr, nullptr, o, lse, device_status,
                          (cudaStream_t)stream);
}

int sva_attn_prepare_v(const sva_problem_t* p, const void* v, void* workspace, size_t workspace_bytes,
                       void* stream) {
  int rc = validate_problem(p);
  if (rc) return rc;
  if (!v) return SVA_ERR_INVALID_ARG;
  if (!aligned16(v)) return SVA_ERR_ALIGNMENT;
  if ((rc = check_strides(p->v_stride, 8))) return rc;
  if (p->v_stride[2] < p->d) return SVA_ERR_INVALID_ARG;
  Dims m = make_dims(p);
  if (!attn_ts_serves(m)) return SVA_ERR_UNSUPPORTED;
  return launch_prepare_v_ts(m, p, v, workspace, workspace_bytes, (cudaStream_t)stream);
}

int sva_block_sparse_attn_fwd_prepared(const sva_problem_t* p, const void* q, const void* k, const float* q_scale,
                                       const float* k_scale, const int32_t* row_ptr, const int32_t* col_idx, void* o,
                                       float* lse, int32_t* device_status, void* workspace, size_t workspace_bytes,
                                       void* stream) {
  // (q stands in for v in the shared checks: the prepared call takes no V pointer; the v strides of p are still checked)
  int rc = validate_attn(p, q, k, q, q_scale, k_scale, o);
  if (rc) return rc;
  if (row_ptr && !col_idx) return SVA_ERR_INVALID_ARG;
  Dims m = make_dims(p);
  if (!attn_ts_serves(m)) return SVA_ERR_UNSUPPORTED;
  return launch_attn_ts(m, p, q, k, nullptr, q_scale, k_scale, row_ptr, col_idx, o, lse, device_status, workspace,
                        workspace_bytes, (cudaStream_t)stream);
}

int sva_block_sparse_attn_fwd_simt(const sva_problem_t* p, const void* q, const void* k,
                                   const void* v, const float* q_scale, const float* k_scale,
                                   const int32_t* row_ptr, const int32_t* col_idx, void* o,
                                   float* lse, int32_t* device_status, void* stream) {
  int rc = validate_attn(p, q, k, v, q_scale, k_scale, o);
  if (rc) return rc;
  if (row_ptr && !col_idx) return SVA_ERR_INVALID_ARG;
  Dims m = make_dims(p);
  return launch_attn_simt(m, p, q, k, v, q_scale, k_scale, row_ptr, col_idx, o, lse, device_status,
                          (cudaStream_t)stream);
}

int sva_quantize_qk_fp8(const sva_problem_t* p, const void* q_bf16, const void* k_bf16, void* q8,
                        void* k8, float* q_scale, float* k_scale, void* stream) {
  int rc = validate_problem(p);
  if (rc) return rc;
  if (!q_bf16 || !k_bf16 || !q8 || !k8 || !q_scale || !k_scale) return SVA_ERR_INVALID_ARG;
  if (!aligned16(q_bf16) || !aligned16(k_bf16) || !aligned16(q8) || !aligned16(k8)) return SVA_ERR_ALIGNMENT;
  if ((rc = check_strides(p->q_stride, 16))) return rc;
  if ((rc = check_strides(p->k_stride, 16))) return rc;
  Dims m = make_dims(p);
  return launch_quantize(m, p, q_bf16, k_bf16, q8, k8, q_scale, k_scale, nullptr, nullptr, nullptr, (cudaStream_t)stream);
}

int sva_quantize_qk_fp4(const sva_problem_t* p, const void* q_bf16, const void* k_bf16, void* q4, void* k4,
                        void* q_sf, void* k_sf, float* q_g, float* k_g, void* workspace, size_t workspace_bytes,
                        void* stream) {
  int rc = validate_problem(p);
  if (rc) return rc;
  if (!q_bf16 || !k_bf16 || !q4 || !k4 || !q_sf || !k_sf || !q_g || !k_g) return SVA_ERR_INVALID_ARG;
  if (!aligned16(q_bf16) || !aligned16(k_bf16) || !aligned16(q4) || !aligned16(k4) || !aligned16(q_sf) || !aligned16(k_sf))
    return SVA_ERR_ALIGNMENT;
  if ((rc = check_strides(p->q_stride, 16))) return rc;
  if ((rc = check_strides(p->k_stride, 16))) return rc;
  Dims m = make_dims(p);
  if (m.d != 128 || m.block != 128) return SVA_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < (size_t)8 * m.B * m.H) return SVA_ERR_WORKSPACE;
  if (!aligned16(workspace)) return SVA_ERR_ALIGNMENT;
  return launch_quantize4(m, p, q_bf16, k_bf16, q4, k4, q_sf, k_sf, q_g, k_g, workspace, (cudaStream_t)stream);
}

size_t sva_smooth_workspace_bytes(const sva_problem_t* p) {
  if (validate_problem(p)) return 0;
  return smooth_workspace_bytes(make_dims(p));
}

int sva_quantize_qk_fp8_smooth_k(const sva_problem_t* p, const void* q_bf16, const void* k_bf16, void* q8,
                                 void* k8, float* q_scale, float* k_scale, float* k_mean, float* lse_shift,
                                 void* workspace, size_t workspace_bytes, void* stream) {
  int rc = validate_problem(p);
  if (rc) return rc;
  if (!q_bf16 || !k_bf16 || !q8 || !k8 || !q_scale || !k_scale || !k_mean) return SVA_ERR_INVALID_ARG;
  if (!aligned16(q_bf16) || !aligned16(k_bf16) || !aligned16(q8) || !aligned16(k8) || !aligned16(k_mean))
    return SVA_ERR_ALIGNMENT;
  if ((rc = check_strides(p->q_stride, 16))) return rc;
  if ((rc = check_strides(p->k_stride, 16))) return rc;
  Dims m = make_dims(p);
  if (!workspace || workspace_bytes < smooth_workspace_bytes(m)) return SVA_ERR_WORKSPACE;
  if (!aligned16(workspace)) return SVA_ERR_ALIGNMENT;
  return launch_quantize(m, p, q_bf16, k_bf16, q8, k8, q_scale, k_scale, k_mean, lse_shift, workspace,
                         (cudaStream_t)stream);
}

static int validate_token_move(const void* a, const int64_t sa[3], const void* b, const int64_t sb[3],
                               const int32_t* idx, int B, int H, int M, int n_full, int d, int elem_bytes) {
  if (!a || !b || !idx || !sa || !sb) return SVA_ERR_INVALID_ARG;
  if (B <= 0 || H <= 0 || M <= 0 || n_full <= 0 || M > n_full || d <= 0) return SVA_ERR_INVALID_ARG;
  if (elem_bytes != 1 && elem_bytes != 2 && elem_bytes != 4) return SVA_ERR_INVALID_ARG;
  if ((d * elem_bytes) % 16 != 0) return SVA_ERR_UNSUPPORTED;
  if (!aligned16(a) || !aligned16(b)) return SVA_ERR_ALIGNMENT;
  for (int i = 0; i < 3; ++i)
    if (sa[i] < 0 || sb[i] < 0 || (sa[i] * elem_bytes) % 16 != 0 || (sb[i] * elem_bytes) % 16 != 0) return SVA_ERR_ALIGNMENT;
  if (sa[2] < d || sb[2] < d) return SVA_ERR_INVALID_ARG;
  return SVA_OK;
}

int sva_gather_tokens(const void* src, const int64_t src_stride[3], const int32_t* token_idx, int32_t B, int32_t H,
                      int32_t M, int32_t n_src, int32_t d, int32_t elem_bytes, void* dst,
                      const int64_t dst_stride[3], int32_t* device_status, void* stream) {
  int rc = validate_token_move(src, src_stride, dst, dst_stride, token_idx, B, H, M, n_src, d, elem_bytes);
  if (rc) return rc;
  return launch_token_move(false, src, src_stride, dst, dst_stride, token_idx, B, H, M, n_src, d, elem_bytes,
                           device_status, (cudaStream_t)stream);
}

int sva_scatter_tokens(const void* src, const int64_t src_stride[3], const int32_t* token_idx, int32_t B, int32_t H,
                       int32_t M, int32_t n_dst, int32_t d, int32_t elem_bytes, void* dst,
                       const int64_t dst_stride[3], int32_t* device_status, void* stream) {
  int rc = validate_token_move(src, src_stride, dst, dst_stride, token_idx, B, H, M, n_dst, d, elem_bytes);
  if (rc) return rc;
  return launch_token_move(true, src, src_stride, dst, dst_stride, token_idx, B, H, M, n_dst, d, elem_bytes,
                           device_status, (cudaStream_t)stream);
}

const char* sva_status_string(int status) {
  switch (status) {
    case SVA_OK: return "ok";
    case SVA_ERR_INVALID_ARG: return "invalid argument";
    case SVA_ERR_UNSUPPORTED: return "unsupported shape";
    case SVA_ERR_WORKSPACE: return "workspace missing or too small";
    case SVA_ERR_CUDA: return "CUDA call failed";
    case SVA_ERR_ALIGNMENT: return "pointer or stride misaligned";
    case SVA_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the built-in no-allocation array holds";
    default: return "unknown status";
  }
}

/* tuning aid (not part of the public header): device buffer of 320 int64; entry 319 receives the longest
   CTA's cycle count of the next attention launches; NULL = off */
void sva_debug_set_prof_buffer(void* p) { ts_set_prof_buffer(p); }
/* bit 0 skips the exponentials (tuning aid: results are wrong); bit 4 (test aid) withholds a row's K
   tiles after the first so that a bounded wait runs out */
void sva_debug_set_mode(int v) { ts_set_debug_mode(v); }
/* test aid: cycles a device-side wait may last before the CTA gives up (<= 0 restores the default) */
int sva_debug_set_wait_limit(long long cycles) { return ts_set_wait_limit(cycles); }

}  // extern "C"
