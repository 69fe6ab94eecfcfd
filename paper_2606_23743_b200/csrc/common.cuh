// Shared host/device helpers of the sva library (CUDA side only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sva.h"

namespace sva {

struct Dims {
  int B, H, N, d, block, Nb, R;
  float scale;
  bool fp8;
};

inline Dims make_dims(const sva_problem_t* p) {
  Dims m;
  m.B = p->B; m.H = p->H; m.N = p->N; m.d = p->d; m.block = p->block;
  m.Nb = (p->N + p->block - 1) / p->block;
  m.R = p->B * p->H * m.Nb;
  m.scale = p->softmax_scale > 0.f ? p->softmax_scale : 1.0f / sqrtf((float)p->d);
  m.fp8 = p->qk_dtype == SVA_FP8_E4M3;
  return m;
}

struct Strides { long long b, h, n; };
inline Strides make_strides(const int64_t s[3]) { return Strides{(long long)s[0], (long long)s[1], (long long)s[2]}; }

__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// e4m3 byte -> float (exact)
__device__ __forceinline__ float e4m3_to_float(uint32_t byte) {
  __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)byte, __NV_E4M3);
  return __half2float(__half(h));
}

// x / s for the e4m3 cast, s and y = RN(1/s) fixed for a whole block: q0 = x*y, one exact residual, one
// correction -- the correctly rounded quotient (Markstein's sequence) in three FMA-pipe operations instead of
// the dozen of a general division, valid while s is in [2^-60, 2^60] and its significand is not all ones
// (div_fast_ok; otherwise the caller divides).  |x| below s*2^-12 may come out one unit off, which the cast
// sends to zero all the same.  The residual is formed negated, t = q0*s - x, so that a zero x keeps its
// sign through both steps (-0 stays -0, as in a true division).
__device__ __forceinline__ bool div_fast_ok(float s) {
  return s >= 8.673617379884035e-19f && s <= 1.152921504606847e18f && (__float_as_uint(s) & 0x7fffffu) != 0x7fffffu;
}
__device__ __forceinline__ float div_fast(float x, float s, float y) {
  const float q0 = x * y;
  const float t = fmaf(q0, s, -x);
  return fmaf(-t, y, q0);
}
// two fp32 -> two e4m3 bytes (round to nearest even, saturating), first value in the low byte
__device__ __forceinline__ uint32_t e4m3x2(float lo, float hi) {
  return (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(lo, hi), __NV_SATFINITE, __NV_E4M3);
}

// host-side argument checks shared by the entry points
int validate_problem(const sva_problem_t* p);

// launchers (each returns an sva_status_t)
int launch_select(const Dims& m, const sva_problem_t* p, const sva_select_t* s, const void* q,
                  const void* k, const float* q_scale, const float* k_scale, int32_t* row_ptr,
                  int32_t* col_idx, float* block_scores, void* ws, size_t ws_bytes,
                  cudaStream_t st);
size_t select_workspace_bytes(const Dims& m, const sva_select_t* s);
int launch_pool(const Dims& m, const sva_problem_t* p, const void* q, const void* k, const float* q_scale,
                const float* k_scale, float* qbar, float* kbar, cudaStream_t st);
int launch_select_pooled(const Dims& m, const sva_problem_t* p, const sva_select_t* s, const float* qbar,
                         const float* kbar, int32_t* row_ptr, int32_t* col_idx, float* block_scores, void* ws,
                         size_t ws_bytes, cudaStream_t st);
int launch_prologue(const Dims& m, const sva_problem_t* p, const void* q, const void* k, const float* gq,
                    const float* gk, const float* cosn, const float* sinn, float eps, void* qo, void* ko,
                    float* qbar, float* kbar, void* q8, void* k8, float* qs, float* ks, cudaStream_t st);
int launch_select_noalloc(const Dims& m, const sva_problem_t* p, const sva_select_t* s,
                          const void* q, const void* k, const float* q_scale, const float* k_scale,
                          int32_t* row_ptr, int32_t* col_idx, float* block_scores, cudaStream_t st);
int select_row_cap(const Dims& m, const sva_select_t* s);
size_t smooth_workspace_bytes(const Dims& m);
int launch_quantize(const Dims& m, const sva_problem_t* p, const void* q, const void* k, void* q8,
                    void* k8, float* qs, float* ks, float* k_mean, float* lse_shift, void* ws, cudaStream_t st);
int launch_quantize4(const Dims& m, const sva_problem_t* p, const void* q, const void* k, void* q4, void* k4,
                     void* q_sf, void* k_sf, float* q_g, float* k_g, void* ws, cudaStream_t st);
int launch_token_move(bool scatter, const void* src, const int64_t ss[3], void* dst, const int64_t sd[3],
                      const int32_t* idx, int B, int H, int M, int n_full, int d, int elem_bytes,
                      int32_t* status, cudaStream_t st);
int launch_attn_simt(const Dims& m, const sva_problem_t* p, const void* q, const void* k,
                     const void* v, const float* qs, const float* ks, const int32_t* row_ptr,
                     const int32_t* col_idx, void* o, float* lse, int32_t* status, cudaStream_t st);
int launch_attn_ts(const Dims& m, const sva_problem_t* p, const void* q, const void* k, const void* v,
                   const float* q_scale, const float* k_scale, const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse, int32_t* status,
                   void* ws, size_t ws_bytes, cudaStream_t st, int remainder_order = -1,
                   const float* block_scores = nullptr);
int launch_attn_ts_fp4(const Dims& m, const sva_problem_t* p, const void* q4, const void* k4, const void* q_sf,
                       const void* k_sf, const float* q_g, const float* k_g, const void* v, const int32_t* row_ptr,
                       const int32_t* col_idx, void* o, float* lse, int32_t* status, void* ws, size_t ws_bytes,
                       cudaStream_t st);
bool attn_ts_fp4_serves(const Dims& m);
size_t attn_ts_workspace_bytes(const Dims& m);
size_t attn_ts_one_call_workspace_bytes(const Dims& m);
size_t attn_ts_remainder_workspace_bytes(const Dims& m, int order);
bool attn_ts_remainder_serves(const Dims& m);
bool attn_ts_serves(const Dims& m);    // d = 128 or 64, bf16 or e4m3 Q/K, 128- or 64-token blocks
int launch_prepare_v_ts(const Dims& m, const sva_problem_t* p, const void* v, void* ws, size_t ws_bytes,
                        cudaStream_t st);

}  // namespace sva
