// Diagnostic block-sparse attention on CUDA cores (fp32 FMA, no tensor cores, no TMA).
// Same contract as the tensor-core kernel; it is the on-device cross-check for it.
// One CTA per query block; two threads per query row (each owns half of d); K and V tiles of
// one kept block at a time in shared memory as fp32; online softmax one key at a time.
#include "common.cuh"

namespace sva {

template <int D>
__global__ void __launch_bounds__(256)
attn_simt_kernel(const uint8_t* __restrict__ q, const uint8_t* __restrict__ k,
                 const __nv_bfloat16* __restrict__ v, Strides sq, Strides sk, Strides sv, Strides so,
                 const float* __restrict__ q_scale, const float* __restrict__ k_scale,
                 const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
                 __nv_bfloat16* __restrict__ o, float* __restrict__ lse, int32_t* __restrict__ status,
                 int H, int N, int block, int Nb, float scale, int fp8) {
  constexpr int HALF = D / 2;
  extern __shared__ float sm[];
  float* ks = sm;                    // [block][D]
  float* vs = sm + (size_t)block * D;

  const int r = blockIdx.x;
  const int bh = r / Nb, I = r % Nb;
  const int b = bh / H, h = bh % H;
  const int row = threadIdx.x >> 1, half = threadIdx.x & 1;
  const int qi = I * block + row;
  const bool q_ok = row < block && qi < N;

  float qr[HALF], acc[HALF];
#pragma unroll
  for (int c = 0; c < HALF; ++c) { qr[c] = 0.f; acc[c] = 0.f; }
  if (q_ok) {
    long long off = (long long)b * sq.b + (long long)h * sq.h + (long long)qi * sq.n + half * HALF;
    if (fp8) {
      float s = q_scale[(long long)bh * Nb + I];
#pragma unroll
      for (int c = 0; c < HALF; ++c) qr[c] = e4m3_to_float(q[off + c]) * s;
    } else {
      const __nv_bfloat16* qp = reinterpret_cast<const __nv_bfloat16*>(q) + off;
#pragma unroll
      for (int c = 0; c < HALF; ++c) qr[c] = __bfloat162float(qp[c]);
    }
  }
  float m = -INFINITY, l = 0.f;

  int beg, end;
  if (row_ptr) { beg = row_ptr[r]; end = row_ptr[r + 1]; } else { beg = 0; end = Nb; }
  if (beg < 0 || end < beg || end - beg > Nb || (row_ptr && end > row_ptr[gridDim.x])) {
    // corrupt row (not monotone, too long, or reaching beyond the row_ptr[R] entries the CSR says it has):
    // report, read no entry, write the empty-row result
    if (threadIdx.x == 0 && status) atomicOr(status, SVA_DEV_BAD_INDEX);
    end = beg;
  }
  for (int e = beg; e < end; ++e) {
    const int J = row_ptr ? col_idx[e] : e;
    if (J < 0 || J >= Nb) {
      if (threadIdx.x == 0 && status) atomicOr(status, SVA_DEV_BAD_INDEX);
      continue;
    }
    const int nkeys = min(block, N - J * block);
    __syncthreads();
    const float kscale = fp8 ? k_scale[(long long)bh * Nb + J] : 1.f;
    for (int i = threadIdx.x; i < nkeys * D; i += blockDim.x) {
      int t = i / D, c = i % D;
      long long tok = J * block + t;
      long long ko = (long long)b * sk.b + (long long)h * sk.h + tok * sk.n + c;
      ks[i] = fp8 ? e4m3_to_float(k[ko]) * kscale
                  : __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(k)[ko]);
      vs[i] = __bfloat162float(v[(long long)b * sv.b + (long long)h * sv.h + tok * sv.n + c]);
    }
    __syncthreads();
    for (int t = 0; t < nkeys; ++t) {
      const float* kr = ks + t * D + half * HALF;
      float s = 0.f;
#pragma unroll
      for (int c = 0; c < HALF; ++c) s = fmaf(qr[c], kr[c], s);
      s += __shfl_xor_sync(0xffffffffu, s, 1);
      s *= scale;
      const float mn = fmaxf(m, s);
      const float alpha = __expf(m - mn);      // m = -inf at the first key -> 0
      const float pw = __expf(s - mn);
      l = l * alpha + pw;
      const float* vr = vs + t * D + half * HALF;
#pragma unroll
      for (int c = 0; c < HALF; ++c) acc[c] = fmaf(acc[c], alpha, pw * vr[c]);
      m = mn;
    }
  }
  if (q_ok) {
    const float inv = l > 0.f ? 1.f / l : 0.f;
    __nv_bfloat16* op = o + (long long)b * so.b + (long long)h * so.h + (long long)qi * so.n + half * HALF;
#pragma unroll
    for (int c = 0; c < HALF; ++c) op[c] = __float2bfloat16_rn(acc[c] * inv);
    if (lse && half == 0) lse[(long long)bh * N + qi] = l > 0.f ? m + logf(l) : -INFINITY;
  }
}

int launch_attn_simt(const Dims& m, const sva_problem_t* p, const void* q, const void* k,
                     const void* v, const float* qs, const float* ks, const int32_t* row_ptr,
                     const int32_t* col_idx, void* o, float* lse, int32_t* status, cudaStream_t st) {
  if (m.block > 128) return SVA_ERR_UNSUPPORTED;
  size_t smem = (size_t)2 * m.block * m.d * sizeof(float);
  Strides sq = make_strides(p->q_stride), sk = make_strides(p->k_stride),
          sv = make_strides(p->v_stride), so = make_strides(p->o_stride);
#define SVA_SIMT_LAUNCH(DD)                                                                       \
  do {                                                                                            \
    if (cudaFuncSetAttribute(attn_simt_kernel<DD>, cudaFuncAttributeMaxDynamicSharedMemorySize,  \
                             (int)smem) != cudaSuccess)                                           \
      return SVA_ERR_CUDA;                                                                        \
    attn_simt_kernel<DD><<<m.R, 256, smem, st>>>(                                                  \
        (const uint8_t*)q, (const uint8_t*)k, (const __nv_bfloat16*)v, sq, sk, sv, so, qs, ks,   \
        row_ptr, col_idx, (__nv_bfloat16*)o, lse, status, m.H, m.N, m.block, m.Nb, m.scale,      \
        m.fp8 ? 1 : 0);                                                                           \
  } while (0)
  if (m.d == 128) SVA_SIMT_LAUNCH(128);
  else if (m.d == 64) SVA_SIMT_LAUNCH(64);
  else return SVA_ERR_UNSUPPORTED;
#undef SVA_SIMT_LAUNCH
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

}  // namespace sva
