// FP8 variant's quantiser: one absmax scale per (b, h, block), e4m3 codes.
// One CTA per (block, head, tensor) keeps its 128 x d bf16 tile in registers between the
// absmax pass and the cast, so Q and K are read once and written once (HBM-bound).
#include "common.cuh"

namespace sva {

static constexpr int QT = 256;

template <int D, int MAX_ROWS>
__global__ void __launch_bounds__(QT)
quantize_kernel(const uint8_t* __restrict__ q, const uint8_t* __restrict__ k, Strides sq, Strides sk,
                uint8_t* __restrict__ q8, uint8_t* __restrict__ k8, float* __restrict__ q_scale,
                float* __restrict__ k_scale, int H, int N, int block, int Nb) {
  constexpr int VPR = D / 8;             // 16-byte vectors (8 bf16) per token row
  constexpr int GROUPS = QT / VPR;
  constexpr int PER = MAX_ROWS / GROUPS; // rows per thread
  __shared__ float red[QT / 32];
  __shared__ float s_scale;

  const int I = blockIdx.x, bh = blockIdx.y, which = blockIdx.z;
  const int b = bh / H, h = bh % H;
  const Strides s = which ? sk : sq;
  const long long head_off = (long long)b * s.b + (long long)h * s.h;
  const uint8_t* src = (which ? k : q) + head_off * 2;
  uint8_t* dst = (which ? k8 : q8) + head_off;
  const int lo = I * block, cnt = min(block, N - lo);
  const int vec = threadIdx.x % VPR, grp = threadIdx.x / VPR;

  uint4 u[PER];
  float a = 0.f;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    int t = grp + j * GROUPS;
    u[j] = make_uint4(0, 0, 0, 0);
    if (t < cnt) u[j] = __ldg(reinterpret_cast<const uint4*>(src + (long long)(lo + t) * s.n * 2) + vec);
    const uint32_t w[4] = {u[j].x, u[j].y, u[j].z, u[j].w};
#pragma unroll
    for (int e = 0; e < 4; ++e) a = fmaxf(a, fmaxf(fabsf(bf16lo(w[e])), fabsf(bf16hi(w[e]))));
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int i = 0; i < QT / 32; ++i) m = fmaxf(m, red[i]);
    float sc = m == 0.f ? 1.0f : __fdiv_rn(m, 448.0f);
    s_scale = sc;
    (which ? k_scale : q_scale)[(long long)bh * Nb + I] = sc;
  }
  __syncthreads();
  const float sc = s_scale;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    int t = grp + j * GROUPS;
    if (t >= cnt) continue;
    const uint32_t w[4] = {u[j].x, u[j].y, u[j].z, u[j].w};
    uint32_t out[2] = {0, 0};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      uint32_t c0 = __nv_cvt_float_to_fp8(__fdiv_rn(bf16lo(w[e]), sc), __NV_SATFINITE, __NV_E4M3);
      uint32_t c1 = __nv_cvt_float_to_fp8(__fdiv_rn(bf16hi(w[e]), sc), __NV_SATFINITE, __NV_E4M3);
      out[e >> 1] |= (c0 | (c1 << 8)) << (16 * (e & 1));
    }
    *reinterpret_cast<uint2*>(dst + (long long)(lo + t) * s.n + vec * 8) = make_uint2(out[0], out[1]);
  }
}

int launch_quantize(const Dims& m, const sva_problem_t* p, const void* q, const void* k, void* q8,
                    void* k8, float* qs, float* ks, cudaStream_t st) {
  dim3 g(m.Nb, m.B * m.H, 2);
  Strides sq = make_strides(p->q_stride), sk = make_strides(p->k_stride);
  if (m.d == 128 && m.block <= 128)
    quantize_kernel<128, 128><<<g, QT, 0, st>>>((const uint8_t*)q, (const uint8_t*)k, sq, sk, (uint8_t*)q8,
                                                (uint8_t*)k8, qs, ks, m.H, m.N, m.block, m.Nb);
  else if (m.d == 64 && m.block <= 128)
    quantize_kernel<64, 128><<<g, QT, 0, st>>>((const uint8_t*)q, (const uint8_t*)k, sq, sk, (uint8_t*)q8,
                                               (uint8_t*)k8, qs, ks, m.H, m.N, m.block, m.Nb);
  else
    return SVA_ERR_UNSUPPORTED;
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

}  // namespace sva
