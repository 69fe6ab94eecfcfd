// Block-scaled 4-bit quantiser for Q and K (the paper's quantisation format is NVFP4; it prints no formula).
// Per (b, h): tensor scale g = amax / (6 * 448) (1 if amax = 0).  Per token and 16 consecutive elements of the
// head dimension: sf = e4m3((amax_block / 6) / g), code = e2m1(x / (value(sf) * g)), both round-to-nearest-even
// and saturating; every scalar step is one fp32 operation rounded to nearest, so the bytes are reproducible.
//
// Output layout, chosen for the block-scaled tensor-core MMA that consumes it:
//   codes   [B*H][Nb*128 tokens][64 bytes]   two codes per byte (even element in the low nibble), rows >= N zero
//   scales  [B*H][Nb][2][32][4][4] bytes     per 128-token block and half of the head dimension (64 elements = 4
//                                            scale blocks) one 512-byte group: byte ((t % 32) * 4 + t / 32) * 4 + kb
//                                            holds the scale of token t (within the block), scale block kb -- the
//                                            order in which a 32-lane x 128-bit copy into tensor memory wants them
// Two kernels: the per-(b,h) amax (an integer atomicMax on the non-negative fp32 bit pattern), then the cast.
#include <cuda_fp4.h>

#include "common.cuh"

namespace sva {

static constexpr int Q4_THREADS = 256;

// amax[tensor * BH + bh] (as fp32 bits; the launcher zeroes it) = max |x| over the existing tokens
__global__ void __launch_bounds__(Q4_THREADS)
amax_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k, Strides sq, Strides sk, int H, int N,
            int BH, uint32_t* __restrict__ amax) {
  const int I = blockIdx.x, bh = blockIdx.y, which = blockIdx.z;
  const Strides s = which ? sk : sq;
  const __nv_bfloat16* base = (which ? k : q) + (long long)(bh / H) * s.b + (long long)(bh % H) * s.h;
  const int lo = I * 128, cnt = min(128, N - lo);
  uint32_t m = 0u;                                            // max of the |x| bit patterns (bf16 in the upper half)
  uint4 u[8];                                                 // 16 vectors of 8 elements per token: 8 loads in flight per thread
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const int i = threadIdx.x + r * Q4_THREADS;
    u[r] = make_uint4(0u, 0u, 0u, 0u);
    if (i < cnt * 16) u[r] = __ldg(reinterpret_cast<const uint4*>(base + (long long)(lo + (i >> 4)) * s.n) + (i & 15));
  }
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const uint32_t w[4] = {u[r].x, u[r].y, u[r].z, u[r].w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      m = max(m, (w[e] << 16) & 0x7fffffffu);
      m = max(m, w[e] & 0x7fff0000u);
    }
  }
  m = __reduce_max_sync(0xffffffffu, m);
  if ((threadIdx.x & 31) == 0 && m) atomicMax(amax + which * BH + bh, m);
}

// One CTA per (128-token block, head, tensor); a thread casts one 16-element scale block at a time.
__global__ void __launch_bounds__(Q4_THREADS)
quantize4_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k, Strides sq, Strides sk, int H,
                 int N, int Nb, int BH, const uint32_t* __restrict__ amax, uint8_t* __restrict__ q4,
                 uint8_t* __restrict__ k4, uint8_t* __restrict__ q_sf, uint8_t* __restrict__ k_sf, float* __restrict__ q_g,
                 float* __restrict__ k_g) {
  const int I = blockIdx.x, bh = blockIdx.y, which = blockIdx.z;
  const Strides s = which ? sk : sq;
  const __nv_bfloat16* base = (which ? k : q) + (long long)(bh / H) * s.b + (long long)(bh % H) * s.h;
  uint8_t* codes = (which ? k4 : q4) + ((long long)bh * Nb + I) * 128 * 64;
  uint8_t* sfo = (which ? k_sf : q_sf) + ((long long)bh * Nb + I) * 1024;
  const float am = __uint_as_float(__ldg(amax + which * BH + bh));
  const float g = am > 0.f ? __fdiv_rn(am, 2688.0f) : 1.0f;
  if (I == 0 && threadIdx.x == 0) (which ? k_g : q_g)[bh] = g;
  const int lo = I * 128;
  for (int i = threadIdx.x; i < 128 * 8; i += Q4_THREADS) {
    const int t = i >> 3, kb = i & 7;                         // token of the block, scale block of the token
    uint32_t w[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    uint8_t sf = 0;
    uint2 out = make_uint2(0u, 0u);
    if (lo + t < N) {
      const uint4* src = reinterpret_cast<const uint4*>(base + (long long)(lo + t) * s.n + kb * 16);
      const uint4 u0 = __ldg(src), u1 = __ldg(src + 1);
      w[0] = u0.x; w[1] = u0.y; w[2] = u0.z; w[3] = u0.w; w[4] = u1.x; w[5] = u1.y; w[6] = u1.z; w[7] = u1.w;
      float a = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) a = fmaxf(a, fmaxf(fabsf(bf16lo(w[e])), fabsf(bf16hi(w[e]))));
      const float u = __fdiv_rn(__fdiv_rn(a, 6.0f), g);
      sf = (uint8_t)__nv_cvt_float_to_fp8(u, __NV_SATFINITE, __NV_E4M3);
      const float sd = e4m3_to_float(sf);
      if (sd > 0.f) {
        const float sc = __fmul_rn(sd, g);
        // x / sc: the correctly rounded quotient from one reciprocal per scale block (div_fast), a true
        // division where that sequence is not exact
        const bool fast = div_fast_ok(sc);
        const float rc = __frcp_rn(sc);
        uint32_t pk[2] = {0u, 0u};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float x0 = bf16lo(w[e]), x1 = bf16hi(w[e]);
          const float2 y = fast ? make_float2(div_fast(x0, sc, rc), div_fast(x1, sc, rc))
                                : make_float2(__fdiv_rn(x0, sc), __fdiv_rn(x1, sc));
          const uint32_t byte = (uint32_t)__nv_cvt_float2_to_fp4x2(y, __NV_E2M1, cudaRoundNearest);
          pk[e >> 2] |= (byte & 0xffu) << (8 * (e & 3));
        }
        out = make_uint2(pk[0], pk[1]);
      } else {
        sf = 0;
      }
    }
    *reinterpret_cast<uint2*>(codes + t * 64 + kb * 8) = out;
    sfo[(kb >> 2) * 512 + ((t & 31) * 4 + (t >> 5)) * 4 + (kb & 3)] = sf;
  }
}

int launch_quantize4(const Dims& m, const sva_problem_t* p, const void* q, const void* k, void* q4, void* k4,
                     void* q_sf, void* k_sf, float* q_g, float* k_g, void* ws, cudaStream_t st) {
  if (m.d != 128 || m.block != 128) return SVA_ERR_UNSUPPORTED;
  const int BH = m.B * m.H;
  uint32_t* amax = static_cast<uint32_t*>(ws);
  if (cudaMemsetAsync(amax, 0, (size_t)2 * BH * sizeof(uint32_t), st) != cudaSuccess) return SVA_ERR_CUDA;
  const Strides sq = make_strides(p->q_stride), sk = make_strides(p->k_stride);
  dim3 grid(m.Nb, BH, 2);
  amax_kernel<<<grid, Q4_THREADS, 0, st>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, sq, sk, m.H, m.N, BH, amax);
  if (cudaGetLastError() != cudaSuccess) return SVA_ERR_CUDA;
  quantize4_kernel<<<grid, Q4_THREADS, 0, st>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, sq, sk, m.H, m.N, m.Nb, BH,
                                                amax, (uint8_t*)q4, (uint8_t*)k4, (uint8_t*)q_sf, (uint8_t*)k_sf, q_g, k_g);
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

}  // namespace sva
