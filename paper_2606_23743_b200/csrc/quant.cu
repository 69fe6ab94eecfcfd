// FP8 variant's quantiser: one absmax scale per (b, h, block), e4m3 codes.
// One CTA per (block, head, tensor) keeps its 128 x d bf16 tile in registers between the
// absmax pass and the cast, so Q and K are read once and written once (HBM-bound).
// With K smoothing, two small kernels first reduce K to its mean key per (b, h) -- per-block sums
// in a fixed order, then the blocks in index order, so the mean is reproducible -- and the
// quantiser subtracts it from K in fp32 and writes scale * <q_i, mean> per query token.
#include <type_traits>

#include "common.cuh"

namespace sva {

static constexpr int QT = 256;

// part[(bh*Nb + I)*D + c] = sum over the valid tokens of block I of k[.., c]   (grid Nb x BH)
template <int D>
__global__ void __launch_bounds__(QT)
block_sum_kernel(const uint8_t* __restrict__ k, Strides sk, float* __restrict__ part, int H, int N, int block, int Nb) {
  constexpr int VPR = D / 8, GROUPS = QT / VPR;
  __shared__ float acc[GROUPS][D];
  const int I = blockIdx.x, bh = blockIdx.y;
  const uint8_t* src = k + ((long long)(bh / H) * sk.b + (long long)(bh % H) * sk.h) * 2;
  const int lo = I * block, cnt = min(block, N - lo);
  const int vec = threadIdx.x % VPR, grp = threadIdx.x / VPR;
  float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int t = grp; t < cnt; t += GROUPS) {
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(src + (long long)(lo + t) * sk.n * 2) + vec);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) { a[2 * e] += bf16lo(w[e]); a[2 * e + 1] += bf16hi(w[e]); }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[grp][vec * 8 + e] = a[e];
  __syncthreads();
  for (int c = threadIdx.x; c < D; c += QT) {
    float t = 0.f;
    for (int g = 0; g < GROUPS; ++g) t += acc[g][c];
    part[((long long)bh * Nb + I) * D + c] = t;
  }
}

// mean[bh*D + c] = (sum over blocks, in index order) / N                        (grid BH, D threads)
__global__ void mean_key_kernel(const float* __restrict__ part, float* __restrict__ mean, int Nb, int D, int N) {
  const int bh = blockIdx.x, c = threadIdx.x;
  const float* src = part + (long long)bh * Nb * D + c;
  float t = 0.f;
  int I = 0;
  for (; I + 16 <= Nb; I += 16) {          // 16 loads in flight; the order of the sum stays the index order
    float v[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) v[e] = __ldg(src + (long long)(I + e) * D);
#pragma unroll
    for (int e = 0; e < 16; ++e) t += v[e];
  }
  for (; I < Nb; ++I) t += __ldg(src + (long long)I * D);
  mean[(long long)bh * D + c] = __fdiv_rn(t, (float)N);
}

// SMOOTH: the K smoothing variant (k_mean given).
template <int D, int MAX_ROWS, bool SMOOTH>
__global__ void __launch_bounds__(QT)
quantize_kernel(const uint8_t* __restrict__ q, const uint8_t* __restrict__ k, Strides sq, Strides sk,
                uint8_t* __restrict__ q8, uint8_t* __restrict__ k8, float* __restrict__ q_scale,
                float* __restrict__ k_scale, int H, int N, int block, int Nb,
                const float* __restrict__ k_mean, float* __restrict__ lse_shift, float scale) {
  constexpr int VPR = D / 8;             // 16-byte vectors (8 bf16) per token row
  constexpr int GROUPS = QT / VPR;
  constexpr int PER = MAX_ROWS / GROUPS; // rows per thread
  __shared__ float red[QT / 32];
  __shared__ float s_scale, s_rcp;
  __shared__ int s_fast;

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
  // K smoothing: this thread's 8 components of the head's mean key (K: subtracted; Q: dotted)
  float mk[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (SMOOTH) {
    const float4* mp = reinterpret_cast<const float4*>(k_mean + (long long)bh * D + vec * 8);
    const float4 m0 = __ldg(mp), m1 = __ldg(mp + 1);
    mk[0] = m0.x; mk[1] = m0.y; mk[2] = m0.z; mk[3] = m0.w; mk[4] = m1.x; mk[5] = m1.y; mk[6] = m1.z; mk[7] = m1.w;
  }
  const bool sub = SMOOTH && which == 1;
  __nv_bfloat162 am2 = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll
  for (int j = 0; j < PER; ++j) {          // all loads first: nothing below stands between them
    int t = grp + j * GROUPS;
    u[j] = make_uint4(0, 0, 0, 0);
    if (t < cnt) u[j] = __ldg(reinterpret_cast<const uint4*>(src + (long long)(lo + t) * s.n * 2) + vec);
  }
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    int t = grp + j * GROUPS;
    const uint32_t w[4] = {u[j].x, u[j].y, u[j].z, u[j].w};
    if (sub) {
      if (t < cnt) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          a = fmaxf(a, fmaxf(fabsf(__fsub_rn(bf16lo(w[e]), mk[2 * e])), fabsf(__fsub_rn(bf16hi(w[e]), mk[2 * e + 1]))));
      }
    } else {
      // |.| and max on the packed pairs; folded into `a` after the loop
#pragma unroll
      for (int e = 0; e < 4; ++e) am2 = __hmax2(am2, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[e])));
    }
    if (SMOOTH && which == 0 && lse_shift) {
      // scale * <q_t, mean>: 8 products here, the rest of the row in the other VPR-1 lanes of the group
      float dot = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) dot += bf16lo(w[e]) * mk[2 * e] + bf16hi(w[e]) * mk[2 * e + 1];
#pragma unroll
      for (int o = VPR / 2; o; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      if (vec == 0 && t < cnt) lse_shift[(long long)bh * N + lo + t] = dot * scale;
    }
  }
  a = fmaxf(a, fmaxf(__low2float(am2), __high2float(am2)));
#pragma unroll
  for (int o = 16; o; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int i = 0; i < QT / 32; ++i) m = fmaxf(m, red[i]);
    float sc = m == 0.f ? 1.0f : __fdiv_rn(m, 448.0f);
    s_scale = sc;
    s_rcp = __frcp_rn(sc);
    s_fast = div_fast_ok(sc) ? 1 : 0;
    (which ? k_scale : q_scale)[(long long)bh * Nb + I] = sc;
  }
  __syncthreads();
  const float sc = s_scale, rcp = s_rcp;
  // (one loop per division method, chosen per block, so that the common case carries no trace of the other)
  auto cast_rows = [&](auto fast_tag) {
    constexpr bool FAST = decltype(fast_tag)::value;
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      int t = grp + j * GROUPS;
      if (t >= cnt) continue;
      const uint32_t w[4] = {u[j].x, u[j].y, u[j].z, u[j].w};
      uint32_t c[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float x0 = sub ? __fsub_rn(bf16lo(w[e]), mk[2 * e]) : bf16lo(w[e]);
        const float x1 = sub ? __fsub_rn(bf16hi(w[e]), mk[2 * e + 1]) : bf16hi(w[e]);
        c[e] = FAST ? e4m3x2(div_fast(x0, sc, rcp), div_fast(x1, sc, rcp))
                    : e4m3x2(__fdiv_rn(x0, sc), __fdiv_rn(x1, sc));
      }
      *reinterpret_cast<uint2*>(dst + (long long)(lo + t) * s.n + vec * 8) =
          make_uint2(__byte_perm(c[0], c[1], 0x5410), __byte_perm(c[2], c[3], 0x5410));
    }
  };
  if (s_fast) cast_rows(std::true_type{}); else cast_rows(std::false_type{});
}

size_t smooth_workspace_bytes(const Dims& m) { return (size_t)m.B * m.H * m.Nb * m.d * sizeof(float); }

// k_mean == nullptr: the plain quantiser.  Otherwise K smoothing: k_mean [B,H,d] is computed here (ws holds
// the per-block sums), subtracted from K before the cast, and lse_shift (optional) [B,H,N] is written.
int launch_quantize(const Dims& m, const sva_problem_t* p, const void* q, const void* k, void* q8,
                    void* k8, float* qs, float* ks, float* k_mean, float* lse_shift, void* ws, cudaStream_t st) {
  dim3 g(m.Nb, m.B * m.H, 2);
  Strides sq = make_strides(p->q_stride), sk = make_strides(p->k_stride);
  if (!((m.d == 128 || m.d == 64) && m.block <= 128)) return SVA_ERR_UNSUPPORTED;
  if (k_mean) {
    dim3 g1(m.Nb, m.B * m.H);
    if (m.d == 128)
      block_sum_kernel<128><<<g1, QT, 0, st>>>((const uint8_t*)k, sk, (float*)ws, m.H, m.N, m.block, m.Nb);
    else
      block_sum_kernel<64><<<g1, QT, 0, st>>>((const uint8_t*)k, sk, (float*)ws, m.H, m.N, m.block, m.Nb);
    if (cudaGetLastError() != cudaSuccess) return SVA_ERR_CUDA;
    mean_key_kernel<<<m.B * m.H, m.d, 0, st>>>((const float*)ws, k_mean, m.Nb, m.d, m.N);
    if (cudaGetLastError() != cudaSuccess) return SVA_ERR_CUDA;
  }
#define SVA_QUANT_LAUNCH(DD, SM)                                                                            \
  quantize_kernel<DD, 128, SM><<<g, QT, 0, st>>>((const uint8_t*)q, (const uint8_t*)k, sq, sk, (uint8_t*)q8, \
                                                 (uint8_t*)k8, qs, ks, m.H, m.N, m.block, m.Nb, k_mean, lse_shift, m.scale)
  if (m.d == 128) { if (k_mean) SVA_QUANT_LAUNCH(128, true); else SVA_QUANT_LAUNCH(128, false); }
  else { if (k_mean) SVA_QUANT_LAUNCH(64, true); else SVA_QUANT_LAUNCH(64, false); }
#undef SVA_QUANT_LAUNCH
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

}  // namespace sva
