// Attention prologue in one pass over Q and K: RMS norm over the head dimension, rotary embedding on
// adjacent pairs, bf16 write-back, and -- from the values just written, while the tile is still in
// registers -- the block means the routing needs and (optionally) the e4m3 codes and block scales of the
// FP8 variant.  The paper lists the fused QK-norm + RoPE among its lossless fusion flags; folding the
// pooling and the cast in as well removes the two further reads of Q and K that the separate pooling and
// quantising kernels make.  HBM-bound: 8*d bytes per token per head (10*d with the codes).
//
// One CTA per (block, head, tensor), 256 threads; a thread owns one 16-byte vector (8 elements, 4 rotary
// pairs) of up to PER token rows, the D/8 threads of a row sit in one warp.
#include <type_traits>

#include "common.cuh"

namespace sva {

static constexpr int PT = 256;

struct PrologueParams {
  const uint8_t *q, *k;            // bf16 in
  uint8_t *qo, *ko;                // bf16 out (may be the inputs)
  Strides sq, sk;
  const float *gq, *gk;            // [d] norm weights
  const float *cosn, *sinn;        // [N, d/2]
  float eps;
  float *qbar, *kbar;              // [B,H,Nb,d] block means of the outputs, or null
  uint8_t *q8, *k8;                // e4m3 codes (strides of q / k, in bytes), or null
  float *q_scale, *k_scale;        // [B,H,Nb]
  int H, N, block, Nb;
};

__device__ __forceinline__ uint32_t pack_bf16_rn(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int D, int MAX_ROWS, bool CODES>
__global__ void __launch_bounds__(PT, 3)
prologue_kernel(const PrologueParams prm) {
  constexpr int VPR = D / 8;             // 16-byte vectors per token row
  constexpr int GROUPS = PT / VPR;       // rows in flight
  constexpr int PER = MAX_ROWS / GROUPS; // rows per thread
  constexpr int NB = PER < 4 ? PER : 4;  // rows whose loads are issued together
  __shared__ float part[GROUPS][D + 1];
  __shared__ float red[PT / 32];
  __shared__ float s_scale, s_rcp;
  __shared__ int s_fast;

  const int I = blockIdx.x, bh = blockIdx.y, which = blockIdx.z;
  const int b = bh / prm.H, h = bh % prm.H;
  const Strides s = which ? prm.sk : prm.sq;
  const long long head_off = (long long)b * s.b + (long long)h * s.h;
  // No thread reads what another writes, and a thread reads an element before it writes it (the written
  // value depends on the read one), so "restrict" holds in the sense that matters even when the outputs
  // are the inputs -- and it lets the loads of a batch of rows go out ahead of the earlier rows' stores.
  const uint8_t* __restrict__ src = (which ? prm.k : prm.q) + head_off * 2;
  uint8_t* __restrict__ dst = (which ? prm.ko : prm.qo) + head_off * 2;
  const float* __restrict__ cosn = prm.cosn;
  const float* __restrict__ sinn = prm.sinn;
  const int lo = I * prm.block, cnt = min(prm.block, prm.N - lo);
  const int vec = threadIdx.x % VPR, grp = threadIdx.x / VPR;

  float g[8];
  {
    const float4* gp = reinterpret_cast<const float4*>((which ? prm.gk : prm.gq) + vec * 8);
    const float4 g0 = __ldg(gp), g1 = __ldg(gp + 1);
    g[0] = g0.x; g[1] = g0.y; g[2] = g0.z; g[3] = g0.w; g[4] = g1.x; g[5] = g1.y; g[6] = g1.z; g[7] = g1.w;
  }

  uint4 u[CODES ? PER : 1];              // the finished bf16 rows (kept only for the cast)
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  __nv_bfloat162 am2 = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll
  for (int j0 = 0; j0 < PER; j0 += NB) {
    uint4 in[NB];
    float4 cs[NB], sn[NB];
#pragma unroll
    for (int jj = 0; jj < NB; ++jj) {
      const int t = grp + (j0 + jj) * GROUPS;
      in[jj] = make_uint4(0, 0, 0, 0);
      cs[jj] = make_float4(1.f, 1.f, 1.f, 1.f);
      sn[jj] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (t < cnt) {
        in[jj] = __ldg(reinterpret_cast<const uint4*>(src + (long long)(lo + t) * s.n * 2) + vec);
        cs[jj] = __ldg(reinterpret_cast<const float4*>(cosn + (long long)(lo + t) * (D / 2)) + vec);
        sn[jj] = __ldg(reinterpret_cast<const float4*>(sinn + (long long)(lo + t) * (D / 2)) + vec);
      }
    }
#pragma unroll
    for (int jj = 0; jj < NB; ++jj) {
      const int t = grp + (j0 + jj) * GROUPS;
      const uint32_t w[4] = {in[jj].x, in[jj].y, in[jj].z, in[jj].w};
      float x[8];
#pragma unroll
      for (int e = 0; e < 4; ++e) { x[2 * e] = bf16lo(w[e]); x[2 * e + 1] = bf16hi(w[e]); }
      float ss = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) ss = fmaf(x[e], x[e], ss);
#pragma unroll
      for (int o = VPR / 2; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      const float r = rsqrtf(ss * (1.0f / D) + prm.eps);         // (2 units of error at most: far inside the bf16 rounding)
      const float c[4] = {cs[jj].x, cs[jj].y, cs[jj].z, cs[jj].w}, sv[4] = {sn[jj].x, sn[jj].y, sn[jj].z, sn[jj].w};
      uint32_t out[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float a0 = x[2 * e] * (r * g[2 * e]), a1 = x[2 * e + 1] * (r * g[2 * e + 1]);
        out[e] = pack_bf16_rn(a0 * c[e] - a1 * sv[e], a1 * c[e] + a0 * sv[e]);
      }
      const uint4 o4 = make_uint4(out[0], out[1], out[2], out[3]);
      if (CODES) u[j0 + jj] = o4;
      if (t < cnt) {
        *(reinterpret_cast<uint4*>(dst + (long long)(lo + t) * s.n * 2) + vec) = o4;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          // from what was written, so that routing and the cast see the stored Q, K
          acc[2 * e] += bf16lo(out[e]);
          acc[2 * e + 1] += bf16hi(out[e]);
          if (CODES) am2 = __hmax2(am2, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&out[e])));
        }
      }
    }
  }

  // ---- block means (fixed summation order: rows of a thread in order, then the groups in order)
  if (prm.qbar) {
#pragma unroll
    for (int e = 0; e < 8; ++e) part[grp][vec * 8 + e] = acc[e];
    __syncthreads();
    if (threadIdx.x < D) {
      float sum = 0.f;
#pragma unroll 8
      for (int gidx = 0; gidx < GROUPS; ++gidx) sum += part[gidx][threadIdx.x];
      (which ? prm.kbar : prm.qbar)[((long long)bh * prm.Nb + I) * D + threadIdx.x] = sum / (float)cnt;
    }
  }
  if (!CODES) return;

  // ---- e4m3 codes of the rows just written: absmax scale per block, as the stand-alone quantiser
  float amax = fmaxf(__low2float(am2), __high2float(am2));
#pragma unroll
  for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int i = 0; i < PT / 32; ++i) m = fmaxf(m, red[i]);
    const float sc = m == 0.f ? 1.0f : __fdiv_rn(m, 448.0f);
    s_scale = sc;
    s_rcp = __frcp_rn(sc);
    s_fast = div_fast_ok(sc) ? 1 : 0;
    (which ? prm.k_scale : prm.q_scale)[(long long)bh * prm.Nb + I] = sc;
  }
  __syncthreads();
  const float sc = s_scale, rcp = s_rcp;
  uint8_t* __restrict__ dst8 = (which ? prm.k8 : prm.q8) + head_off;
  auto cast_rows = [&](auto fast_tag) {
    constexpr bool FAST = decltype(fast_tag)::value;
#pragma unroll
    for (int j = 0; j < (CODES ? PER : 1); ++j) {
      const int t = grp + j * GROUPS;
      if (t >= cnt) continue;
      const uint32_t w[4] = {u[j].x, u[j].y, u[j].z, u[j].w};
      uint32_t c[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float x0 = bf16lo(w[e]), x1 = bf16hi(w[e]);
        c[e] = FAST ? e4m3x2(div_fast(x0, sc, rcp), div_fast(x1, sc, rcp))
                    : e4m3x2(__fdiv_rn(x0, sc), __fdiv_rn(x1, sc));
      }
      *reinterpret_cast<uint2*>(dst8 + (long long)(lo + t) * s.n + vec * 8) =
          make_uint2(__byte_perm(c[0], c[1], 0x5410), __byte_perm(c[2], c[3], 0x5410));
    }
  };
  if (s_fast) cast_rows(std::true_type{}); else cast_rows(std::false_type{});
}

int launch_prologue(const Dims& m, const sva_problem_t* p, const void* q, const void* k, const float* gq,
                    const float* gk, const float* cosn, const float* sinn, float eps, void* qo, void* ko,
                    float* qbar, float* kbar, void* q8, void* k8, float* qs, float* ks, cudaStream_t st) {
  if (!((m.d == 128 || m.d == 64) && m.block <= 128)) return SVA_ERR_UNSUPPORTED;
  PrologueParams prm;
  prm.q = (const uint8_t*)q; prm.k = (const uint8_t*)k; prm.qo = (uint8_t*)qo; prm.ko = (uint8_t*)ko;
  prm.sq = make_strides(p->q_stride); prm.sk = make_strides(p->k_stride);
  prm.gq = gq; prm.gk = gk; prm.cosn = cosn; prm.sinn = sinn; prm.eps = eps;
  prm.qbar = qbar; prm.kbar = kbar; prm.q8 = (uint8_t*)q8; prm.k8 = (uint8_t*)k8; prm.q_scale = qs; prm.k_scale = ks;
  prm.H = m.H; prm.N = m.N; prm.block = m.block; prm.Nb = m.Nb;
  dim3 g(m.Nb, m.B * m.H, 2);
  const bool codes = q8 != nullptr;
  if (m.d == 128) {
    if (codes) prologue_kernel<128, 128, true><<<g, PT, 0, st>>>(prm);
    else prologue_kernel<128, 128, false><<<g, PT, 0, st>>>(prm);
  } else {
    if (codes) prologue_kernel<64, 128, true><<<g, PT, 0, st>>>(prm);
    else prologue_kernel<64, 128, false><<<g, PT, 0, st>>>(prm);
  }
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

}  // namespace sva
