// First-order term of the approximate remainder (the paper's "first-order Taylor" compensation of dropped
// blocks, as this build reads it): for a query block I
//     T_i = scale * A_I^T q_i,   A_I = sum_{J dropped by I} exp(sbar_IJ) C_J,   C_J = sum_{j in J} (k_j - kbar_J) v_j^T,
// one d x d matrix per query block.  Three kernels prepare A_I for the attention kernel, which then treats it as one
// more tile of the row (its "P" are the scaled query values, its "V" is A_I -- or, for the attention kernel that runs
// on a transposed copy of V, its "V^T" is A_I^T; the kernels below are written for the transposed form and produce
// the other one when the launcher hands the covariance kernel K and V in each other's place):
//   cov_kernel        C_J^T = V_J^T K_J - n_J vbar_J kbar_J^T per key block: one 128 x 128 x block tcgen05 MMA, both
//                     operands read where they lie (MN-major), the rank-one centring in the epilogue; bf16 out
//   weights_kernel    W[I][J] = exp(sbar_IJ - mu_I) for the dropped J (0 for the kept ones), mu_I = their maximum
//   aggregate_kernel  A_I^T = sum_J W[I][J] C_J^T: per head a [Nb x Nb] x [Nb x d*d] GEMM on tcgen05
// All waits are bounded (tc_ptx.cuh); a wait that runs out sets SVA_DEV_TIMEOUT and the CTA leaves.
#include "tc_ptx.cuh"

namespace sva {

namespace rem {
constexpr int D = 128;
constexpr int TILE = BS * D * 2;                  // 32 KB: 128 rows x 256 bytes as two 128-byte panels
}

// ------------------------------------------------------------------ C_J^T
// grid (Nb, B*H), 128 threads.  Shared memory: K tile, V tile ([keys][d] as two 64-element panels, 128-byte swizzle).
__global__ void __launch_bounds__(128)
cov_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, int H, int N, int block,
           int Nb, __nv_bfloat16* __restrict__ ct, int32_t* __restrict__ status) {
  using namespace rem;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  __shared__ __align__(8) unsigned long long bars[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  __shared__ float kb_s[D], vb_s[D];
  volatile int* abort_flag = &abort_s;
  const uint32_t bar_full = smem_u32(&bars[0]), bar_mma = smem_u32(&bars[1]);
  const int J = blockIdx.x, bh = blockIdx.y, hh = bh % H, bb = bh / H;
  const int warp = threadIdx.x >> 5;
  const int cnt = min(block, N - J * block);
  const uint32_t panel = (uint32_t)block * 128u;             // bytes of one 64-element panel of the tile
  if (threadIdx.x == 0) {
    mbar_init(bar_full, 1);
    mbar_init(bar_mma, 1);
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(128u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  if (threadIdx.x == 0) {
    mbar_expect_tx(bar_full, 4u * panel);
    tma_load_4d(sbase, &tm_k, bar_full, 0, J * block, hh, bb);
    tma_load_4d(sbase + panel, &tm_k, bar_full, 64, J * block, hh, bb);
    tma_load_4d(sbase + TILE, &tm_v, bar_full, 0, J * block, hh, bb);
    tma_load_4d(sbase + TILE + panel, &tm_v, bar_full, 64, J * block, hh, bb);
  }
  bool ok = mbar_wait(bar_full, 0u, abort_flag, status);
  if (ok) {
    // column means of the two tiles: thread c owns column c (rows beyond N arrive as zeros)
    const int c = threadIdx.x;
    const uint8_t* kp = smem + (c >> 6) * panel;
    const uint8_t* vp = smem + TILE + (c >> 6) * panel;
    const int chunk = (c & 63) >> 3, within = (c & 7) * 2;
    float sk = 0.f, sv = 0.f;
    for (int j = 0; j < cnt; ++j) {
      const int off = j * 128 + ((chunk ^ (j & 7)) << 4) + within;
      sk += __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(kp + off));
      sv += __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(vp + off));
    }
    kb_s[c] = sk / (float)cnt;
    vb_s[c] = sv / (float)cnt;
    if (threadIdx.x == 0) {
      // D[e][c] = sum_j V[j][e] K[j][c]: A = V^T and B = K^T, both MN-major from the tiles as they lie
      tc_fence_after();
      const uint32_t idesc = instr_desc(128, 128, 1, true) | (1u << 15);
      const uint64_t ad = smem_desc(sbase + TILE, panel, 1024), bd = smem_desc(sbase, panel, 1024);
      for (int kk = 0; kk < block / 16; ++kk)
        tc_mma_ss_bf16(tmem_base, ad + (uint64_t)(kk * 128), bd + (uint64_t)(kk * 128), idesc, kk > 0 ? 1u : 0u);
      tc_commit(bar_mma, 1u);
    }
  }
  __syncthreads();
  ok = ok && mbar_wait(bar_mma, 0u, abort_flag, status);
  if (ok) {
    tc_fence_after();
    const int e = threadIdx.x;                                // TMEM lane = row e of C_J^T
    const float nv = (float)cnt * vb_s[e];
    __nv_bfloat16* dst = ct + (((long long)bh * Nb + J) * D + e) * D;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
    for (int c0 = 0; c0 < D; c0 += 32) {
      uint32_t v[32];
      tmem_ld32(lane_addr + c0, v);
      tc_wait_ld();
      uint32_t o[16];
#pragma unroll
      for (int t = 0; t < 32; t += 2)
        o[t >> 1] = pack_bf16(__uint_as_float(v[t]) - nv * kb_s[c0 + t], __uint_as_float(v[t + 1]) - nv * kb_s[c0 + t + 1]);
#pragma unroll
      for (int t = 0; t < 4; ++t)
        *reinterpret_cast<uint4*>(dst + c0 + 8 * t) = make_uint4(o[4 * t], o[4 * t + 1], o[4 * t + 2], o[4 * t + 3]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128u) : "memory");
  }
}

// ------------------------------------------------------------------ W and mu
// One warp per CSR row: W[r][J] (bf16, Nbw columns, zero beyond Nb and for kept J), mu[r].
__global__ void __launch_bounds__(256)
weights_kernel(const float* __restrict__ scores, const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx,
               int R, int Nb, int Nbw, __nv_bfloat16* __restrict__ w, float* __restrict__ mu) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (r >= R) return;
  const float* srow = scores + (long long)r * Nb;
  const int nnz = __ldg(row_ptr + R);
  int cb = __ldg(row_ptr + r), ce = __ldg(row_ptr + r + 1);
  if (cb < 0 || ce < cb || ce - cb > Nb || ce > nnz) ce = cb;          // corrupt pair: treated as keeping nothing
  // first pass: the maximum over the dropped blocks (the row's kept list is ascending: walk it alongside)
  float mx = -INFINITY;
  for (int J0 = 0; J0 < Nb; J0 += 32) {
    const int J = J0 + lane;
    bool kept = false;
    for (int t = cb; t < ce; ++t) kept |= (__ldg(col_idx + t) == J);
    const float s = J < Nb ? __ldg(srow + J) : -INFINITY;
    if (!kept) mx = fmaxf(mx, s);
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  const bool none = mx == -INFINITY;                                      // nothing dropped
  for (int J0 = 0; J0 < Nbw; J0 += 32) {
    const int J = J0 + lane;
    bool kept = J >= Nb;
    for (int t = cb; t < ce; ++t) kept |= (__ldg(col_idx + t) == J);
    float x = 0.f;
    if (!kept && !none) x = __expf(__ldg(srow + J) - mx);
    if (J < Nbw) w[(long long)r * Nbw + J] = __float2bfloat16_rn(x);
  }
  if (lane == 0) mu[r] = none ? 0.f : mx;
}

// ------------------------------------------------------------------ A_I^T = sum_J W[I][J] C_J^T
// grid (128 n-tiles of 128 columns of the flattened (e, c) index, ceil(Nb/128) I-tiles, B*H), 128 threads.
// A operand: W tile [128 I][64 J] K-major; B operand: C^T rows [64 J][128 n] as two 64-element panels, MN-major.
__global__ void __launch_bounds__(128)
aggregate_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_c, int Nb, int Nbw,
                 __nv_bfloat16* __restrict__ at, int32_t* __restrict__ status) {
  using namespace rem;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  __shared__ __align__(8) unsigned long long bars[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s;
  volatile int* abort_flag = &abort_s;
  const uint32_t bar_full = smem_u32(&bars[0]), bar_mma = smem_u32(&bars[1]);
  const int nt = blockIdx.x, it = blockIdx.y, bh = blockIdx.z;
  const int warp = threadIdx.x >> 5;
  constexpr uint32_t A_BYTES = 128 * 128, B_PANEL = 64 * 128;           // 16 KB W tile; two 8 KB panels of C^T rows
  if (threadIdx.x == 0) {
    mbar_init(bar_full, 1);
    mbar_init(bar_mma, 1);
    abort_s = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(128u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  bool ok = true;
  if (threadIdx.x == 0) {
    const uint32_t idesc = instr_desc(128, 128, 1, true);
    const uint64_t ad = smem_desc(sbase, 16, 1024), bd = smem_desc(sbase + A_BYTES, B_PANEL, 1024);
    const int chunks = Nbw / 64;
    for (int ch = 0; ch < chunks && ok; ++ch) {
      if (ch > 0) ok = mbar_wait(bar_mma, (uint32_t)(ch - 1) & 1u, abort_flag, status);     // the tiles are free again
      if (!ok) break;
      mbar_expect_tx(bar_full, A_BYTES + 2 * B_PANEL);
      tma_load_3d(sbase, &tm_w, bar_full, ch * 64, it * 128, bh);
      tma_load_3d(sbase + A_BYTES, &tm_c, bar_full, nt * 128, ch * 64, bh);
      tma_load_3d(sbase + A_BYTES + B_PANEL, &tm_c, bar_full, nt * 128 + 64, ch * 64, bh);
      ok = mbar_wait(bar_full, (uint32_t)ch & 1u, abort_flag, status);
      if (!ok) break;
      tc_fence_after();
      for (int kk = 0; kk < 4; ++kk)                                       // 16 J per instruction
        tc_mma_ss_bf16(tmem_base, ad + (uint64_t)(kk * 2), bd + (uint64_t)(kk * 128), idesc, (ch > 0 || kk > 0) ? 1u : 0u);
      tc_commit(bar_mma, 1u);
    }
    if (ok) ok = mbar_wait(bar_mma, (uint32_t)(chunks - 1) & 1u, abort_flag, status);
    if (!ok) abort_s = 1;
  }
  __syncthreads();
  if (!abort_s) {
    tc_fence_after();
    const int I = it * 128 + threadIdx.x;                    // TMEM lane = query block of the tile
    const uint32_t lane_addr = tmem_base + ((uint32_t)(warp * 32) << 16);
    __nv_bfloat16* dst = at + ((long long)bh * Nb + I) * (D * D) + (long long)nt * 128;
#pragma unroll 1
    for (int c0 = 0; c0 < 128; c0 += 32) {
      uint32_t v[32];
      tmem_ld32(lane_addr + c0, v);
      tc_wait_ld();
      if (I < Nb) {
        uint32_t o[16];
#pragma unroll
        for (int t = 0; t < 32; t += 2) o[t >> 1] = pack_bf16(__uint_as_float(v[t]), __uint_as_float(v[t + 1]));
#pragma unroll
        for (int t = 0; t < 4; ++t)
          *reinterpret_cast<uint4*>(dst + c0 + 8 * t) = make_uint4(o[4 * t], o[4 * t + 1], o[4 * t + 2], o[4 * t + 3]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128u) : "memory");
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*rem_encode_fn_t)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static rem_encode_fn_t rem_encode() {
  static rem_encode_fn_t fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<rem_encode_fn_t>(p);
  }
  return fn;
}
// bf16 map of `rank` dimensions (byte strides for dimensions 1..), box = 64 elements (128 bytes) x box_rows, 128-byte swizzle
static int rem_map(CUtensorMap* map, const void* ptr, int rank, const cuuint64_t* dims, const cuuint64_t* strides, int box_rows) {
  rem_encode_fn_t enc = rem_encode();
  if (!enc) return SVA_ERR_CUDA;
  cuuint64_t st[3] = {0, 0, 0};
  for (int i = 0; i < rank - 1; ++i) {
    st[i] = strides[i];
    if (dims[i + 1] == 1 && i > 0) st[i] = st[i - 1] * dims[i];      // a size-1 dimension may carry any stride: give it a legal one
    if (st[i] % 16 != 0 || st[i] == 0) return SVA_ERR_ALIGNMENT;
  }
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(ptr), dims, st, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS ? SVA_OK : SVA_ERR_CUDA;
}

// Bytes of the four buffers: C^T [B*H*Nb][128][128] bf16, A^T the same, W [R][Nbw] bf16, mu [R] fp32 (each 256-aligned).
static size_t al256(size_t x) { return (x + 255) & ~(size_t)255; }
size_t remainder1_bytes(const Dims& m) {
  const size_t mats = al256((size_t)m.R * rem::D * rem::D * 2);
  const int Nbw = (m.Nb + 63) / 64 * 64;
  return 2 * mats + al256((size_t)m.R * Nbw * 2) + al256((size_t)m.R * 4);
}

// Fills `buf` (remainder1_bytes) from K, V, the routing's score matrix and the CSR.  *at_out / *mu_out: where the
// attention kernel finds A_I^T ([R][128 e][128 c] bf16) and mu_I.
// natural: A_I itself ([R][128 c][128 e]) instead of its transpose -- for an attention kernel that takes its "V" tiles
// keys-major (V read where it lies): the covariance kernel then simply gets K and V in each other's place.
int launch_remainder1(const Dims& m, const sva_problem_t* p, const void* k, const void* v, const float* scores,
                      const int32_t* row_ptr, const int32_t* col_idx, void* buf, const __nv_bfloat16** at_out,
                      const float** mu_out, int32_t* status, cudaStream_t st, bool natural) {
  if (m.d != rem::D || (m.block != 128 && m.block != 64)) return SVA_ERR_UNSUPPORTED;
  const size_t mats = al256((size_t)m.R * rem::D * rem::D * 2);
  const int Nbw = (m.Nb + 63) / 64 * 64;
  uint8_t* b = static_cast<uint8_t*>(buf);
  __nv_bfloat16* ct = reinterpret_cast<__nv_bfloat16*>(b);
  __nv_bfloat16* at = reinterpret_cast<__nv_bfloat16*>(b + mats);
  __nv_bfloat16* w = reinterpret_cast<__nv_bfloat16*>(b + 2 * mats);
  float* mu = reinterpret_cast<float*>(b + 2 * mats + al256((size_t)m.R * Nbw * 2));
  const Strides sk = make_strides(p->k_stride), sv = make_strides(p->v_stride);
  CUtensorMap tk, tv, tw, tc;
  int rc;
  {
    cuuint64_t dims[4] = {(cuuint64_t)m.d, (cuuint64_t)m.N, (cuuint64_t)m.H, (cuuint64_t)m.B};
    cuuint64_t s1[3] = {(cuuint64_t)sk.n * 2, (cuuint64_t)sk.h * 2, (cuuint64_t)sk.b * 2};
    cuuint64_t s2[3] = {(cuuint64_t)sv.n * 2, (cuuint64_t)sv.h * 2, (cuuint64_t)sv.b * 2};
    if (m.H == 1) { s1[1] = s1[0] * m.N; s2[1] = s2[0] * m.N; }
    if (m.B == 1) { s1[2] = s1[1] * m.H; s2[2] = s2[1] * m.H; }
    if ((rc = rem_map(&tk, k, 4, dims, s1, m.block)) != SVA_OK) return rc;
    if ((rc = rem_map(&tv, v, 4, dims, s2, m.block)) != SVA_OK) return rc;
  }
  {
    const int BH = m.B * m.H;
    cuuint64_t dw[3] = {(cuuint64_t)Nbw, (cuuint64_t)m.Nb, (cuuint64_t)BH};
    cuuint64_t sw[2] = {(cuuint64_t)Nbw * 2, (cuuint64_t)Nbw * 2 * m.Nb};
    if ((rc = rem_map(&tw, w, 3, dw, sw, 128)) != SVA_OK) return rc;
    cuuint64_t dc[3] = {(cuuint64_t)rem::D * rem::D, (cuuint64_t)m.Nb, (cuuint64_t)BH};
    cuuint64_t sc[2] = {(cuuint64_t)rem::D * rem::D * 2, (cuuint64_t)rem::D * rem::D * 2 * m.Nb};
    if ((rc = rem_map(&tc, ct, 3, dc, sc, 64)) != SVA_OK) return rc;
  }
  const int smem_cov = 2 * rem::TILE + 1024, smem_agg = 128 * 128 + 2 * 64 * 128 + 1024;
  if (cudaFuncSetAttribute(cov_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_cov) != cudaSuccess) return SVA_ERR_CUDA;
  if (natural) cov_kernel<<<dim3(m.Nb, m.B * m.H), 128, smem_cov, st>>>(tv, tk, m.H, m.N, m.block, m.Nb, ct, status);
  else cov_kernel<<<dim3(m.Nb, m.B * m.H), 128, smem_cov, st>>>(tk, tv, m.H, m.N, m.block, m.Nb, ct, status);
  if (cudaGetLastError() != cudaSuccess) return SVA_ERR_CUDA;
  weights_kernel<<<(m.R + 7) / 8, 256, 0, st>>>(scores, row_ptr, col_idx, m.R, m.Nb, Nbw, w, mu);
  if (cudaGetLastError() != cudaSuccess) return SVA_ERR_CUDA;
  aggregate_kernel<<<dim3(rem::D, (m.Nb + 127) / 128, m.B * m.H), 128, smem_agg, st>>>(tw, tc, m.Nb, Nbw, at, status);
  if (cudaGetLastError() != cudaSuccess) return SVA_ERR_CUDA;
  *at_out = at;
  *mu_out = mu;
  return SVA_OK;
}

}  // namespace sva
