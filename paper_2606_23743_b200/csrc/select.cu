// Block routing: mean pooling of Q and K per block, scaled pooled scores, per-row top-k or
// cumulative-mass selection with ties to the lower block index, optional forced neighbour
// window, CSR assembly.  (Paper: "score-based routing" of the critical blocks; block-wise
// similarity metric of the sparse-attention section.)
//
// Kernel 1 (pool) streams Q and K once from HBM: 128-bit loads, fp32 accumulation in a fixed
// order, one CTA per (block, head, tensor).  Kernel 2 (score+select) is one warp per query
// block row with the head's pooled K staged through shared memory.  When the per-row count is
// not a compile-time constant of the call (mass rule, or a window larger than k), rows are
// staged and kernels 3/4 (scan, compact) build the CSR.
#include <mutex>

#include "common.cuh"

namespace sva {

static constexpr int POOL_THREADS = 256;

// One CTA pools one block of one head of one tensor (blockIdx.z: 0 = Q, 1 = K).
// ELEM_BYTES = 2: bf16 input.  ELEM_BYTES = 1: e4m3 codes, multiplied by the block's scale.
template <int D, int ELEM_BYTES>
__global__ void __launch_bounds__(POOL_THREADS)
pool_kernel(const uint8_t* __restrict__ q, const uint8_t* __restrict__ k, Strides sq, Strides sk,
            const float* __restrict__ q_scale, const float* __restrict__ k_scale, int H, int N,
            int block, int Nb, float* __restrict__ qbar, float* __restrict__ kbar) {
  constexpr int EPV = 16 / ELEM_BYTES;          // elements per 16-byte vector
  constexpr int VPR = D / EPV;                  // vectors per token row
  constexpr int GROUPS = POOL_THREADS / VPR;    // token rows read concurrently
  __shared__ float part[GROUPS][D + 1];

  const int I = blockIdx.x, bh = blockIdx.y, which = blockIdx.z;
  const int b = bh / H, h = bh % H;
  const uint8_t* base = which ? k : q;
  const Strides s = which ? sk : sq;
  base += ((long long)b * s.b + (long long)h * s.h) * ELEM_BYTES;
  const int lo = I * block;
  const int cnt = min(block, N - lo);
  const int vec = threadIdx.x % VPR, grp = threadIdx.x / VPR;

  float acc[EPV];
#pragma unroll
  for (int e = 0; e < EPV; ++e) acc[e] = 0.f;

  for (int t0 = grp; t0 < cnt; t0 += GROUPS * 4) {
    uint4 u[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int t = t0 + j * GROUPS;
      u[j] = make_uint4(0, 0, 0, 0);
      if (t < cnt)
        u[j] = __ldg(reinterpret_cast<const uint4*>(base + (long long)(lo + t) * s.n * ELEM_BYTES) + vec);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t w[4] = {u[j].x, u[j].y, u[j].z, u[j].w};
      if constexpr (ELEM_BYTES == 2) {
#pragma unroll
        for (int e = 0; e < 4; ++e) { acc[2 * e] += bf16lo(w[e]); acc[2 * e + 1] += bf16hi(w[e]); }
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
#pragma unroll
          for (int c = 0; c < 4; ++c) acc[4 * e + c] += e4m3_to_float((w[e] >> (8 * c)) & 0xff);
      }
    }
  }
#pragma unroll
  for (int e = 0; e < EPV; ++e) part[grp][vec * EPV + e] = acc[e];
  __syncthreads();
  if (threadIdx.x < D) {
    float sum = 0.f;
#pragma unroll 8
    for (int g = 0; g < GROUPS; ++g) sum += part[g][threadIdx.x];   // fixed order
    float mean = sum / (float)cnt;
    if (ELEM_BYTES == 1) mean *= (which ? k_scale : q_scale)[(long long)bh * Nb + I];
    (which ? kbar : qbar)[((long long)bh * Nb + I) * D + threadIdx.x] = mean;
  }
}

static constexpr int SEL_WARPS = 8;     // query-block rows per CTA
static constexpr int SEL_CHUNK = 32;    // key blocks staged per pass

struct SelParams {
  int H, Nb, mode, k, use_window, win_t, win_s, bpf, cap, fixed_n;
  float scale, tau;
};

__device__ __forceinline__ bool in_window(int I, int J, const SelParams& p) {
  int ti = I / p.bpf, si = I % p.bpf, tj = J / p.bpf, sj = J % p.bpf;
  return abs(ti - tj) <= p.win_t && abs(si - sj) <= p.win_s;
}

// dynamic smem: qs[SEL_WARPS][D] | ks[SEL_CHUNK][D] | sc[SEL_WARPS][Nb32]
template <int D>
__global__ void __launch_bounds__(SEL_WARPS * 32)
score_select_kernel(const float* __restrict__ qbar, const float* __restrict__ kbar, SelParams p,
                    int32_t* __restrict__ row_ptr, int32_t* __restrict__ col_idx,
                    int32_t* __restrict__ tmp_idx, int32_t* __restrict__ counts,
                    float* __restrict__ block_scores, int R) {
  extern __shared__ float smem[];
  const int Nb = p.Nb;
  const int Nb32 = (Nb + 31) & ~31;
  float* qs = smem;
  float* ks = qs + SEL_WARPS * D;
  float* sc = ks + SEL_CHUNK * D;

  const int bh = blockIdx.y;
  const int I0 = blockIdx.x * SEL_WARPS;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int I = I0 + warp;
  const bool row_ok = I < Nb;

  for (int i = threadIdx.x; i < SEL_WARPS * D; i += blockDim.x) {
    int w = i / D;
    qs[i] = (I0 + w < Nb) ? qbar[((long long)bh * Nb + I0 + w) * D + (i % D)] : 0.f;
  }
  const float* kb = kbar + (long long)bh * Nb * D;
  float* my_sc = sc + warp * Nb32;

  for (int c0 = 0; c0 < Nb; c0 += SEL_CHUNK) {
    __syncthreads();
    const int nrow = min(SEL_CHUNK, Nb - c0);
    for (int i = threadIdx.x; i < SEL_CHUNK * D / 4; i += blockDim.x) {
      int rr = i / (D / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (rr < nrow) v = __ldg(reinterpret_cast<const float4*>(kb + (long long)c0 * D) + i);
      reinterpret_cast<float4*>(ks)[i] = v;
    }
    __syncthreads();
    // lane j scores key block c0+j; the column index is rotated by the lane so that the 32
    // lanes touch 32 different banks
    float acc = 0.f;
    const float* qrow = qs + warp * D;
    const float* krow = ks + lane * D;
#pragma unroll 8
    for (int c = 0; c < D; ++c) {
      int idx = (c + lane) & (D - 1);
      acc = fmaf(qrow[idx], krow[idx], acc);
    }
    acc *= p.scale;
    int J = c0 + lane;
    my_sc[J] = (J < Nb) ? acc : -INFINITY;
    if (block_scores && row_ok && J < Nb) block_scores[((long long)bh * Nb + I) * Nb + J] = acc;
  }
  __syncwarp();
  if (!row_ok) return;

  // ---- per-row selection, one warp.  Item (it, lane) <-> key block J = it*32 + lane.
  const int items = Nb32 / 32;
  uint32_t mask = 0;            // bit it set <=> block it*32+lane is kept
  int n = 0;
  float cum = 0.f, mx = 0.f, inv_z = 0.f;

  if (p.mode == 1) {
    float m = -INFINITY;
    for (int it = 0; it < items; ++it) m = fmaxf(m, my_sc[it * 32 + lane]);
#pragma unroll
    for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float z = 0.f;
    for (int it = 0; it < items; ++it) z += expf(my_sc[it * 32 + lane] - m);   // exp(-inf) = 0
#pragma unroll
    for (int o = 16; o; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    mx = m; inv_z = 1.0f / z;
  }
  if (p.use_window) {
    float fm = 0.f;
    int cnt = 0;
    for (int it = 0; it < items; ++it) {
      int J = it * 32 + lane;
      if (J < Nb && in_window(I, J, p)) {
        mask |= 1u << it; ++cnt;
        if (p.mode == 1) fm += expf(my_sc[J] - mx) * inv_z;
      }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
      fm += __shfl_xor_sync(0xffffffffu, fm, o);
    }
    n = cnt; cum = fm;
  }
  const int kk = min(p.k, Nb);
  while (true) {
    if (n >= kk) break;
    if (p.mode == 1 && n >= 1 && cum >= p.tau) break;
    float bv = -INFINITY;
    int bj = 0x7fffffff;
    for (int it = 0; it < items; ++it) {
      if (mask >> it & 1u) continue;
      int J = it * 32 + lane;
      float v = my_sc[J];
      if (J < Nb && v == v && (bj == 0x7fffffff || v > bv || (v == bv && J < bj))) { bv = v; bj = J; }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      int oj = __shfl_xor_sync(0xffffffffu, bj, o);
      if (oj != 0x7fffffff && (bj == 0x7fffffff || ov > bv || (ov == bv && oj < bj))) { bv = ov; bj = oj; }
    }
    if (bj == 0x7fffffff) break;            // nothing selectable left (all NaN)
    if ((bj & 31) == lane) mask |= 1u << (bj >> 5);
    ++n;
    if (p.mode == 1) cum += expf(bv - mx) * inv_z;
  }

  // ---- emit ascending
  const int r = bh * Nb + I;
  int32_t* out;
  if (p.fixed_n) {
    out = col_idx + (long long)r * p.fixed_n;
    if (lane == 0) {
      row_ptr[r] = r * p.fixed_n;
      if (r == R - 1) row_ptr[R] = R * p.fixed_n;
    }
  } else {
    out = tmp_idx + (long long)r * p.cap;
    if (lane == 0) counts[r] = n;
  }
  int base = 0;
  for (int it = 0; it < items; ++it) {
    bool sel = mask >> it & 1u;
    uint32_t bal = __ballot_sync(0xffffffffu, sel);
    if (sel) out[base + __popc(bal & ((1u << lane) - 1u))] = it * 32 + lane;
    base += __popc(bal);
  }
}

// Exclusive scan of counts[R] -> row_ptr[R+1]; one CTA, chunks of 1024 with a running carry.
__global__ void __launch_bounds__(1024) scan_kernel(const int32_t* __restrict__ counts, int R,
                                                     int32_t* __restrict__ row_ptr) {
  __shared__ int warp_sum[32];
  __shared__ int carry_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < R; base += 1024) {
    int i = base + threadIdx.x;
    int v = i < R ? counts[i] : 0;
    int x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) warp_sum[warp] = x;
    __syncthreads();
    if (warp == 0) {
      int w = warp_sum[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int y = __shfl_up_sync(0xffffffffu, w, o);
        if (lane >= o) w += y;
      }
      warp_sum[lane] = w;
    }
    __syncthreads();
    int incl = x + (warp ? warp_sum[warp - 1] : 0) + carry_s;
    if (i < R) row_ptr[i] = incl - v;
    __syncthreads();
    if (threadIdx.x == 1023) carry_s = incl;
    __syncthreads();
  }
  if (threadIdx.x == 0) row_ptr[R] = carry_s;
}

// One warp per row copies its staged indices to their CSR position.
__global__ void compact_kernel(const int32_t* __restrict__ tmp_idx, const int32_t* __restrict__ counts,
                               const int32_t* __restrict__ row_ptr, int cap, int R,
                               int32_t* __restrict__ col_idx) {
  int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  int lane = threadIdx.x & 31;
  if (r >= R) return;
  int n = counts[r], dst = row_ptr[r];
  for (int t = lane; t < n; t += 32) col_idx[dst + t] = tmp_idx[(long long)r * cap + t];
}

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

int select_row_cap(const Dims& m, const sva_select_t* s) {
  int kk = s->k < m.Nb ? s->k : m.Nb;
  int cap = kk;
  if (s->win_t >= 0 && s->win_s >= 0 && s->blocks_per_frame > 0) {
    long long w = (long long)(2 * s->win_t + 1) * (2 * s->win_s + 1);
    if (w > m.Nb) w = m.Nb;
    if (w > cap) cap = (int)w;
  }
  return cap;
}

// The row count is known on the host when the rule is top-k and the window cannot exceed k.
static int fixed_count(const Dims& m, const sva_select_t* s) {
  int kk = s->k < m.Nb ? s->k : m.Nb;
  if (s->mode != 0) return 0;
  return select_row_cap(m, s) == kk ? kk : 0;
}

size_t select_workspace_bytes(const Dims& m, const sva_select_t* s) {
  size_t pooled = align256((size_t)m.B * m.H * m.Nb * m.d * sizeof(float));
  size_t bytes = 2 * pooled;
  if (!fixed_count(m, s)) {
    bytes += align256((size_t)m.R * select_row_cap(m, s) * sizeof(int32_t));
    bytes += align256((size_t)m.R * sizeof(int32_t));
  }
  return bytes;
}

template <int D>
static int launch_select_d(const Dims& m, const sva_problem_t* p, const sva_select_t* s,
                           const void* q, const void* k, const float* q_scale,
                           const float* k_scale, int32_t* row_ptr, int32_t* col_idx,
                           float* block_scores, void* ws, cudaStream_t st) {
  size_t pooled = align256((size_t)m.B * m.H * m.Nb * m.d * sizeof(float));
  char* w = static_cast<char*>(ws);
  float* qbar = reinterpret_cast<float*>(w);
  float* kbar = reinterpret_cast<float*>(w + pooled);
  const int cap = select_row_cap(m, s);
  const int fixed_n = fixed_count(m, s);
  int32_t* tmp_idx = nullptr;
  int32_t* counts = nullptr;
  if (!fixed_n) {
    tmp_idx = reinterpret_cast<int32_t*>(w + 2 * pooled);
    counts = reinterpret_cast<int32_t*>(w + 2 * pooled + align256((size_t)m.R * cap * sizeof(int32_t)));
  }
  dim3 pg(m.Nb, m.B * m.H, 2);
  Strides sq = make_strides(p->q_stride), sk = make_strides(p->k_stride);
  if (m.fp8)
    pool_kernel<D, 1><<<pg, POOL_THREADS, 0, st>>>((const uint8_t*)q, (const uint8_t*)k, sq, sk, q_scale,
                                                   k_scale, m.H, m.N, m.block, m.Nb, qbar, kbar);
  else
    pool_kernel<D, 2><<<pg, POOL_THREADS, 0, st>>>((const uint8_t*)q, (const uint8_t*)k, sq, sk, nullptr,
                                                   nullptr, m.H, m.N, m.block, m.Nb, qbar, kbar);
  SelParams sp;
  sp.H = m.H; sp.Nb = m.Nb; sp.mode = s->mode; sp.k = s->k;
  sp.use_window = (s->win_t >= 0 && s->win_s >= 0 && s->blocks_per_frame > 0) ? 1 : 0;
  sp.win_t = s->win_t; sp.win_s = s->win_s; sp.bpf = sp.use_window ? s->blocks_per_frame : 1;
  sp.cap = cap; sp.fixed_n = fixed_n; sp.scale = m.scale; sp.tau = s->mass;
  const int Nb32 = (m.Nb + 31) & ~31;
  size_t smem = (size_t)(SEL_WARPS * D + SEL_CHUNK * D + SEL_WARPS * Nb32) * sizeof(float);
  if (cudaFuncSetAttribute(score_select_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024) != cudaSuccess)
    return SVA_ERR_CUDA;
  dim3 sg((m.Nb + SEL_WARPS - 1) / SEL_WARPS, m.B * m.H);
  score_select_kernel<D><<<sg, SEL_WARPS * 32, smem, st>>>(qbar, kbar, sp, row_ptr, col_idx, tmp_idx,
                                                           counts, block_scores, m.R);
  if (!fixed_n) {
    scan_kernel<<<1, 1024, 0, st>>>(counts, m.R, row_ptr);
    compact_kernel<<<(m.R * 32 + 255) / 256, 256, 0, st>>>(tmp_idx, counts, row_ptr, cap, m.R, col_idx);
  }
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

int launch_select(const Dims& m, const sva_problem_t* p, const sva_select_t* s, const void* q,
                  const void* k, const float* q_scale, const float* k_scale, int32_t* row_ptr,
                  int32_t* col_idx, float* block_scores, void* ws, size_t ws_bytes,
                  cudaStream_t st) {
  if (ws_bytes < select_workspace_bytes(m, s)) return SVA_ERR_WORKSPACE;
  if (m.Nb > 1024) return SVA_ERR_UNSUPPORTED;    // score rows live in shared memory, kept flags in one word per lane
  if (m.d == 128)
    return launch_select_d<128>(m, p, s, q, k, q_scale, k_scale, row_ptr, col_idx, block_scores, ws, st);
  if (m.d == 64)
    return launch_select_d<64>(m, p, s, q, k, q_scale, k_scale, row_ptr, col_idx, block_scores, ws, st);
  return SVA_ERR_UNSUPPORTED;
}

// ---------------------------------------------------------------- no-allocation variant
// Scratch for callers that cannot call cudaMalloc: it lives in the library image, so every
// GPU that loads the library carries these bytes until the process exits.  In host code the
// array's name is only a stand-in for the symbol -- not a device address -- so the address
// is looked up once per device with cudaGetSymbolAddress and that pointer is what the kernels
// receive.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SVA_NOALLOC_SCRATCH_BYTES];

static constexpr int MAX_DEVICES = 64;
static std::mutex g_noalloc_mutex;
static void* g_noalloc_addr[MAX_DEVICES];   // device address of g_noalloc_scratch, per device

int launch_select_noalloc(const Dims& m, const sva_problem_t* p, const sva_select_t* s,
                          const void* q, const void* k, const float* q_scale, const float* k_scale,
                          int32_t* row_ptr, int32_t* col_idx, float* block_scores, cudaStream_t st) {
  if (select_workspace_bytes(m, s) > (size_t)SVA_NOALLOC_SCRATCH_BYTES) return SVA_ERR_SCRATCH_LIMIT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return SVA_ERR_CUDA;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_addr[dev]) {
      // first call on this device (it is the current one): resolve the symbol
      void* addr = nullptr;
      if (cudaGetSymbolAddress(&addr, g_noalloc_scratch) != cudaSuccess || !addr) return SVA_ERR_CUDA;
      g_noalloc_addr[dev] = addr;
    }
    scratch = g_noalloc_addr[dev];
  }
  // Nothing in the scratch has to start at zero: pooled means, staged rows and counts are all
  // written by this call's kernels before they are read.
  return launch_select(m, p, s, q, k, q_scale, k_scale, row_ptr, col_idx, block_scores, scratch,
                       (size_t)SVA_NOALLOC_SCRATCH_BYTES, st);
}

}  // namespace sva
