// Block routing: mean pooling of Q and K per block, scaled pooled scores, per-row top-k or
// cumulative-mass selection with ties to the lower block index, optional forced neighbour
// window, CSR assembly.  (Paper: "score-based routing" of the critical blocks; block-wise
// similarity metric of the sparse-attention section.)
//
// pool_kernel streams Q and K once from HBM: 128-bit loads, fp32 accumulation in a fixed order, one
// CTA per (block, head, tensor).  block_scores_kernel computes a head's score matrix as a small fp32
// GEMM (64 x 64 tiles from two shared-memory panels, fixed summation order).  select_rows_kernel is one
// warp per query-block row: it reads the row's scores from that matrix (no shared memory), finds the
// threshold of the rule by bisection on order-preserving integer keys and emits the kept blocks in
// ascending order.  When the per-row count is known on the host (top-k with no window larger than k)
// rows go straight into the CSR; otherwise they are staged and csr_kernel builds it in one launch.
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


struct SelParams {
  int H, Nb, mode, k, use_window, win_t, win_s, bpf, cap, fixed_n;
  float scale, tau;
};

__device__ __forceinline__ bool in_window(int I, int J, const SelParams& p) {
  int ti = I / p.bpf, si = I % p.bpf, tj = J / p.bpf, sj = J % p.bpf;
  return abs(ti - tj) <= p.win_t && abs(si - sj) <= p.win_s;
}

// Order-preserving map float -> uint32 (larger score <=> larger key, every real score maps to a
// non-zero key); +0 and -0 share a key; NaN maps to 0, which is never selected.
__device__ __forceinline__ uint32_t score_key(float v) {
  if (!(v == v)) return 0u;
  uint32_t u = __float_as_uint(v + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_score(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key ^ 0x80000000u) : ~key);
}

// Selection and emission of one query-block row by one warp.  Lane j owns the key blocks
// J = it*32 + j, it < ITEMS, whose scores arrive as sortable keys (0 = no candidate).
template <int ITEMS>
__device__ __forceinline__ void select_and_emit(uint32_t (&key)[ITEMS], const int I, const int bh, const int lane,
                                                const SelParams& p, int32_t* __restrict__ row_ptr,
                                                int32_t* __restrict__ col_idx, int32_t* __restrict__ tmp_idx,
                                                int32_t* __restrict__ counts, const int R) {
  const int Nb = p.Nb;
  // ---- selection
  // The rule is sequential -- forced window first, then candidates by score (descending, ties to the
  // lower index) until k blocks are kept or, in mode 1, the kept softmax mass reaches tau -- but what it
  // keeps is "every candidate above a threshold key plus the first few of the candidates equal to it",
  // so the threshold is found by a 32-step bisection on the key bits (each step: one compare per
  // register, a warp reduction of the count and, in mode 1, of the mass) instead of up to k rounds of
  // arg-max.  The masses are summed in fixed point (weights in units of 2^-31: a warp-wide integer add is
  // one instruction where a float sum is five shuffle rounds, and the result does not depend on the order),
  // so decisions agree with the round-by-round form except where the mass comes within about 1e-7 --
  // fp32 summation noise -- of tau.
  uint32_t mask = 0;            // bit it set <=> block it*32+lane is kept
  int n = 0;
  uint32_t cum = 0u;            // kept mass so far, units of 2^-31
  const uint32_t tau_q = __float2uint_rn(fminf(fmaxf(p.tau, 0.f), 1.f) * 2147483648.f);
  float mx = 0.f, inv_z = 0.f;
  uint32_t wgt[ITEMS];          // mode 1: softmax weight of every candidate, units of 2^-31
#pragma unroll
  for (int it = 0; it < ITEMS; ++it) wgt[it] = 0u;
  if (p.mode == 1) {
    uint32_t km = 0u;
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) km = max(km, key[it]);
    km = __reduce_max_sync(0xffffffffu, km);
    mx = key_score(km);
    float z = 0.f, ew[ITEMS];
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
      ew[it] = 0.f;
      if (key[it]) { ew[it] = expf(key_score(key[it]) - mx); z += ew[it]; }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    inv_z = 1.0f / z;
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) wgt[it] = __float2uint_rn(ew[it] * inv_z * 2147483648.f);
  }
  if (p.use_window) {
    uint32_t fm = 0u;
    int cnt = 0;
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
      const int J = it * 32 + lane;
      if (J < Nb && in_window(I, J, p)) {
        mask |= 1u << it; ++cnt;
        fm += wgt[it];
        key[it] = 0u;                        // no longer a candidate
        wgt[it] = 0u;
      }
    }
    n = (int)__reduce_add_sync(0xffffffffu, (unsigned)cnt);
    cum = __reduce_add_sync(0xffffffffu, fm);
  }
  const int kk = min(p.k, Nb);
  if (n < kk && !(p.mode == 1 && n >= 1 && cum >= tau_q)) {
    // count and mass of the candidates with key >= t
    auto above = [&](uint32_t t, int& cnt, uint32_t& mass) {
      int c = 0;
      uint32_t g = 0u;
#pragma unroll
      for (int it = 0; it < ITEMS; ++it) {
        const bool ge = key[it] >= t && key[it] != 0u;
        c += ge;
        if (ge) g += wgt[it];
      }
      cnt = (int)__reduce_add_sync(0xffffffffu, (unsigned)c);
      mass = p.mode == 1 ? __reduce_add_sync(0xffffffffu, g) : 0u;
    };
    // largest threshold at which taking every candidate >= it ends the rule (0: never -> take them all)
    uint32_t T = 0u;
#pragma unroll 1
    for (int bit = 31; bit >= 0; --bit) {
      const uint32_t t = T | (1u << bit);
      int c;
      uint32_t g;
      above(t, c, g);
      if (n + c >= kk || (p.mode == 1 && c >= 1 && cum + g >= tau_q)) T = t;
    }
    // everything above T, then ties at T in index order while the rule still runs
    int G;
    uint32_t Mg;
    above(T + 1u, G, Mg);                    // T = 0: all candidates; T = 0xffffffff cannot be reached (see below)
    int have = n + G;
    uint32_t acc = cum + Mg;
    int ties_wanted = 0;
    if (T != 0u) {
      int E = 0;
      uint32_t wT = 0u;                      // weight of a candidate equal to T (they all have the same)
#pragma unroll
      for (int it = 0; it < ITEMS; ++it) {
        E += (key[it] == T);
        if (key[it] == T) wT = wgt[it];
      }
      E = (int)__reduce_add_sync(0xffffffffu, (unsigned)E);
      wT = __reduce_max_sync(0xffffffffu, wT);
      while (ties_wanted < E) {
        if (have >= kk) break;
        if (p.mode == 1 && have >= 1 && acc >= tau_q) break;
        ++ties_wanted; ++have; acc += wT;
      }
    }
    int seen = 0;                            // ties met so far, in index order
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
      const bool cand = key[it] != 0u;
      const bool gt = cand && key[it] > T;
      const bool eq = cand && T != 0u && key[it] == T;
      const uint32_t bal = __ballot_sync(0xffffffffu, eq);
      const bool take = gt || (eq && seen + __popc(bal & ((1u << lane) - 1u)) < ties_wanted);
      if (take) mask |= 1u << it;
      seen += __popc(bal);
    }
    n = have;
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
#pragma unroll
  for (int it = 0; it < ITEMS; ++it) {
    if (it * 32 >= Nb) break;
    bool sel = mask >> it & 1u;
    uint32_t bal = __ballot_sync(0xffffffffu, sel);
    if (sel) out[base + __popc(bal & ((1u << lane) - 1u))] = it * 32 + lane;
    base += __popc(bal);
  }
}

// Block scores of one head as a small fp32 GEMM: S[I][J] = scale * <qbar_I, kbar_J>.  A CTA computes a
// 64 x 64 tile from the two 64 x D panels in shared memory (row stride D + 4 floats: 128-bit reads of
// eight consecutive rows touch every bank once); a thread owns a 4 x 4 patch -- rows 4*ty..4*ty+3 (one
// address per half-warp: a broadcast), keys tx, tx+16, tx+32, tx+48 -- and keeps two partial sums per
// entry (dimensions 0,2 mod 4 and 1,3 mod 4, each in ascending order; that order is part of the
// result: it is what makes the scores reproducible bit for bit).  32 independent FMA chains per thread
// hide the shared-memory latency that bounded the earlier one-warp-per-row form.
static constexpr int SC_TILE = 64;
template <int D>
__global__ void __launch_bounds__(256)
block_scores_kernel(const float* __restrict__ qbar, const float* __restrict__ kbar, int Nb, float scale,
                    float* __restrict__ scores) {
  constexpr int LD = D + 4;
  extern __shared__ __align__(16) float sc_smem[];
  float* qs = sc_smem;                     // [64][LD]
  float* ks = sc_smem + SC_TILE * LD;      // [64][LD]
  const int bh = blockIdx.z, I0 = blockIdx.y * SC_TILE, J0 = blockIdx.x * SC_TILE;
  const float* qb = qbar + (long long)bh * Nb * D;
  const float* kb = kbar + (long long)bh * Nb * D;
  for (int idx = threadIdx.x; idx < SC_TILE * (D / 4); idx += 256) {
    const int row = idx / (D / 4), c4 = idx % (D / 4);
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    if (I0 + row < Nb) a = __ldg(reinterpret_cast<const float4*>(qb + (long long)(I0 + row) * D) + c4);
    if (J0 + row < Nb) b = __ldg(reinterpret_cast<const float4*>(kb + (long long)(J0 + row) * D) + c4);
    *reinterpret_cast<float4*>(qs + row * LD + 4 * c4) = a;
    *reinterpret_cast<float4*>(ks + row * LD + 4 * c4) = b;
  }
  __syncthreads();
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float a0[4][4], a1[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { a0[i][j] = 0.f; a1[i][j] = 0.f; }
#pragma unroll 2
  for (int c = 0; c < D; c += 4) {
    float4 qv[4], kv[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) qv[i] = *reinterpret_cast<const float4*>(qs + (ty * 4 + i) * LD + c);
#pragma unroll
    for (int j = 0; j < 4; ++j) kv[j] = *reinterpret_cast<const float4*>(ks + (tx + 16 * j) * LD + c);
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        a0[i][j] = fmaf(qv[i].x, kv[j].x, a0[i][j]);
        a1[i][j] = fmaf(qv[i].y, kv[j].y, a1[i][j]);
        a0[i][j] = fmaf(qv[i].z, kv[j].z, a0[i][j]);
        a1[i][j] = fmaf(qv[i].w, kv[j].w, a1[i][j]);
      }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int I = I0 + ty * 4 + i;
    if (I >= Nb) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int J = J0 + tx + 16 * j;
      if (J < Nb) scores[((long long)bh * Nb + I) * Nb + J] = (a0[i][j] + a1[i][j]) * scale;
    }
  }
}

// Selection: one warp per query-block row, its Nb scores read straight from the score matrix (lane j owns
// the key blocks it*32 + j).  No shared memory and few registers, so the SMs hold enough warps to hide the
// serial chain of the threshold search.
static constexpr int SEL_WARPS = 8;
template <int ITEMS>
__global__ void __launch_bounds__(SEL_WARPS * 32)
select_rows_kernel(const float* __restrict__ scores, SelParams p, int32_t* __restrict__ row_ptr,
                   int32_t* __restrict__ col_idx, int32_t* __restrict__ tmp_idx, int32_t* __restrict__ counts, int R) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * SEL_WARPS + (threadIdx.x >> 5);
  if (r >= R) return;
  const int Nb = p.Nb, bh = r / Nb, I = r % Nb;
  const float* srow = scores + (long long)r * Nb;
  uint32_t key[ITEMS];
#pragma unroll
  for (int it = 0; it < ITEMS; ++it) {
    const int J = it * 32 + lane;
    key[it] = J < Nb ? score_key(__ldg(srow + J)) : 0u;
  }
  select_and_emit<ITEMS>(key, I, bh, lane, p, row_ptr, col_idx, tmp_idx, counts, R);
}

// CSR assembly for rows of varying length, one launch: a CTA owns 32 consecutive rows (one warp each).  It
// first adds up the counts of all rows before its own (every thread a strided share, then a block
// reduction: at most R counts = a few KB from the L2 per CTA, which is cheaper than a scan kernel of its
// own plus its launch), then scans its 32 counts, writes row_ptr and copies the staged indices.
static constexpr int CSR_ROWS = 32;
__global__ void __launch_bounds__(CSR_ROWS * 32)
csr_kernel(const int32_t* __restrict__ tmp_idx, const int32_t* __restrict__ counts, int cap, int R,
           int32_t* __restrict__ row_ptr, int32_t* __restrict__ col_idx) {
  __shared__ int warp_sum[32];
  __shared__ int row_off[CSR_ROWS + 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int r0 = blockIdx.x * CSR_ROWS;
  int part = 0;
  for (int i = threadIdx.x; i < r0; i += CSR_ROWS * 32) part += __ldg(counts + i);
#pragma unroll
  for (int o = 16; o; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
  if (lane == 0) warp_sum[warp] = part;
  __syncthreads();
  if (warp == 0) {
    int base = warp_sum[lane];
#pragma unroll
    for (int o = 16; o; o >>= 1) base += __shfl_xor_sync(0xffffffffu, base, o);   // rows before this CTA
    const int r = r0 + lane;
    const int c = r < R ? __ldg(counts + r) : 0;
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    row_off[lane] = base + incl - c;
    if (r < R) row_ptr[r] = base + incl - c;
    if (r == R - 1) row_ptr[R] = base + incl;
  }
  __syncthreads();
  const int r = r0 + warp;
  if (r >= R) return;
  const int n = __ldg(counts + r), dst = row_off[warp];
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
  bytes += align256((size_t)m.R * m.Nb * sizeof(float));      // the score matrix (unused when the caller asks for it)
  return bytes;
}

template <int D>
static int launch_select_d(const Dims& m, const sva_problem_t* p, const sva_select_t* s,
                           const void* q, const void* k, const float* q_scale,
                           const float* k_scale, int32_t* row_ptr, int32_t* col_idx,
                           float* block_scores, void* ws, cudaStream_t st,
                           const float* qbar_in = nullptr, const float* kbar_in = nullptr) {
  size_t pooled = align256((size_t)m.B * m.H * m.Nb * m.d * sizeof(float));
  char* w = static_cast<char*>(ws);
  // (block means supplied by the caller -- the fused prologue writes them -- are used where they are)
  float* qbar = qbar_in ? const_cast<float*>(qbar_in) : reinterpret_cast<float*>(w);
  float* kbar = kbar_in ? const_cast<float*>(kbar_in) : reinterpret_cast<float*>(w + pooled);
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
  if (qbar_in) {
  } else if (m.fp8)
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
  // scores: into the caller's matrix if it wants one, else into the workspace (after the staging arrays)
  float* scores = block_scores;
  if (!scores) {
    size_t off = 2 * pooled;
    if (!fixed_n) off += align256((size_t)m.R * cap * sizeof(int32_t)) + align256((size_t)m.R * sizeof(int32_t));
    scores = reinterpret_cast<float*>(w + off);
  }
  {
    auto kern = block_scores_kernel<D>;
    constexpr int smem = 2 * SC_TILE * (D + 4) * (int)sizeof(float);
    // (the shared-memory attribute is set once per device and instantiation, not per call)
    static std::mutex attr_mutex;
    static bool attr_set[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SVA_ERR_CUDA;
    {
      std::lock_guard<std::mutex> lock(attr_mutex);
      if (!attr_set[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return SVA_ERR_CUDA;
        attr_set[dev] = true;
      }
    }
    const int nt = (m.Nb + SC_TILE - 1) / SC_TILE;
    kern<<<dim3(nt, nt, m.B * m.H), 256, smem, st>>>(qbar, kbar, m.Nb, m.scale, scores);
  }
  const int items = (m.Nb + 31) / 32;
  const int sg = (m.R + SEL_WARPS - 1) / SEL_WARPS;
#define SVA_SEL_LAUNCH(IT) \
  select_rows_kernel<IT><<<sg, SEL_WARPS * 32, 0, st>>>(scores, sp, row_ptr, col_idx, tmp_idx, counts, m.R)
  if (items <= 4) SVA_SEL_LAUNCH(4);
  else if (items <= 8) SVA_SEL_LAUNCH(8);
  else if (items <= 12) SVA_SEL_LAUNCH(12);
  else if (items <= 16) SVA_SEL_LAUNCH(16);
  else SVA_SEL_LAUNCH(32);
#undef SVA_SEL_LAUNCH
  if (!fixed_n) {
    csr_kernel<<<(m.R + CSR_ROWS - 1) / CSR_ROWS, CSR_ROWS * 32, 0, st>>>(tmp_idx, counts, cap, m.R, row_ptr, col_idx);
  }
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

int launch_select(const Dims& m, const sva_problem_t* p, const sva_select_t* s, const void* q,
                  const void* k, const float* q_scale, const float* k_scale, int32_t* row_ptr,
                  int32_t* col_idx, float* block_scores, void* ws, size_t ws_bytes,
                  cudaStream_t st) {
  if (ws_bytes < select_workspace_bytes(m, s)) return SVA_ERR_WORKSPACE;
  if (m.Nb > 1024) return SVA_ERR_UNSUPPORTED;    // a lane holds at most 32 scores of a row, kept flags in one word per lane
  if (m.d == 128)
    return launch_select_d<128>(m, p, s, q, k, q_scale, k_scale, row_ptr, col_idx, block_scores, ws, st);
  if (m.d == 64)
    return launch_select_d<64>(m, p, s, q, k, q_scale, k_scale, row_ptr, col_idx, block_scores, ws, st);
  return SVA_ERR_UNSUPPORTED;
}

// Pooling alone: block means of Q and K into the caller's arrays ([B,H,Nb,d] fp32 each).
int launch_pool(const Dims& m, const sva_problem_t* p, const void* q, const void* k, const float* q_scale,
                const float* k_scale, float* qbar, float* kbar, cudaStream_t st) {
  dim3 pg(m.Nb, m.B * m.H, 2);
  Strides sq = make_strides(p->q_stride), sk = make_strides(p->k_stride);
#define SVA_POOL_LAUNCH(DD)                                                                                        \
  do {                                                                                                             \
    if (m.fp8)                                                                                                     \
      pool_kernel<DD, 1><<<pg, POOL_THREADS, 0, st>>>((const uint8_t*)q, (const uint8_t*)k, sq, sk, q_scale, k_scale, \
                                                      m.H, m.N, m.block, m.Nb, qbar, kbar);                       \
    else                                                                                                           \
      pool_kernel<DD, 2><<<pg, POOL_THREADS, 0, st>>>((const uint8_t*)q, (const uint8_t*)k, sq, sk, nullptr, nullptr, \
                                                      m.H, m.N, m.block, m.Nb, qbar, kbar);                       \
  } while (0)
  if (m.d == 128) SVA_POOL_LAUNCH(128);
  else if (m.d == 64) SVA_POOL_LAUNCH(64);
  else return SVA_ERR_UNSUPPORTED;
#undef SVA_POOL_LAUNCH
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

// Routing from block means the caller already has (qbar, kbar: [B,H,Nb,d] fp32).
int launch_select_pooled(const Dims& m, const sva_problem_t* p, const sva_select_t* s, const float* qbar,
                         const float* kbar, int32_t* row_ptr, int32_t* col_idx, float* block_scores, void* ws,
                         size_t ws_bytes, cudaStream_t st) {
  if (ws_bytes < select_workspace_bytes(m, s)) return SVA_ERR_WORKSPACE;
  if (m.Nb > 1024) return SVA_ERR_UNSUPPORTED;
  if (m.d == 128)
    return launch_select_d<128>(m, p, s, nullptr, nullptr, nullptr, nullptr, row_ptr, col_idx, block_scores, ws, st, qbar, kbar);
  if (m.d == 64)
    return launch_select_d<64>(m, p, s, nullptr, nullptr, nullptr, nullptr, row_ptr, col_idx, block_scores, ws, st, qbar, kbar);
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
