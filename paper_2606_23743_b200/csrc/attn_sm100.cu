// Block-sparse / dense attention forward for sm_100a: TMA-staged tiles gathered by block
// index, tcgen05 MMAs with TMEM accumulators for Q K^T and P V, warp-specialised roles,
// online softmax in registers.  (Paper: critical blocks "computed exactly"; dense fallback.)
//
// One CTA owns NT query tiles (NT adjacent query blocks of one head, 128 rows each).
//   warps [0, 4*NT)   softmax: warpgroup t owns tile t, thread <-> query row (TMEM lane)
//   warp  4*NT        producer: one lane issues every TMA load (Q once, then K/V tiles)
//   warp  4*NT + 1    MMA: one lane issues every tcgen05.mma and commit; owns TMEM alloc
// TMEM columns (fp32): S_t at 128*t, O_t at 128*NT + 128*t; P_t (bf16 pairs) overlays the
// first 64 columns of S_t and feeds the P V MMA as the A operand straight from TMEM.
// Per tile and kept block j: S = Q K_j^T -> softmax warpgroup: row max, lazy rescale of O,
// P = exp2(S*c - m) -> O += P V_j.  With NT = 2 the tensor pipe works on one tile while the
// other tile's softmax runs.
//
// Every wait is bounded: when one expires the CTA sets SVA_DEV_TIMEOUT, all roles leave
// their loops, TMEM is released and the kernel returns.
#include <cuda.h>

#include "common.cuh"

namespace sva {

static constexpr int BS = 128;                 // rows per tile (queries and keys)
static constexpr long long WAIT_LIMIT_CYCLES = 3000000000LL;

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// Bounded wait.  Returns false when the CTA is aborting.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
        *abort_flag = 1;
        if (status) atomicOr(status, SVA_DEV_TIMEOUT);
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
template <bool F8>
__device__ __forceinline__ void tc_mma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
  if (F8)
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
  else
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void tc_mma_ts(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
               ::"r"(d), "r"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}

#define SVA_R4(v, i) "=r"(v[i]), "=r"(v[i + 1]), "=r"(v[i + 2]), "=r"(v[i + 3])
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : SVA_R4(v, 0), SVA_R4(v, 4), SVA_R4(v, 8), SVA_R4(v, 12), SVA_R4(v, 16), SVA_R4(v, 20),
        SVA_R4(v, 24), SVA_R4(v, 28)
      : "r"(taddr) : "memory");
}
#undef SVA_R4
#define SVA_I4(v, i) "r"(v[i]), "r"(v[i + 1]), "r"(v[i + 2]), "r"(v[i + 3])
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
      ::SVA_I4(v, 0), SVA_I4(v, 4), SVA_I4(v, 8), SVA_I4(v, 12), SVA_I4(v, 16), SVA_I4(v, 20),
        SVA_I4(v, 24), SVA_I4(v, 28), "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
      ::SVA_I4(v, 0), SVA_I4(v, 4), SVA_I4(v, 8), SVA_I4(v, 12), "r"(taddr) : "memory");
}
#undef SVA_I4

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// ------------------------------------------------------------------ descriptors
// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version of sm_100.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
         ((uint64_t)(sbo_bytes >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, A/B format code, B major, N, M.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int fmt, bool b_mn_major) {
  return (1u << 4) | ((uint32_t)fmt << 7) | ((uint32_t)fmt << 10) | (b_mn_major ? (1u << 16) : 0u) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

struct AttnParams {
  const int32_t* row_ptr;     // null = dense
  const int32_t* col_idx;
  const float* q_scale;       // fp8 only
  const float* k_scale;
  __nv_bfloat16* o;
  float* lse;
  int32_t* status;
  Strides so;
  int H, N, Nb, R;
  float scale_log2;           // softmax_scale * log2(e)
};

template <int D, int NT, bool F8>
struct Cfg {
  static constexpr int QK_ELEM = F8 ? 1 : 2;
  static constexpr int Q_BYTES = BS * D * QK_ELEM;       // one Q (or K) tile
  static constexpr int V_BYTES = BS * D * 2;
  static constexpr int STAGE_BYTES = V_BYTES;            // K tiles use a prefix of a stage
  static constexpr int STAGES = NT == 2 ? (D == 128 ? 5 : 8) : 4;
  static constexpr int THREADS = NT * 128 + 64;
  static constexpr int TMEM_COLS = 512;
  // dynamic shared memory: 1024-aligned tiles first, then the control block
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_RING = OFF_Q + NT * ((Q_BYTES + 1023) / 1024 * 1024);
  static constexpr int OFF_CTRL = OFF_RING + STAGES * STAGE_BYTES;
  static constexpr int CTRL_BYTES = 256;
  static constexpr int SMEM_BYTES = OFF_CTRL + CTRL_BYTES + 1024;   // + alignment slack
};

// control block layout (bytes from OFF_CTRL):
//   0   q_full[2]     16  s_full[2]    32  p_full[2]    48  o_done[2]
//   64  kv_full[8]    128 kv_empty[8]  192 tmem_base    196 abort   200 n_list[2]   208 beg[2]

template <int D, int NT, bool F8>
__global__ void __launch_bounds__(NT * 128 + 64, 1)
attn_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const AttnParams prm) {
  using C = Cfg<D, NT, F8>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  uint8_t* ctrl = smem + C::OFF_CTRL;
  const uint32_t cbase = sbase + C::OFF_CTRL;
  const uint32_t bar_q_full = cbase + 0, bar_s_full = cbase + 16, bar_p_full = cbase + 32,
                 bar_o_done = cbase + 48, bar_kv_full = cbase + 64, bar_kv_empty = cbase + 128;
  volatile uint32_t* tmem_base_p = reinterpret_cast<volatile uint32_t*>(ctrl + 192);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 196);
  volatile int* n_list = reinterpret_cast<volatile int*>(ctrl + 200);
  volatile int* beg_list = reinterpret_cast<volatile int*>(ctrl + 208);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int W_PROD = 4 * NT, W_MMA = 4 * NT + 1;
  const int row0 = blockIdx.x * NT;                 // first CSR row of this CTA
  const int Nb = prm.Nb;
  const bool dense = prm.row_ptr == nullptr;

  // ---------------------------------------------------------------- set-up
  if (threadIdx.x == 0) {
    for (int t = 0; t < 2; ++t) {
      mbar_init(bar_q_full + 8 * t, 1);
      mbar_init(bar_s_full + 8 * t, 1);
      mbar_init(bar_p_full + 8 * t, 128);
      mbar_init(bar_o_done + 8 * t, 1);
    }
    for (int s = 0; s < 8; ++s) {
      mbar_init(bar_kv_full + 8 * s, 1);
      mbar_init(bar_kv_empty + 8 * s, 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == W_PROD && lane == 0) {
    prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
  }
  if (warp == W_MMA) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(cbase + 192), "r"((uint32_t)C::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // warp 4t validates the CSR row of tile t; a row holding a bad entry is treated as empty
  if (warp < 4 * NT && (warp & 3) == 0) {
    const int t = warp >> 2;
    const int r = row0 + t;
    int n = 0, beg = 0;
    if (r < prm.R) {
      if (dense) {
        n = Nb;
      } else {
        beg = prm.row_ptr[r];
        const int end = prm.row_ptr[r + 1];
        bool bad = end < beg || end - beg > Nb || beg < 0;
        if (!bad) {
          for (int base = beg; base < end; base += 32) {
            const int e = base + lane;
            const int J = e < end ? __ldg(prm.col_idx + e) : 0;
            bad |= (J < 0 || J >= Nb);
          }
        }
        bad = __any_sync(0xffffffffu, bad);
        if (bad) {
          if (lane == 0 && prm.status) atomicOr(prm.status, SVA_DEV_BAD_INDEX);
        } else {
          n = end - beg;
        }
      }
    }
    if (lane == 0) { n_list[t] = n; beg_list[t] = beg; }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_p;
  int nl[2];
  nl[0] = n_list[0];
  nl[1] = NT == 2 ? n_list[1] : 0;
  int lbeg[2];
  lbeg[0] = beg_list[0];
  lbeg[1] = NT == 2 ? beg_list[1] : 0;

  if (warp == W_PROD) {
    // ------------------------------------------------------------ producer
    if (lane == 0) {
      bool ok = true;
      for (int t = 0; t < NT; ++t) {
        if (nl[t] == 0) continue;
        const int I = (row0 + t) % Nb;
        const int bh_t = (row0 + t) / Nb;
        mbar_expect_tx(bar_q_full + 8 * t, C::Q_BYTES);
        const uint32_t dst = sbase + C::OFF_Q + t * C::Q_BYTES;
        if (F8 || D == 64) {
          tma_load_4d(dst, &tm_q, bar_q_full + 8 * t, 0, I * BS, bh_t % prm.H, bh_t / prm.H);
        } else {
          tma_load_4d(dst, &tm_q, bar_q_full + 8 * t, 0, I * BS, bh_t % prm.H, bh_t / prm.H);
          tma_load_4d(dst + C::Q_BYTES / 2, &tm_q, bar_q_full + 8 * t, 64, I * BS, bh_t % prm.H, bh_t / prm.H);
        }
      }
      int stage = 0;
      uint32_t phase = 0;
      auto load_tile = [&](bool is_v, int t, int j) -> bool {
        if (!mbar_wait(bar_kv_empty + 8 * stage, phase ^ 1u, abort_flag, prm.status)) return false;
        const int J = dense ? j : __ldg(prm.col_idx + lbeg[t] + j);
        const int bh_t = (row0 + t) / Nb;
        const int hh = bh_t % prm.H, bb = bh_t / prm.H;
        const uint32_t dst = sbase + C::OFF_RING + stage * C::STAGE_BYTES;
        const uint32_t bar = bar_kv_full + 8 * stage;
        if (is_v) {
          mbar_expect_tx(bar, C::V_BYTES);
          tma_load_4d(dst, &tm_v, bar, 0, J * BS, hh, bb);
          if (D == 128) tma_load_4d(dst + C::V_BYTES / 2, &tm_v, bar, 64, J * BS, hh, bb);
        } else {
          mbar_expect_tx(bar, C::Q_BYTES);
          tma_load_4d(dst, &tm_k, bar, 0, J * BS, hh, bb);
          if (!F8 && D == 128) tma_load_4d(dst + C::Q_BYTES / 2, &tm_k, bar, 64, J * BS, hh, bb);
        }
        if (++stage == C::STAGES) { stage = 0; phase ^= 1u; }
        return true;
      };
      // tile order must match the MMA warp's consumption order exactly
      for (int t = 0; t < NT && ok; ++t)
        if (nl[t] > 0) ok = load_tile(false, t, 0);
      const int nmax = nl[0] > nl[1] ? nl[0] : nl[1];
      for (int j = 0; j < nmax && ok; ++j)
        for (int t = 0; t < NT && ok; ++t) {
          if (j < nl[t]) ok = load_tile(true, t, j);
          if (ok && j + 1 < nl[t]) ok = load_tile(false, t, j + 1);
        }
    }
  } else if (warp == W_MMA) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t IDESC_QK = instr_desc(128, BS, F8 ? 0 : 1, false);
      constexpr uint32_t IDESC_PV = instr_desc(128, D, 1, true);
      constexpr int QK_KSTEP_BYTES = 32;                          // 16 bf16 or 32 e4m3
      constexpr int QK_KSTEPS = D * C::QK_ELEM / QK_KSTEP_BYTES;
      constexpr int QK_PANEL_BYTES = BS * 128;                    // 128 rows x 128-byte swizzle row
      bool ok = true;
      int stage = 0;
      uint32_t phase = 0;
      auto advance = [&]() { if (++stage == C::STAGES) { stage = 0; phase ^= 1u; } };
      auto issue_s = [&](int t, int j) -> bool {
        if (j == 0 && !mbar_wait(bar_q_full + 8 * t, 0, abort_flag, prm.status)) return false;
        if (!mbar_wait(bar_kv_full + 8 * stage, phase, abort_flag, prm.status)) return false;
        tc_fence_after();
        const uint32_t qa = sbase + C::OFF_Q + t * C::Q_BYTES;
        const uint32_t ka = sbase + C::OFF_RING + stage * C::STAGE_BYTES;
        const uint32_t d_tmem = tmem_base + 128 * t;
#pragma unroll
        for (int kk = 0; kk < QK_KSTEPS; ++kk) {
          const uint32_t off = (kk / 4) * QK_PANEL_BYTES + (kk % 4) * QK_KSTEP_BYTES;
          tc_mma_ss<F8>(d_tmem, smem_desc(qa + off, 16, 1024), smem_desc(ka + off, 16, 1024), IDESC_QK,
                        kk > 0 ? 1u : 0u);
        }
        tc_commit(bar_kv_empty + 8 * stage);
        tc_commit(bar_s_full + 8 * t);
        advance();
        return true;
      };
      auto issue_pv = [&](int t, int j) -> bool {
        if (!mbar_wait(bar_p_full + 8 * t, (uint32_t)(j & 1), abort_flag, prm.status)) return false;
        if (!mbar_wait(bar_kv_full + 8 * stage, phase, abort_flag, prm.status)) return false;
        tc_fence_after();
        const uint32_t va = sbase + C::OFF_RING + stage * C::STAGE_BYTES;
        const uint32_t p_tmem = tmem_base + 128 * t;
        const uint32_t o_tmem = tmem_base + 128 * NT + 128 * t;
#pragma unroll
        for (int kk = 0; kk < BS / 16; ++kk)
          tc_mma_ts(o_tmem, p_tmem + 8 * kk, smem_desc(va + kk * 2048, BS * 128, 1024), IDESC_PV,
                    (j > 0 || kk > 0) ? 1u : 0u);
        tc_commit(bar_kv_empty + 8 * stage);
        if (j == nl[t] - 1) tc_commit(bar_o_done + 8 * t);
        advance();
        return true;
      };
      for (int t = 0; t < NT && ok; ++t)
        if (nl[t] > 0) ok = issue_s(t, 0);
      const int nmax = nl[0] > nl[1] ? nl[0] : nl[1];
      for (int j = 0; j < nmax && ok; ++j)
        for (int t = 0; t < NT && ok; ++t) {
          if (j < nl[t]) ok = issue_pv(t, j);
          if (ok && j + 1 < nl[t]) ok = issue_s(t, j + 1);
        }
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue
    const int t = warp >> 2;
    const int r = row0 + t;
    const int n = nl[t];
    const int row = (warp & 3) * 32 + lane;                  // row of the tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t s_tmem = tmem_base + lane_addr + 128 * t;
    const uint32_t o_tmem = tmem_base + lane_addr + 128 * NT + 128 * t;
    if (r < prm.R) {
      const int I = r % Nb;
      const int bh_t = r / Nb;
      const int qi = I * BS + row;
      const int tail_keys = prm.N - (Nb - 1) * BS;           // valid keys of the last block
      float m_used = -INFINITY, l = 0.f;
      float c = prm.scale_log2;
      float qs = 1.f;
      if (F8) qs = prm.q_scale[(long long)bh_t * Nb + I];
      bool ok = true;
      for (int j = 0; j < n; ++j) {
        const int J = dense ? j : __ldg(prm.col_idx + lbeg[t] + j);
        if (F8) c = prm.scale_log2 * qs * __ldg(prm.k_scale + (long long)bh_t * Nb + J);
        if (!mbar_wait(bar_s_full + 8 * t, (uint32_t)(j & 1), abort_flag, prm.status)) { ok = false; break; }
        tc_fence_after();
        uint32_t sv[128];
        tmem_ld32(s_tmem + 0, sv + 0);
        tmem_ld32(s_tmem + 32, sv + 32);
        tmem_ld32(s_tmem + 64, sv + 64);
        tmem_ld32(s_tmem + 96, sv + 96);
        tc_wait_ld();
        if (J == Nb - 1 && tail_keys < BS) {
#pragma unroll
          for (int i = 0; i < 128; ++i)
            if (i >= tail_keys) sv[i] = 0xff800000u;          // -inf
        }
        float mx = -INFINITY;
#pragma unroll
        for (int i = 0; i < 128; ++i) mx = fmaxf(mx, __uint_as_float(sv[i]));
        mx *= c;
        // lazy rescale: move the reference maximum only when it would grow by more than 2^8
        const bool need = mx > m_used + 8.0f;
        if (__any_sync(0xffffffffu, need)) {
          const float m_new = fmaxf(m_used, mx);
          const float alpha = ex2(m_used - m_new);            // first block: exp2(-inf) = 0
          l *= alpha;
          m_used = m_new;
          if (j > 0) {
#pragma unroll
            for (int cc = 0; cc < D; cc += 32) {
              uint32_t ov[32];
              tmem_ld32(o_tmem + cc, ov);
              tc_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
              tmem_st32(o_tmem + cc, ov);
            }
          }
        }
        float sum = 0.f;
#pragma unroll
        for (int cc = 0; cc < 128; cc += 32) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float p0 = ex2(fmaf(__uint_as_float(sv[cc + 2 * i]), c, -m_used));
            const float p1 = ex2(fmaf(__uint_as_float(sv[cc + 2 * i + 1]), c, -m_used));
            sum += p0 + p1;
            pk[i] = pack_bf16(p0, p1);
          }
          tmem_st16(s_tmem + cc / 2, pk);
        }
        l += sum;
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p_full + 8 * t);
      }
      // ---- epilogue
      __nv_bfloat16* orow = prm.o + (long long)(bh_t / prm.H) * prm.so.b + (long long)(bh_t % prm.H) * prm.so.h +
                            (long long)qi * prm.so.n;
      if (n == 0) {
        if (qi < prm.N) {
#pragma unroll
          for (int cc = 0; cc < D; cc += 8) *reinterpret_cast<uint4*>(orow + cc) = make_uint4(0, 0, 0, 0);
          if (prm.lse) prm.lse[(long long)bh_t * prm.N + qi] = -INFINITY;
        }
      } else if (ok && mbar_wait(bar_o_done + 8 * t, 0, abort_flag, prm.status)) {
        tc_fence_after();
        const float inv = 1.0f / l;
#pragma unroll
        for (int cc = 0; cc < D; cc += 32) {
          uint32_t ov[32];
          tmem_ld32(o_tmem + cc, ov);
          tc_wait_ld();
          if (qi < prm.N) {
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint4 w;
              w.x = pack_bf16(__uint_as_float(ov[i + 0]) * inv, __uint_as_float(ov[i + 1]) * inv);
              w.y = pack_bf16(__uint_as_float(ov[i + 2]) * inv, __uint_as_float(ov[i + 3]) * inv);
              w.z = pack_bf16(__uint_as_float(ov[i + 4]) * inv, __uint_as_float(ov[i + 5]) * inv);
              w.w = pack_bf16(__uint_as_float(ov[i + 6]) * inv, __uint_as_float(ov[i + 7]) * inv);
              *reinterpret_cast<uint4*>(orow + cc + i) = w;
            }
          }
        }
        if (prm.lse && qi < prm.N)
          prm.lse[(long long)bh_t * prm.N + qi] = (m_used + log2f(l)) * 0.6931471805599453f;
      }
    }
  }

  // ---------------------------------------------------------------- tear-down
  if (*abort_flag) {
    // give copies and MMAs still in flight time to land before shared memory and TMEM go away
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == W_MMA) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*encode_fn_t)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                CUtensorMapFloatOOBfill);

static encode_fn_t get_encode() {
  static encode_fn_t fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<encode_fn_t>(p);
  }
  return fn;
}

// [B,H,N,d] tensor with element strides s, as a 4-D map (d, N, H, B); box = 128 bytes x 128 rows.
static int make_map(CUtensorMap* map, const void* ptr, int elem_bytes, int B, int H, int N, int d,
                    const Strides& s) {
  encode_fn_t enc = get_encode();
  if (!enc) return SVA_ERR_CUDA;
  cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)H, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)s.n * elem_bytes, (cuuint64_t)s.h * elem_bytes, (cuuint64_t)s.b * elem_bytes};
  // a size-1 dimension may carry any stride; give it a legal one
  if (H == 1) strides[1] = strides[0] * (cuuint64_t)N;
  if (B == 1) strides[2] = strides[1] * (cuuint64_t)H;
  for (int i = 0; i < 3; ++i)
    if (strides[i] % 16 != 0 || strides[i] == 0) return SVA_ERR_ALIGNMENT;
  int inner = 128 / elem_bytes;
  if (inner > d) inner = d;
  cuuint32_t box[4] = {(cuuint32_t)inner, (cuuint32_t)BS, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult rc = enc(map, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
                    const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    (inner * elem_bytes == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? SVA_OK : SVA_ERR_CUDA;
}

static int g_tiles_per_cta = 2;   // bring-up switch, see sva_debug_set_tiles_per_cta

template <int D, int NT, bool F8>
static int launch_cfg(const Dims& m, const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                      const AttnParams& prm, cudaStream_t st) {
  using C = Cfg<D, NT, F8>;
  auto kern = attn_sm100_kernel<D, NT, F8>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess)
    return SVA_ERR_CUDA;
  const int grid = (m.R + NT - 1) / NT;
  kern<<<grid, C::THREADS, C::SMEM_BYTES, st>>>(tq, tk, tv, prm);
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

int launch_attn_sm100(const Dims& m, const sva_problem_t* p, const void* q, const void* k,
                      const void* v, const float* qs, const float* ks, const int32_t* row_ptr,
                      const int32_t* col_idx, void* o, float* lse, int32_t* status,
                      cudaStream_t st) {
  if (m.block != BS || m.d != 128) return SVA_ERR_UNSUPPORTED;
  CUtensorMap tq, tk, tv;
  const int eb = m.fp8 ? 1 : 2;
  int rc;
  if ((rc = make_map(&tq, q, eb, m.B, m.H, m.N, m.d, make_strides(p->q_stride))) != SVA_OK) return rc;
  if ((rc = make_map(&tk, k, eb, m.B, m.H, m.N, m.d, make_strides(p->k_stride))) != SVA_OK) return rc;
  if ((rc = make_map(&tv, v, 2, m.B, m.H, m.N, m.d, make_strides(p->v_stride))) != SVA_OK) return rc;
  AttnParams prm;
  prm.row_ptr = row_ptr; prm.col_idx = col_idx; prm.q_scale = qs; prm.k_scale = ks;
  prm.o = (__nv_bfloat16*)o; prm.lse = lse; prm.status = status;
  prm.so = make_strides(p->o_stride);
  prm.H = m.H; prm.N = m.N; prm.Nb = m.Nb; prm.R = m.R;
  prm.scale_log2 = m.scale * 1.4426950408889634f;
  // a CTA's tiles must belong to one head: pair tiles only when Nb is even
  const int nt = (g_tiles_per_cta == 2 && m.Nb % 2 == 0) ? 2 : 1;
  if (m.fp8) return nt == 2 ? launch_cfg<128, 2, true>(m, tq, tk, tv, prm, st)
                            : launch_cfg<128, 1, true>(m, tq, tk, tv, prm, st);
  return nt == 2 ? launch_cfg<128, 2, false>(m, tq, tk, tv, prm, st)
                 : launch_cfg<128, 1, false>(m, tq, tk, tv, prm, st);
}

void set_tiles_per_cta(int n) { g_tiles_per_cta = n == 1 ? 1 : 2; }

}  // namespace sva
