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
#include "tc_ptx.cuh"

namespace sva {

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
  long long* prof;            // optional timeline buffer (tuning aid), normally null
  int debug;                  // tuning aid: bit0 = skip the softmax arithmetic (wrong results)
};

// Timeline probe: CTA 64 records clock64() for iterations 16..23, [role][j-16][event].
#define SVA_PROF(role, j, ev)                                                                   \
  do {                                                                                          \
    if (prm.prof && blockIdx.x == 64 && (j) >= 16 && (j) < 24)                                  \
      prm.prof[(((role) * 8) + ((j) - 16)) * 8 + (ev)] = clock64();                             \
  } while (0)

template <int D, int NT, bool F8>
struct Cfg {
  static constexpr int QK_ELEM = F8 ? 1 : 2;
  static constexpr int Q_BYTES = BS * D * QK_ELEM;       // one Q (or K) tile
  static constexpr int VH_BYTES = (BS / 2) * D * 2;      // half a V tile: 64 keys
  static constexpr int K_SLOT = BS * D * 2;              // slot size of a K tile (bf16 size also for e4m3)
  static constexpr int KS = NT == 2 ? 1 : 2;             // K tiles in flight per query tile
  static constexpr int VS = NT == 2 ? 3 : 6;             // V half-tiles in flight per query tile
  static constexpr int THREADS = NT * 128 + 128;         // softmax warpgroups + one warpgroup for TMA/MMA
  static constexpr int TMEM_COLS = 512;
  // dynamic shared memory: 1024-aligned tiles first, then the control block
  static constexpr int OFF_Q = 0;
  static constexpr int Q_SLOT = (Q_BYTES + 1023) / 1024 * 1024;
  static constexpr int OFF_K = OFF_Q + NT * Q_SLOT;      // K slots of tile t at OFF_K + t*KS*K_SLOT
  static constexpr int OFF_V = OFF_K + NT * KS * K_SLOT; // V half slots of tile t at OFF_V + t*VS*VH_BYTES
  static constexpr int OFF_CTRL = OFF_V + NT * VS * VH_BYTES;
  static constexpr int CTRL_BYTES = 384;
  static constexpr int SMEM_BYTES = OFF_CTRL + CTRL_BYTES + 1024;   // + alignment slack
};

// control block layout (bytes from OFF_CTRL):
//   0   q_full[2]   16 s_full[2]   32 p_full[t] at 32 + 16*t   64 o_done[2]
//   96 + 128*t : k_full[2] | +16 k_empty[2] | +32 v_full[6] | +80 v_empty[6]
//   352 tmem_base   356 abort   360 n_list[2]   368 beg[2]   376 issue lock

template <int D, int NT, bool F8>
__global__ void __launch_bounds__(NT * 128 + 128, 1)
attn_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const AttnParams prm) {
  using C = Cfg<D, NT, F8>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  uint8_t* ctrl = smem + C::OFF_CTRL;
  const uint32_t cbase = sbase + C::OFF_CTRL;
  const uint32_t bar_q_full = cbase + 0, bar_s_full = cbase + 16, bar_p_half = cbase + 32,
                 bar_o_done = cbase + 64, bar_tile = cbase + 96;
  volatile uint32_t* tmem_base_p = reinterpret_cast<volatile uint32_t*>(ctrl + 352);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 356);
  volatile int* n_list = reinterpret_cast<volatile int*>(ctrl + 360);
  volatile int* beg_list = reinterpret_cast<volatile int*>(ctrl + 368);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int W_PROD = 4 * NT, W_MMA = 4 * NT + 2;   // producers: W_PROD + t; MMA issuers: W_MMA + t
  const int row0 = blockIdx.x * NT;                    // first CSR row of this CTA
  const int Nb = prm.Nb;
  const bool dense = prm.row_ptr == nullptr;

  // ---------------------------------------------------------------- set-up
  if (threadIdx.x == 0) {
    for (int t = 0; t < 2; ++t) {
      mbar_init(bar_q_full + 8 * t, 1);
      mbar_init(bar_s_full + 8 * t, 1);
      mbar_init(bar_p_half + 16 * t, 128);
      mbar_init(bar_p_half + 16 * t + 8, 128);
      mbar_init(bar_o_done + 8 * t, 1);
    }
    for (int s = 0; s < 32; ++s) mbar_init(bar_tile + 8 * s, 1);      // k/v full and empty, both tiles
    *abort_flag = 0;
    *reinterpret_cast<volatile int*>(ctrl + 376) = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == W_PROD && lane == 0) {
    prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
  }
  if (warp == W_MMA) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(cbase + 352), "r"((uint32_t)C::TMEM_COLS) : "memory");
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

  // Register re-partition: the TMA/MMA warpgroup needs few registers, a softmax thread holds a
  // whole 128-wide row.  Issued at the top of each branch so the limit is tied to that branch.
  if (warp >= 4 * NT) {
    if (NT == 2) asm volatile("setmaxnreg.dec.sync.aligned.u32 96;");
    if (warp >= W_PROD && warp < W_PROD + NT) {
      // ---------------------------------------------------------- producer of tile t
      // lane 0 streams Q and the K tiles, lane 1 the V half-tiles (64 keys each); the two streams
      // have their own slots and barriers so that V runs a whole block ahead.
      const int t = warp - W_PROD;
      const int n = nl[t];
      const int bh_t = (row0 + t) / Nb;
      const int hh = bh_t % prm.H, bb = bh_t / prm.H;
      const uint32_t bt = bar_tile + 128 * t;
      if (lane == 0 && n > 0) {
        const int I = (row0 + t) % Nb;
        mbar_expect_tx(bar_q_full + 8 * t, C::Q_BYTES);
        const uint32_t qdst = sbase + C::OFF_Q + t * C::Q_SLOT;
        tma_load_4d(qdst, &tm_q, bar_q_full + 8 * t, 0, I * BS, hh, bb);
        if (!F8 && D == 128) tma_load_4d(qdst + C::Q_BYTES / 2, &tm_q, bar_q_full + 8 * t, 64, I * BS, hh, bb);
        int ks = 0;
        uint32_t kphase = 0;
        for (int j = 0; j < n; ++j) {
          if ((prm.debug & 16) && t == 0 && j >= 1) break;   // test aid: starve the pipeline so that a wait runs out
          if (!mbar_wait(bt + 16 + 8 * ks, kphase ^ 1u, abort_flag, prm.status)) break;
          const int J = dense ? j : __ldg(prm.col_idx + lbeg[t] + j);
          const uint32_t dst = sbase + C::OFF_K + (t * C::KS + ks) * C::K_SLOT;
          const uint32_t bar = bt + 8 * ks;
          mbar_expect_tx(bar, C::Q_BYTES);
          tma_load_4d(dst, &tm_k, bar, 0, J * BS, hh, bb);
          if (!F8 && D == 128) tma_load_4d(dst + C::Q_BYTES / 2, &tm_k, bar, 64, J * BS, hh, bb);
          if (++ks == C::KS) { ks = 0; kphase ^= 1u; }
        }
      } else if (lane == 1 && n > 0) {
        int vs = 0;
        uint32_t vphase = 0;
        for (int i = 0; i < 2 * n; ++i) {
          if (!mbar_wait<60>(bt + 80 + 8 * vs, vphase ^ 1u, abort_flag, prm.status)) break;
          const int J = dense ? (i >> 1) : __ldg(prm.col_idx + lbeg[t] + (i >> 1));
          const uint32_t dst = sbase + C::OFF_V + (t * C::VS + vs) * C::VH_BYTES;
          const uint32_t bar = bt + 32 + 8 * vs;
          mbar_expect_tx(bar, C::VH_BYTES);
          tma_load_4d(dst, &tm_v, bar, 0, J * BS + (i & 1) * (BS / 2), hh, bb);
          if (D == 128) tma_load_4d(dst + C::VH_BYTES / 2, &tm_v, bar, 64, J * BS + (i & 1) * (BS / 2), hh, bb);
          if (++vs == C::VS) { vs = 0; vphase ^= 1u; }
        }
      }
    } else if (warp >= W_MMA && warp < W_MMA + NT) {
      // ---------------------------------------------------------- MMA issuer of tile t (one lane)
      // Per block j: P V (two V half-tiles), then S(j+1).  Each issuer blocks only on its own
      // tile's barriers; a lock taken around every group of MMAs makes the two tiles' groups
      // reach the tensor pipe one after the other, which keeps the two softmax warpgroups out of
      // phase (so that one tile's exponentials overlap the other tile's MMAs).
      const int t = warp - W_MMA;
      if (lane == 0 && nl[t] > 0) {
        const uint32_t IDESC_QK = instr_desc(128, BS, F8 ? 0 : 1, false);
        const uint32_t IDESC_PV = instr_desc(128, D, 1, true);
        constexpr int QK_KSTEPS = D * C::QK_ELEM / 32;              // 32 bytes of K per MMA
        const int n = nl[t];
        int* lock = reinterpret_cast<int*>(ctrl + 376);
        const uint32_t bt = bar_tile + 128 * t;
        const uint64_t qd = smem_desc(sbase + C::OFF_Q + t * C::Q_SLOT, 16, 1024);
        const uint64_t kdesc0 = smem_desc(sbase + C::OFF_K + t * C::KS * C::K_SLOT, 16, 1024);
        // V half-tile: two 64-wide d panels of 64 keys x 128 bytes, panel stride = half of the slot
        const uint64_t vdesc0 = smem_desc(sbase + C::OFF_V + t * C::VS * C::VH_BYTES, C::VH_BYTES / 2, 1024);
        const uint32_t s_tmem = tmem_base + 128 * t;
        const uint32_t o_tmem = tmem_base + 128 * NT + 128 * t;
        int ks = 0, vs = 0;
        uint32_t kphase = 0, vphase = 0;
        auto acquire = [&]() -> bool {
          if (NT == 1 || (prm.debug & 8)) return true;
          uint32_t spins = 0;
          const long long t0 = clock64();
          while (atomicCAS(lock, 0, 1) != 0) {
            if ((++spins & 63u) == 0u) {
              if (*abort_flag) return false;
              if (clock64() - t0 > g_wait_limit) {
                *abort_flag = 1;
                if (prm.status) atomicOr(prm.status, SVA_DEV_TIMEOUT);
                return false;
              }
            }
          }
          return true;
        };
        auto release = [&]() { if (NT == 2 && !(prm.debug & 8)) atomicExch(lock, 0); };
        auto issue_s = [&](int j) {                                  // K(j) must be resident
          const uint64_t kd = kdesc0 + (uint64_t)(ks * (C::K_SLOT >> 4));
#pragma unroll
          for (int kk = 0; kk < QK_KSTEPS; ++kk) {
            constexpr int PANEL16 = (BS * 128) >> 4;
            const uint64_t off = (uint64_t)((kk / 4) * PANEL16 + (kk % 4) * 2);
            tc_mma_ss<F8>(s_tmem, qd + off, kd + off, IDESC_QK, kk > 0 ? 1u : 0u, 1u);
          }
          tc_commit(bt + 16 + 8 * ks, 1u);
          tc_commit(bar_s_full + 8 * t, 1u);
          SVA_PROF(2 + t, j - 1, 5);
          if (++ks == C::KS) { ks = 0; kphase ^= 1u; }
        };
        auto issue_pv_half = [&](int j, int half) {                  // V half-tile vs must be resident
          const uint64_t vd = vdesc0 + (uint64_t)(vs * (C::VH_BYTES >> 4));
#pragma unroll
          for (int kk = 0; kk < BS / 32; ++kk)
            tc_mma_ts(o_tmem, s_tmem + 8 * (kk + half * (BS / 32)), vd + (uint64_t)(kk * (2048 >> 4)), IDESC_PV,
                      (j > 0 || half > 0 || kk > 0) ? 1u : 0u, 1u);
          tc_commit(bt + 80 + 8 * vs, 1u);
          if (++vs == C::VS) { vs = 0; vphase ^= 1u; }
        };
        bool ok = mbar_wait(bar_q_full + 8 * t, 0, abort_flag, prm.status) &&
                  mbar_wait(bt + 8 * ks, kphase, abort_flag, prm.status);
        if (ok) {
          tc_fence_after();
          ok = acquire();
          if (ok) { issue_s(0); release(); }
        }
        for (int j = 0; j < n && ok; ++j) {
          // One group per block: P V (two V half-tiles) directly followed by S of the next block.
          // The tensor pipe drains whenever consecutive MMAs change kind (A from shared memory
          // vs tensor memory, or another instruction descriptor), so kinds are kept together and
          // the other tile's group never lands in the middle.
          const bool more = j + 1 < n;
          int vs2 = vs + 1;
          uint32_t vphase2 = vphase;
          if (vs2 == C::VS) { vs2 = 0; vphase2 ^= 1u; }
          ok = mbar_wait(bar_p_half + 16 * t, (uint32_t)(j & 1), abort_flag, prm.status) &&
               mbar_wait(bt + 32 + 8 * vs, vphase, abort_flag, prm.status) &&
               mbar_wait(bt + 32 + 8 * vs2, vphase2, abort_flag, prm.status);
          if (!ok) break;
          SVA_PROF(2 + t, j, 1);
          tc_fence_after();
          ok = acquire();
          if (!ok) break;
          SVA_PROF(2 + t, j, 0);
          issue_pv_half(j, 0);
          issue_pv_half(j, 1);
          if (j == n - 1) tc_commit(bar_o_done + 8 * t, 1u);
          SVA_PROF(2 + t, j, 2);
          if (more && !mbar_test(bt + 8 * ks, kphase)) {
            // K(j+1) has not landed yet: let the other tile use the pipe meanwhile
            release();
            ok = mbar_wait(bt + 8 * ks, kphase, abort_flag, prm.status) && acquire();
            if (!ok) break;
          }
          if (more) issue_s(j + 1);
          release();
        }
      }
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue
    // warpgroup t owns tile t; thread <-> query row <-> TMEM lane, all 128 key columns
    if (NT == 2) asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
    const int t = warp >> 2;
    const int r = row0 + t;
    const int n = nl[t];
    const int row = (warp & 3) * 32 + lane;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t s_tmem = tmem_base + lane_addr + 128 * t;
    const uint32_t o_tmem = tmem_base + lane_addr + 128 * NT + 128 * t;
    const bool probe = (threadIdx.x & 127) == 0;
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
        const int valid = (J == Nb - 1) ? tail_keys : BS;      // key columns of this block that exist
        if (probe) SVA_PROF(t, j, 0);
        if (!mbar_wait(bar_s_full + 8 * t, (uint32_t)(j & 1), abort_flag, prm.status)) { ok = false; break; }
        if (probe) SVA_PROF(t, j, 1);
        tc_fence_after();
        if (prm.debug & 1) {
          tc_fence_before();
          mbar_arrive(bar_p_half + 16 * t);
          l = 1.f;
          continue;
        }
        if (valid < BS) {
          // ragged last key block: keys that do not exist become -inf in TMEM before S is read (a short
          // rolled loop -- this keeps 128 compare/select pairs out of the hot instruction stream)
#pragma unroll 1
          for (int i = valid; i < BS; ++i) tmem_st1(s_tmem + i, 0xff800000u);
          tc_wait_st();
        }
        // ---- row maximum over the 128 columns (whole row in registers)
        uint32_t sv[128];
        tmem_ld32(s_tmem + 0, sv + 0);
        tmem_ld32(s_tmem + 32, sv + 32);
        tmem_ld32(s_tmem + 64, sv + 64);
        tmem_ld32(s_tmem + 96, sv + 96);
        tc_wait_ld();
        if (probe) SVA_PROF(t, j, 2);
        float mxa = -INFINITY, mxb = -INFINITY, mxc = -INFINITY, mxd = -INFINITY;
#pragma unroll
        for (int i = 0; i < 128; i += 8) {
          mxa = max3(mxa, __uint_as_float(sv[i + 0]), __uint_as_float(sv[i + 1]));
          mxb = max3(mxb, __uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3]));
          mxc = max3(mxc, __uint_as_float(sv[i + 4]), __uint_as_float(sv[i + 5]));
          mxd = max3(mxd, __uint_as_float(sv[i + 6]), __uint_as_float(sv[i + 7]));
        }
        const float mx = fmaxf(fmaxf(mxa, mxb), fmaxf(mxc, mxd)) * c;
        // lazy rescale: move the reference maximum only when it would grow by more than 2^32 (P then stays
        // below 2^32 and a row sum below 2^32 * N: far inside fp32 and bf16 range, and rescales of O are rare)
        if (__any_sync(0xffffffffu, mx > m_used + 32.0f)) {
          const float m_new = fmaxf(m_used, mx);
          const float alpha = ex2(m_used - m_new);            // first block: exp2(-inf) = 0
          l *= alpha;
          m_used = m_new;
          if (j > 0) {
#pragma unroll 1
            for (int cc = 0; cc < D; cc += 16) {
              uint32_t ov[16];
              tmem_ld16(o_tmem + cc, ov);
              tc_wait_ld();
#pragma unroll
              for (int i = 0; i < 16; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha);
              tmem_st16(o_tmem + cc, ov);
            }
          }
        }
        if (probe) SVA_PROF(t, j, 3);
        // ---- P = 2^(S*c - m_used); the packed bf16 pairs overwrite sv[0..63]
        const float nm = -m_used;
        const uint64_t c2 = pack2(c, c), nm2 = pack2(nm, nm);
        uint64_t sum2 = pack2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 128; i += 2) {
          float x0, x1;
          unpack2(fma2(pack2(__uint_as_float(sv[i]), __uint_as_float(sv[i + 1])), c2, nm2), x0, x1);
          const float p0 = ex2(x0), p1 = ex2(x1);
          sum2 = add2(sum2, pack2(p0, p1));
          sv[i / 2] = pack_bf16(p0, p1);
          if (i == 62) tmem_st32(s_tmem, sv);
        }
        float sum_a, sum_b;
        unpack2(sum2, sum_a, sum_b);
        tmem_st32(s_tmem + 32, sv + 32);
        l += sum_a + sum_b;
        if (probe) SVA_PROF(t, j, 4);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p_half + 16 * t);
        if (probe) SVA_PROF(t, j, 5);
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
                    const Strides& s, int box_rows) {
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
  cuuint32_t box[4] = {(cuuint32_t)inner, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult rc = enc(map, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
                    const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    (inner * elem_bytes == 128) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? SVA_OK : SVA_ERR_CUDA;
}

static int g_tiles_per_cta = 2;   // bring-up switch, see sva_debug_set_tiles_per_cta
static long long* g_prof = nullptr;   // tuning aid, see sva_debug_set_prof_buffer
static int g_debug = 0;

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
  if ((rc = make_map(&tq, q, eb, m.B, m.H, m.N, m.d, make_strides(p->q_stride), BS)) != SVA_OK) return rc;
  if ((rc = make_map(&tk, k, eb, m.B, m.H, m.N, m.d, make_strides(p->k_stride), BS)) != SVA_OK) return rc;
  if ((rc = make_map(&tv, v, 2, m.B, m.H, m.N, m.d, make_strides(p->v_stride), BS / 2)) != SVA_OK) return rc;
  AttnParams prm;
  prm.row_ptr = row_ptr; prm.col_idx = col_idx; prm.q_scale = qs; prm.k_scale = ks;
  prm.o = (__nv_bfloat16*)o; prm.lse = lse; prm.status = status;
  prm.so = make_strides(p->o_stride);
  prm.H = m.H; prm.N = m.N; prm.Nb = m.Nb; prm.R = m.R;
  prm.scale_log2 = m.scale * 1.4426950408889634f;
  prm.prof = g_prof;
  prm.debug = g_debug;
  // a CTA's tiles must belong to one head: pair tiles only when Nb is even
  const int nt = (g_tiles_per_cta == 2 && m.Nb % 2 == 0) ? 2 : 1;
  if (m.fp8) return nt == 2 ? launch_cfg<128, 2, true>(m, tq, tk, tv, prm, st) : launch_cfg<128, 1, true>(m, tq, tk, tv, prm, st);
  return nt == 2 ? launch_cfg<128, 2, false>(m, tq, tk, tv, prm, st) : launch_cfg<128, 1, false>(m, tq, tk, tv, prm, st);
}

void set_tiles_per_cta(int n) { g_tiles_per_cta = n == 1 ? 1 : 2; }
void set_prof_buffer(void* p) { g_prof = (long long*)p; }
void set_debug_mode(int v) { g_debug = v; }
int set_wait_limit(long long cycles) {
  if (cycles <= 0) cycles = WAIT_LIMIT_CYCLES;
  return cudaMemcpyToSymbol(g_wait_limit, &cycles, sizeof(cycles)) == cudaSuccess ? 0 : 1;
}

}  // namespace sva
