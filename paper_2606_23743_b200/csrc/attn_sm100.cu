// Block-sparse / dense attention forward for sm_100a (tcgen05 / TMEM / TMA): every MMA of one form.
// (Paper: critical blocks "computed exactly"; dense fallback.)
//
// The tensor pipe drains (~280 cycles, measured) whenever two consecutive MMAs differ in kind:
// A operand from shared memory vs tensor memory, or another instruction descriptor.  Here both
// S = Q K^T and O += P V have the same form -- A from TENSOR memory (Q resp. P, bf16 pairs), B
// from shared memory, K-major, M = N = 128 -- so the pipe never drains:
//   * Q is written into TMEM once per row by the softmax threads (128-token blocks: by the group that finishes
//     the row first, about a tile before the row ends, from a tile that TMA has put into the group's idle output
//     staging panel; otherwise by both groups in the epilogue, straight from global memory);
//   * V: in the two-step form it is consumed transposed (V^T tiles: d rows, keys contiguous) from a tiled transposed
//     copy that a small kernel writes into the caller's workspace first, so that P V has the form of S.  The one-call
//     entry points read V where it lies instead (template switch VMN: an MN-major B operand, a second instruction
//     descriptor): the pipe is idle often enough for the switch to cost 1 % of the cycles, and the step is faster
//     without the copy's pass over the HBM.
// The kernel is persistent: one CTA per SM takes rows (one row = one query block of one head, 128
// query rows) from a device-wide counter until none is left.  All barriers keep running across rows
// (every role derives the same phase counters from the same row sequence), so the producers run
// ahead into the next row while the softmax groups finish the current one.
//   warps 0-3, 4-7  two softmax warpgroups; they take the kept key blocks alternately (even / odd
//                   position in the row's list); thread <-> query row <-> TMEM lane
//   warp  8         producer of the K tiles (TMA, one lane)
//   warp  9         issues the Q K^T MMAs (one lane); owns the TMEM allocation
//   warp  10        issues the P V MMAs (one lane)
//   warp  11        producer of the V^T tiles (TMA, one lane)
// TMEM columns: S of even blocks 0..127, S of odd blocks 128..255, O 256..383, Q 384..447 (bf16
// pairs), P 448..511 (bf16 pairs).  Because P has columns of its own, an S buffer is free again as
// soon as its warpgroup has read it into registers: the MMA warp computes S(j+2) while the softmax
// of block j is still running.  P is single-buffered: block j's P is stored once P V(j-1) has
// completed, which also staggers the two warpgroups so that one group's exponentials overlap the
// other group's maximum pass and stores.
//
// The two warpgroups share one O accumulator, so they share the reference exponent of every row:
// the group working on block j takes the reference left by block j-1 (published through shared
// memory right after that block's row-maximum pass), raises it only when the new row maximum
// exceeds it by more than 2^LAZY_LOG2, and in that (rare) case rescales its row of O once P V(j-1)
// has completed.  Row sums are kept per group and merged in the epilogue, where each group
// normalises its half of O into a swizzled staging panel that one TMA tile store writes out.
//
// e4m3 Q/K (template switch): Q goes into TMEM as bytes (32 columns), a K tile is one 128 x 128-byte
// panel, S takes four kind::f8f6f4 MMAs (A from TMEM like everything else), and the exponent's scale is
// softmax_scale * q_scale[query block] * k_scale[key block] per block; P, V and O stay bf16 / fp32.
//
// 64-token blocks (template switch): the MMA tile stays 128 x 128, so one row of work is two adjacent
// query blocks (A, B) and one tile two key blocks out of the ascending union of A's and B's lists
// (pair_lists_kernel builds the tile lists).  The K / V^T producers fetch the two halves of a tile
// from two key blocks; the softmax excludes, per query block, the half it does not keep -- with -inf
// as the additive constant of the exponentials' FMA, at no cost -- and masks a ragged tail per half.
// The price is the part of the union one of the two query blocks does not keep (adjacent query
// blocks share most of their lists).
//
// Every wait is bounded: when one expires the CTA sets SVA_DEV_TIMEOUT, all roles leave their
// loops, TMEM is released and the kernel returns.  Parity waits never run a whole phase ahead of
// their barrier (each wait on a barrier is preceded by a wait on its previous phase).
#include <mutex>
#include <type_traits>

#include "tc_ptx.cuh"

// Timeline stamps for tuning builds only (-DSVA_TIMELINE; never in the shipped library): CTA 0 appends
// {cycle << 20 | role << 16 | row << 12 | tile << 4 | event} to prof[512..] for its rows 2..4 (350 per role).
#ifdef SVA_TIMELINE
#define SVA_STAMP(role, row, j, ev)                                                                       \
  do {                                                                                                    \
    if (blockIdx.x == 0 && (row) >= 2 && (row) <= 4 && stamp_n < 350u) {                                  \
      stamp_buf[(role) * 350 + stamp_n++] = ((unsigned long long)(unsigned)clock() << 20) |               \
          ((unsigned long long)(role) << 16) | ((unsigned long long)((row) & 15) << 12) |                 \
          ((unsigned long long)((j) & 255) << 4) | (unsigned long long)(ev);                              \
    }                                                                                                     \
  } while (0)
#else
#define SVA_STAMP(role, row, j, ev) do { } while (0)
#endif

namespace sva {

struct TsParams {
  const __nv_bfloat16* q;     // e4m3 variant: bytes (strides in elements either way)
  Strides sq;
  const float* q_scale;       // e4m3 variant: one scale per (b, h, block) for Q and for K; 4-bit variant: one per (b, h)
  const float* k_scale;
  const uint8_t* q_sf;        // 4-bit variant: e4m3 scale factors, 1024 bytes per (b, h, 128-token block), tile order
  const uint8_t* k_sf;
  const int32_t* row_ptr;     // null = dense
  const int32_t* col_idx;
  __nv_bfloat16* o;
  float* lse;
  int32_t* status;
  Strides so;
  int H, N, Nb, R;            // Nb: key blocks per head; R: rows handed out (128-query tiles)
  int d;                      // head dimension of the tensors: 128, or 64 (computed as 128 with the upper half zero)
  int Nt;                     // 128-query tiles per head (= Nb for 128-token blocks, ceil(Nb/2) for 64-token blocks)
  const int32_t* tile_cnt;    // 64-token blocks only: per tile row, number of 128-key tiles ...
  const int32_t* tile_beg;    // ... and where its descriptors start
  const uint32_t* tile_desc;  // two 16-bit halves {key block (14 bits), kept by query block A, kept by B}
  float scale_log2;           // softmax_scale * log2(e)
  int32_t* next_row;          // two device counters (both start at 0): the next row to hand out, CTAs done drawing
  // approximate remainder (REM kernels): every row's list is followed by np tiles whose "keys" are the
  // block means of K (and whose "values" the block means of V), 128 blocks per tile
  int n1;                     // first-order tiles after them: 0 (order 0), 1, or 2 with 64-token blocks (one per query block)
  const float* mu;            // first-order term: the reference mu_I of every query block's weights, [R of the CSR]
  int np;                     // pooled tiles per head = ceil(Nb / 128); 0 = no remainder
  int rem_mask;               // 1: the K producer leaves a bit mask of every row's kept blocks in shared memory (Nb <= 1024)
  float log2_block;           // log2(tokens per block): a block mean stands for that many keys
  float tail_bias;            // (log2(keys of the last block) - log2_block) / scale_log2: added to the last block's pooled logit
  long long* prof;            // tuning aid, normally null: entry 319 receives the longest CTA's cycle count
  int debug;                  // bit0: skip the exponentials (tuning aid, wrong results);
                              // bit4: starve the pipeline so that a wait runs out (test aid)
                              // (bit 7 acts in the launcher: the remainder looks kept blocks up in the CSR, without the mask)
};

namespace ts {
constexpr int D = 128;
constexpr int TILE = BS * D * 2;            // one bf16 tile: 32 KB
constexpr int KS = 2;                       // K tiles in flight
constexpr int VS = 3;                       // V^T tiles in flight
constexpr int THREADS = 384;
constexpr int QD = 4;                       // depth of the row queue
constexpr int OFF_K = 0;
constexpr int OFF_V = OFF_K + KS * TILE;
constexpr int OFF_O = OFF_V + VS * TILE;    // output staging: two [128 rows][128 B] panels (one per softmax group)
constexpr int OFF_CTRL = OFF_O + TILE;      // 6 tiles = 192 KB
constexpr int CTRL_BYTES = 256 + 2 * 128 * 4 + 4 * 128 * 4 + 256;   // barriers, reference exponents, row sums (two rows), row queue
constexpr int OFF_Q4 = OFF_CTRL + 4096;     // 4-bit variant: the row's Q codes (8 KB) and their scale factors (1 KB)
constexpr int OFF_QS = OFF_CTRL + 4096;     // bf16, 128-token blocks: staging of the second half (d 64..127) of a row's Q tile (16 KB)
#ifdef SVA_TIMELINE
constexpr int OFF_KMASK = OFF_QS + 16384;   // remainder: kept-block bit masks, [8 rows in flight][32 words]
constexpr int SMEM_BYTES = OFF_KMASK + 1024 + 1024 + 1400 * 8;
#else
constexpr int OFF_KMASK = OFF_QS + 16384;   // remainder: kept-block bit masks, [8 rows in flight][32 words]
constexpr int SMEM_BYTES = OFF_KMASK + 1024 + 1024;          // + alignment slack
#endif
constexpr uint32_t COL_SFA = 384, COL_SFB = 392;              // 4-bit variant: scale factors in the Q columns (8 + 2 x 8)
constexpr uint32_t COL_O = 256, COL_Q = 384, COL_P = 448;
// The reference exponent of a row is raised only when a block's maximum exceeds it by more than this
// many powers of two.  P then reaches at most 2^32 and a row sum 2^32 * N: far inside fp32 (and bf16
// has fp32's exponent range), while raises -- each one a pass over the row's O accumulator -- become rare.
constexpr float LAZY_LOG2 = 32.0f;
}  // namespace ts

// control block (bytes from OFF_CTRL):
//   0 q_ready | 8 o_free | 16 s_full[2] | 32 p_full[2] | 48 pv_done[2] | 64 ref_ready[2] | 80 xch
//   96 s_free[2] | 112 k_full[3] | 136 k_empty[3] | 160 v_full[3] | 184 v_empty[3]
//   216 tmem_base | 220 abort | 224 o_staged[2] | 240 q_staged | 256 ref[2][128] floats | 1280 lx[2 rows][2][128] floats
//   3328 row queue: QD entries {row, count, start, first entry, second entry, -, -, -} | 3456 rq_full[QD] | 3488 rq_empty[QD]

// Work list of row r (a 128-query tile): count and start; returns false for a corrupt row_ptr pair.
// 128-token blocks: the CSR row itself.  A pair that is not monotone, longer than Nb, negative or that
// reaches beyond nnz_bound (= row_ptr[R], the number of entries the CSR says it has) gives an empty row,
// so no col_idx entry outside [0, row_ptr[R]) is ever read.  64-token blocks: the tile row's list of
// 128-key tiles that pair_lists_kernel built (and checked) from the two CSR rows of the tile.
// Only the K producer calls this; the other roles take its answer from the row queue.
// (REM: the count includes the np pooled tiles that follow the row's own entries.)
template <bool B64, bool REM = false>
__device__ __forceinline__ bool row_list(const TsParams& prm, int r, int nnz_bound, int& n, int& beg) {
  if (B64) {
    if (prm.row_ptr == nullptr) { n = (prm.Nb + 1) >> 1; beg = 0; return true; }     // dense: every pair of key blocks
    n = __ldg(prm.tile_cnt + r) + (REM ? prm.np + prm.n1 : 0); beg = __ldg(prm.tile_beg + r);
    return true;
  }
  if (prm.row_ptr == nullptr) { n = prm.Nb; beg = 0; return true; }
  beg = __ldg(prm.row_ptr + r);
  const int end = __ldg(prm.row_ptr + r + 1);
  n = end - beg;
  if (beg < 0 || end < beg || n > prm.Nb || end > nnz_bound) { n = REM ? prm.np + prm.n1 : 0; beg = 0; return false; }
  if (REM) n += prm.np + prm.n1;
  return true;
}
// Pooled tiles (REM) are marked in their list entry: bit 31 (128-token blocks) resp. an upper half of
// 0xffff (64-token blocks: block index 0x3fff cannot occur, Nb <= 16383); the low 16 bits are the chunk.
// First-order tiles: bit 30 resp. an upper half of 0xfffe; the low bits say which query block of the tile row.
template <bool B64>
__device__ __forceinline__ bool entry_is_pooled(uint32_t e) {
  return B64 ? (e >> 16) == 0xffffu : (e >> 31) != 0u;
}
template <bool B64>
__device__ __forceinline__ bool entry_is_first_order(uint32_t e) {
  return B64 ? (e >> 16) == 0xfffeu : (e >> 30) == 1u;
}
// Entry j of a work list.  128-token blocks: the key block (an out-of-range entry is replaced by block 0;
// the producer reports it).  64-token blocks: the tile descriptor.
template <bool B64, bool REM = false>
__device__ __forceinline__ uint32_t list_block(const TsParams& prm, int beg, int j, int n_own = 0) {
  if (REM && j >= n_own + prm.np) return (B64 ? 0xfffe0000u : 0x40000000u) | (uint32_t)(j - n_own - prm.np);
  if (REM && j >= n_own) return (B64 ? 0xffff0000u : 0x80000000u) | (uint32_t)(j - n_own);
  if (B64) {
    if (prm.row_ptr == nullptr) {        // dense: key blocks 2j and 2j+1 (if it exists), kept by both query blocks
      const uint32_t u0 = 2u * (uint32_t)j, u1 = u0 + 1u;
      return (u0 | 0xc000u) | (u1 < (uint32_t)prm.Nb ? (u1 | 0xc000u) << 16 : 0u);
    }
    return __ldg(prm.tile_desc + beg + j);
  }
  if (prm.row_ptr == nullptr) return (uint32_t)j;
  const int J = __ldg(prm.col_idx + beg + j);
  return (J < 0 || J >= prm.Nb) ? 0u : (uint32_t)J;
}

// Persistent kernel.  Rows are handed out in their natural order from one device-wide counter (so the
// CTAs work on neighbouring rows at any time -- their K/V tiles share the L2 -- and rows of unequal
// length balance by themselves): the K producer, which runs furthest ahead, draws the next row,
// zero-fills it if its list is empty, and otherwise publishes {row, count, start, first two entries}
// in a small shared-memory queue that every other role reads in the same order.  All barriers keep running across rows, so the producers and the S
// issuer run ahead into the next row while the softmax groups finish the current one.
// F4: Q and K as packed e2m1 codes with e4m3 scales per 16 elements and one fp32 scale per (b,h).  S is then a
// block-scaled 4-bit MMA whose operands both come from shared memory (the Q tile is fetched by TMA once per row
// instead of being written to tensor memory; tm_kp is the map of the Q codes), with the scale factors copied
// into the tensor-memory columns the bf16 Q would have used.  128-token blocks, d = 128 only.
// VMN: V is read where it lies ([keys][d], d contiguous) and enters P V as an MN-major B operand -- another
// instruction descriptor than S, which costs a tensor-pipe drain per switch (hidden in the pipe's idle time: +1 % of
// the cycles), but no transposed copy of V and no workspace for it.  Every one-call entry point uses it; tm_vt is then
// the map of V (and, with REM, tm_vtp the block means of V as rows and tm_at the matrices A_I rather than their transposes).
template <bool B64, bool F8, bool REM, bool F4 = false, bool VMN = false>
__global__ void __launch_bounds__(384, 1)
attn_ts_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_vt,
               const __grid_constant__ CUtensorMap tm_o, const __grid_constant__ CUtensorMap tm_kp,
               const __grid_constant__ CUtensorMap tm_vtp, const __grid_constant__ CUtensorMap tm_at,
               const __grid_constant__ CUtensorMap tm_q, const TsParams prm) {
  using namespace ts;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  uint8_t* ctrl = smem + OFF_CTRL;
  const uint32_t cb = sbase + OFF_CTRL;
  const uint32_t bar_q_ready = cb + 0, bar_o_free = cb + 8, bar_s_full = cb + 16, bar_p_full = cb + 32,
                 bar_pv_done = cb + 48, bar_ref = cb + 64, bar_xch = cb + 80, bar_s_free = cb + 96,
                 bar_k_full = cb + 112, bar_k_empty = cb + 136, bar_v_full = cb + 160, bar_v_empty = cb + 184,
                 bar_ost = cb + 224, bar_qs = cb + 240, bar_rq_full = cb + 3456, bar_rq_empty = cb + 3488;
  volatile uint32_t* tmem_base_p = reinterpret_cast<volatile uint32_t*>(ctrl + 216);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 220);
  volatile float* ref = reinterpret_cast<volatile float*>(ctrl + 256);      // [2][128]
  volatile float* lx = reinterpret_cast<volatile float*>(ctrl + 1280);      // [2][2][128]
  volatile int* rowq = reinterpret_cast<volatile int*>(ctrl + 3328);        // [QD][8]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int Nb = prm.Nt;             // row index arithmetic: rows per head
  constexpr int KB = B64 ? 64 : BS;  // tokens per key block
  constexpr bool RMASK = REM && !B64; // remainder, 128-token blocks: kept-block bit masks (64-token blocks: the CSR look-up measured faster)

  // ---------------------------------------------------------------- set-up
  const long long t_cta0 = prm.prof ? clock64() : 0;
#ifdef SVA_TIMELINE
  uint32_t stamp_n = 0;
  unsigned long long* stamp_buf = reinterpret_cast<unsigned long long*>(smem + OFF_KMASK + 1024);   // 1400 entries
  if (blockIdx.x == 0) for (int i_ = threadIdx.x; i_ < 1400; i_ += THREADS) stamp_buf[i_] = 0ull;
  __syncthreads();
#endif
  if (threadIdx.x == 0) {
    mbar_init(bar_q_ready, (!F4 && !B64) ? 128 : 256);   // (128-token blocks, bf16 / e4m3 Q: one softmax group writes a row's Q)
    mbar_init(bar_o_free, 256);
    mbar_init(bar_xch, 256);
    mbar_init(bar_qs, 1);
    for (int w = 0; w < 2; ++w) {
      mbar_init(bar_s_full + 8 * w, 1);
      mbar_init(bar_p_full + 8 * w, 128);
      mbar_init(bar_pv_done + 8 * w, 1);
      mbar_init(bar_ref + 8 * w, 128);
      mbar_init(bar_s_free + 8 * w, 128);
      mbar_init(bar_ost + 8 * w, 128);
    }
    for (int s = 0; s < 3; ++s) {
      mbar_init(bar_k_full + 8 * s, 1);
      mbar_init(bar_k_empty + 8 * s, 1);
      mbar_init(bar_v_full + 8 * s, 1);
      mbar_init(bar_v_empty + 8 * s, 1);
    }
    for (int i = 0; i < QD; ++i) {
      mbar_init(bar_rq_full + 8 * i, 1);
      mbar_init(bar_rq_empty + 8 * i, 11);       // 3 producer / issuer lanes + one lane of each softmax warp
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 8 && lane == 0) { prefetch_tmap(&tm_k); if (REM) prefetch_tmap(&tm_kp); }
  if (warp == 11 && lane == 0) { prefetch_tmap(&tm_vt); if (REM) { prefetch_tmap(&tm_vtp); prefetch_tmap(&tm_at); } }
  if (warp == 0 && lane == 0) { prefetch_tmap(&tm_o); if (!F4 && !B64) prefetch_tmap(&tm_q); }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(cb + 216), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_p;
  constexpr uint32_t IDESC = instr_desc(128, 128, 1, false);   // bf16 x bf16 -> fp32, A and B K-major
  constexpr uint32_t IDESC_QK = F8 ? instr_desc(128, 128, 0, false) : IDESC;   // e4m3 x e4m3 for S in the e4m3 variant
  constexpr int KTILE = F8 ? TILE / 2 : TILE;                  // bytes of one K tile
  constexpr int PANEL16 = (BS * 128) >> 4;                      // one 128-row x 128-byte panel

  // Entry i of the row sequence (the same for every role): false when a wait ran out.  r >= R ends the
  // sequence.  `arrive` tells whether this thread signs the entry off (one thread per consumer).
  auto fetch_row = [&](uint32_t i, int& r, int& n, int& beg, uint32_t& e0, uint32_t& e1, bool arrive) -> bool {
    const uint32_t slot = i % QD;
    if (!mbar_wait(bar_rq_full + 8 * slot, (i / QD) & 1u, abort_flag, prm.status)) return false;
    r = rowq[8 * slot];
    n = rowq[8 * slot + 1];
    beg = rowq[8 * slot + 2];
    e0 = (uint32_t)rowq[8 * slot + 3];
    e1 = (uint32_t)rowq[8 * slot + 4];
    if (warp < 8) __syncwarp();                  // softmax warps: every lane has read the entry before lane 0 signs
    if (arrive) mbar_arrive(bar_rq_empty + 8 * slot);
    return true;
  };

  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 96;");
    if (warp == 8) {
      // ---------------------------------------------------------- K producer (one lane)
      if (lane == 0) {
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        const int nnz_bound = (!B64 && prm.row_ptr) ? __ldg(prm.row_ptr + prm.R) : 0;
        for (uint32_t i = 0; ok; ++i) {
          // ---- row scheduling: draw the next row with a non-empty list and publish it
          const uint32_t slot = i % QD;
          if (i >= QD && !mbar_wait(bar_rq_empty + 8 * slot, (i / QD - 1u) & 1u, abort_flag, prm.status)) break;
          int r, n = 0, beg = 0;
          for (;;) {
            r = atomicAdd(prm.next_row, 1);
            if (r >= prm.R) break;
            if (!row_list<B64, REM>(prm, r, nnz_bound, n, beg) && prm.status) atomicOr(prm.status, SVA_DEV_BAD_INDEX);
            if (n > 0) break;
            // nothing kept (or a corrupt row_ptr pair): zeros and lse = -inf; rare, so this one lane does it
            const int I = r % Nb, bh0 = r / Nb;
            for (int t = 0; t < BS; ++t) {
              const int qi = I * BS + t;
              if (qi >= prm.N) break;
              __nv_bfloat16* orow = prm.o + (long long)(bh0 / prm.H) * prm.so.b + (long long)(bh0 % prm.H) * prm.so.h +
                                    (long long)qi * prm.so.n;
              for (int cc = 0; cc < prm.d; cc += 8) *reinterpret_cast<uint4*>(orow + cc) = make_uint4(0, 0, 0, 0);
              if (prm.lse) prm.lse[(long long)bh0 * prm.N + qi] = -INFINITY;
            }
          }
          uint32_t e0 = 0u, e1 = 0u;
          const int n_own = n - ((REM && prm.row_ptr) ? prm.np + prm.n1 : 0);        // entries of the row's own list
          if (r < prm.R) { e0 = list_block<B64, REM>(prm, beg, 0, n_own); if (n > 1) e1 = list_block<B64, REM>(prm, beg, 1, n_own); }
          if (!F4 && !B64 && r < prm.R) {
            // the row's Q tile will be fetched about a row from now: start it on its way into the L2
            const int I = r % Nb, bh0 = r / Nb, rows = min(BS, prm.N - I * BS);
            const uint32_t eb = F8 ? 1u : 2u, row_bytes = (uint32_t)prm.d * eb;
            const uint8_t* qrow = reinterpret_cast<const uint8_t*>(prm.q) +
                                  ((long long)(bh0 / prm.H) * prm.sq.b + (long long)(bh0 % prm.H) * prm.sq.h +
                                   (long long)I * BS * prm.sq.n) * eb;
            if (prm.sq.n * (long long)eb == (long long)row_bytes) {
              bulk_prefetch_l2(qrow, (uint32_t)rows * row_bytes);
            } else {
              for (int t = 0; t < rows; ++t) bulk_prefetch_l2(qrow + (long long)t * prm.sq.n * eb, row_bytes);
            }
          }
          rowq[8 * slot] = r;
          rowq[8 * slot + 1] = n;
          rowq[8 * slot + 2] = beg;
          rowq[8 * slot + 3] = (int)e0;
          rowq[8 * slot + 4] = (int)e1;
          mbar_arrive(bar_rq_full + 8 * slot);
          if (r >= prm.R) {
            // Every CTA ends by drawing one value >= R.  The last one to do so puts both counters back to 0,
            // so a prepared workspace serves further attention calls on the same V.
            if (atomicAdd(prm.next_row + 1, 1) == (int)gridDim.x - 1) {
              prm.next_row[1] = 0;
              prm.next_row[0] = 0;
            }
            break;
          }
          // ---- K tiles of the row
          const int bh = r / Nb, hh = bh % prm.H, bb = bh / prm.H;
          // Remainder (128-token blocks): while walking the row's list this lane leaves a bit mask of the kept blocks
          // for the softmax warps, which mask those columns of the block-mean tiles.  Eight masks in
          // rotation: this lane is at most four tiles (two K slots, two S buffers) -- so at most four rows -- ahead.
          // The masks are complete before the first block-mean tile's load is issued, which orders them before the
          // softmax warps' read (expect_tx arrive -> k_full -> S MMA -> s_full).
          volatile uint32_t* kmask = reinterpret_cast<volatile uint32_t*>(smem + OFF_KMASK) + (i & 7u) * 32;
          if (RMASK && prm.rem_mask) {
            for (int t = 0; t < 32; ++t) kmask[t] = 0u;
          }
          for (int j = 0; j < n; ++j) {
            if ((prm.debug & 16) && j >= 1) { ok = false; break; }   // test aid: starve the pipeline so that a wait runs out
            if (!mbar_wait(bar_k_empty + 8 * s, ph ^ 1u, abort_flag, prm.status)) { ok = false; break; }
            const uint32_t dst = sbase + OFF_K + s * TILE;
            mbar_expect_tx(bar_k_full + 8 * s, F4 ? 8192 + 1024 : KTILE);
            if (F4) {
              // packed codes of the key block (128 rows x 64 bytes, 64-byte swizzle) and its 1 KB of scale factors
              int J = j;
              if (prm.row_ptr) {
                J = __ldg(prm.col_idx + beg + j);
                if (J < 0 || J >= prm.Nb) { J = 0; if (prm.status) atomicOr(prm.status, SVA_DEV_BAD_INDEX); }
              }
              tma_load_4d(dst, &tm_k, bar_k_full + 8 * s, 0, J * BS, hh, bb);
              bulk_load(dst + 8192, prm.k_sf + ((long long)bh * prm.Nb + J) * 1024, 1024, bar_k_full + 8 * s);
            } else if (REM && j >= n_own) {
              // pooled tile: 128 block means of K (rows beyond Nb are zero in the pooled tensor)
              // (a first-order tile has no logits of its own: its S is computed from pooled tile 0 and ignored)
              const int c = j - n_own < prm.np ? j - n_own : 0;
              tma_load_4d(dst, &tm_kp, bar_k_full + 8 * s, 0, c * BS, hh, bb);
              tma_load_4d(dst + TILE / 2, &tm_kp, bar_k_full + 8 * s, 64, c * BS, hh, bb);
            } else if (B64) {
              // two 64-key blocks side by side: rows 0..63 and 64..127 of both d-panels
              // (e4m3: one 128-byte panel, so one load per key block)
              const uint32_t dsc = list_block<B64>(prm, beg, j);      // (an own entry: j < n_own)
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                const int J = (int)((dsc >> (16 * h)) & 0x3fffu);

                tma_load_4d(dst + h * (TILE / 4), &tm_k, bar_k_full + 8 * s, 0, J * KB, hh, bb);
                if (!F8) tma_load_4d(dst + TILE / 2 + h * (TILE / 4), &tm_k, bar_k_full + 8 * s, 64, J * KB, hh, bb);
              }
            } else {
              int J = j;
              if (prm.row_ptr) {
                J = __ldg(prm.col_idx + beg + j);
                if (J < 0 || J >= prm.Nb) { J = 0; if (prm.status) atomicOr(prm.status, SVA_DEV_BAD_INDEX); }
                if (RMASK && prm.rem_mask) kmask[J >> 5] |= 1u << (J & 31);
              }
              tma_load_4d(dst, &tm_k, bar_k_full + 8 * s, 0, J * BS, hh, bb);      // e4m3: the whole tile (128 x 128 bytes)
              if (!F8) tma_load_4d(dst + TILE / 2, &tm_k, bar_k_full + 8 * s, 64, J * BS, hh, bb);
            }
            if (++s == KS) { s = 0; ph ^= 1u; }
          }
        }
      }
    } else if (warp == 11) {
      // ---------------------------------------------------------- V^T producer (one lane)
      // tile J of head (b,h): 128 d-rows x 128 keys, contiguous 32 KB, two 64-key panels
      if (lane == 0) {
        int s = 0;
        uint32_t ph = 0;
        bool ok = true;
        for (uint32_t i = 0; ok; ++i) {
          int r, n, beg;
          uint32_t e0, e1;
          if (!fetch_row(i, r, n, beg, e0, e1, true) || r >= prm.R) break;
          const int bh = r / Nb, hh = bh % prm.H, bb = bh / prm.H;
          const int n_own = n - ((REM && prm.row_ptr) ? prm.np + prm.n1 : 0);
          for (int j = 0; j < n; ++j) {
            if (!mbar_wait(bar_v_empty + 8 * s, ph ^ 1u, abort_flag, prm.status)) { ok = false; break; }
            const uint32_t e = list_block<B64, REM>(prm, beg, j, n_own);
            const uint32_t dst = sbase + OFF_V + s * TILE;
            mbar_expect_tx(bar_v_full + 8 * s, TILE);
            if (REM && j >= n_own) {
              // pooled tile: the block means of V ([128 d rows][128 blocks], or [128 blocks][128 d] when V itself is
              // read keys-major; blocks beyond Nb zero)
              const int c = j - n_own;
              if (c < prm.np) {
                tma_load_4d(dst, &tm_vtp, bar_v_full + 8 * s, 0, c * BS, hh, bb);
                tma_load_4d(dst + TILE / 2, &tm_vtp, bar_v_full + 8 * s, 64, c * BS, hh, bb);
              } else {
                // first-order tile: A^T (A when V is read keys-major) of the query block (64-token blocks: of the tile
                // row's first / second one)
                const int qb = B64 ? min(2 * (r % Nb) + (c - prm.np), prm.Nb - 1) : r % Nb;
                tma_load_4d(dst, &tm_at, bar_v_full + 8 * s, 0, qb * BS, hh, bb);
                tma_load_4d(dst + TILE / 2, &tm_at, bar_v_full + 8 * s, 64, qb * BS, hh, bb);
              }
            } else if (VMN) {
              // V itself: two d-panels of [128 keys][64 d] (64-token blocks: each panel's two halves from two key blocks)
              if (B64) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                  const int Jh = (int)((e >> (16 * h)) & 0x3fffu);
                  tma_load_4d(dst + h * (TILE / 4), &tm_vt, bar_v_full + 8 * s, 0, Jh * KB, hh, bb);
                  tma_load_4d(dst + TILE / 2 + h * (TILE / 4), &tm_vt, bar_v_full + 8 * s, 64, Jh * KB, hh, bb);
                }
              } else {
                tma_load_4d(dst, &tm_vt, bar_v_full + 8 * s, 0, (int)e * BS, hh, bb);
                tma_load_4d(dst + TILE / 2, &tm_vt, bar_v_full + 8 * s, 64, (int)e * BS, hh, bb);
              }
            } else if (B64) {
              // each 64-key panel of the tile is one key block's transposed V: [128 d rows][64 keys]
              tma_load_4d(dst, &tm_vt, bar_v_full + 8 * s, 0, (int)(e & 0x3fffu) * D, hh, bb);
              tma_load_4d(dst + TILE / 2, &tm_vt, bar_v_full + 8 * s, 0, (int)((e >> 16) & 0x3fffu) * D, hh, bb);
            } else {
              tma_load_4d(dst, &tm_vt, bar_v_full + 8 * s, 0, (int)e * BS, hh, bb);
              tma_load_4d(dst + TILE / 2, &tm_vt, bar_v_full + 8 * s, 64, (int)e * BS, hh, bb);
            }
            if (++s == VS) { s = 0; ph ^= 1u; }
          }
        }
      }
    } else if (warp == 9) {
      // ---------------------------------------------------------- S issuer (one lane)
      // per row: S(0), S(1), then S(j) into the buffer of S(j-2) as soon as that block's softmax
      // has read it; the first S of a row also needs the row's Q in TMEM
      if (lane == 0) {
        const uint64_t kd0 = smem_desc(sbase + OFF_K, 16, 1024);
        int s = 0;
        uint32_t ph = 0;
        uint32_t cs[2] = {0, 0};            // S tiles issued so far into buffer w
        bool ok = true;
        for (uint32_t i = 0; ok; ++i) {
          int r, n, beg;
          uint32_t e0, e1;
          if (!fetch_row(i, r, n, beg, e0, e1, true) || r >= prm.R) break;
          ok = mbar_wait(bar_q_ready, i & 1u, abort_flag, prm.status);
          for (int j = 0; j < n && ok; ++j) {
            const int w = j & 1;
            if (cs[w] > 0) {
              ok = mbar_wait(bar_s_free + 8 * w, (cs[w] - 1u) & 1u, abort_flag, prm.status);
              if (!ok) break;
            }
            SVA_STAMP(2, i, j, 0);
            ok = mbar_wait(bar_k_full + 8 * s, ph, abort_flag, prm.status);
            if (!ok) break;
            SVA_STAMP(2, i, j, 1);
            tc_fence_after();
            const uint64_t kd = kd0 + (uint64_t)(s * (TILE >> 4));
            if (F4) {
              const uint32_t kslot = sbase + OFF_K + s * TILE;
              if (j == 0) {                                    // the row's Q scale factors (q_ready: they are in shared memory)
                tc_cp_sf(tmem_base + COL_SFA, smem_desc_plain(sbase + OFF_Q4 + 8192), 1u);
                tc_cp_sf(tmem_base + COL_SFA + 4, smem_desc_plain(sbase + OFF_Q4 + 8192 + 512), 1u);
              }
              tc_cp_sf(tmem_base + COL_SFB + 8 * s, smem_desc_plain(kslot + 8192), 1u);
              tc_cp_sf(tmem_base + COL_SFB + 8 * s + 4, smem_desc_plain(kslot + 8192 + 512), 1u);
              const uint64_t qd4 = smem_desc_sw64(sbase + OFF_Q4), kd4 = smem_desc_sw64(kslot);
#pragma unroll
              for (int kk = 0; kk < 2; ++kk)                    // 64 elements (32 bytes) of d per instruction
                tc_mma_bs4_ss(tmem_base + 128 * w, qd4 + (uint64_t)(kk * 2), kd4 + (uint64_t)(kk * 2), instr_desc_bs4(128, 128),
                              tmem_base + COL_SFA + 4 * kk, tmem_base + COL_SFB + 8 * s + 4 * kk, kk > 0 ? 1u : 0u, 1u);
            } else if (F8) {
#pragma unroll
              for (int kk = 0; kk < D / 32; ++kk)               // 32 e4m3 values (32 bytes, 8 TMEM columns) per step
                tc_mma_ts<true>(tmem_base + 128 * w, tmem_base + COL_Q + 8 * kk, kd + (uint64_t)(kk * 2), IDESC_QK,
                                kk > 0 ? 1u : 0u, 1u);
            } else {
#pragma unroll
              for (int kk = 0; kk < D / 16; ++kk) {
                const uint64_t off = (uint64_t)((kk / 4) * PANEL16 + (kk % 4) * 2);
                tc_mma_ts(tmem_base + 128 * w, tmem_base + COL_Q + 8 * kk, kd + off, IDESC, kk > 0 ? 1u : 0u, 1u);
              }
            }
            tc_commit(bar_k_empty + 8 * s, 1u);
            SVA_STAMP(2, i, j, 2);
            tc_commit(bar_s_full + 8 * w, 1u);
            ++cs[w];
            if (++s == KS) { s = 0; ph ^= 1u; }
          }
        }
      }
    } else {
      // ---------------------------------------------------------- P V issuer (one lane)
      if (lane == 0) {
        // (VMN: 64 d-values contiguous, the next 64 one panel = 16 KB on, 8 keys 1 KB apart)
        const uint64_t vd0 = VMN ? smem_desc(sbase + OFF_V, TILE / 2, 1024) : smem_desc(sbase + OFF_V, 16, 1024);
        constexpr uint32_t IDESC_PV = VMN ? instr_desc(128, 128, 1, true) : IDESC;
        int s = 0;
        uint32_t ph = 0;
        uint32_t cp[2] = {0, 0};            // P V groups issued so far for parity w
        bool ok = true;
        for (uint32_t i = 0; ok; ++i) {
          int r, n, beg;
          uint32_t e0, e1;
          if (!fetch_row(i, r, n, beg, e0, e1, true) || r >= prm.R) break;
          // the first P V of a row overwrites O: the previous row's O must have been read
          if (i > 0) ok = mbar_wait(bar_o_free, (i - 1u) & 1u, abort_flag, prm.status);
          for (int j = 0; j < n && ok; ++j) {
            const int w = j & 1;
            const uint64_t vd = vd0 + (uint64_t)(s * (TILE >> 4));
            ok = mbar_wait(bar_p_full + 8 * w, cp[w] & 1u, abort_flag, prm.status);
            SVA_STAMP(3, i, j, 0);
            ok = ok && mbar_wait(bar_v_full + 8 * s, ph, abort_flag, prm.status);
            if (!ok) break;
            SVA_STAMP(3, i, j, 1);
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < BS / 16; ++kk) {
              const uint64_t off = VMN ? (uint64_t)(kk * 128)            // 16 keys = 16 rows of 128 bytes
                                       : (uint64_t)((kk / 4) * PANEL16 + (kk % 4) * 2);
              tc_mma_ts(tmem_base + COL_O, tmem_base + COL_P + 8 * kk, vd + off, IDESC_PV, (j > 0 || kk > 0) ? 1u : 0u, 1u);
            }
            SVA_STAMP(3, i, j, 2);
            tc_commit(bar_v_empty + 8 * s, 1u);
            tc_commit(bar_pv_done + 8 * w, 1u);
            if (!ok) break;
            ++cp[w];
            if (++s == VS) { s = 0; ph ^= 1u; }
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue
    asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
    const int w = warp >> 2;                                 // this group takes blocks j = w, w+2, ... of a row
    const int row = (warp & 3) * 32 + lane;                  // query row of the tile == TMEM lane
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t s_tmem = tmem_base + lane_addr + 128 * w;
    const uint32_t o_tmem = tmem_base + lane_addr + COL_O;
    const uint32_t p_tmem = tmem_base + lane_addr + COL_P;
    const uint32_t q_tmem = tmem_base + lane_addr + COL_Q + (F8 ? 16 : 32) * w;
    const int tail_keys = prm.N - (prm.Nb - 1) * KB;         // valid keys of the last key block
    const int nnz_total = (REM && prm.row_ptr) ? __ldg(prm.row_ptr + (prm.R / prm.Nt) * prm.Nb) : 0;   // row_ptr[R of the CSR]
    const int qh = row >> 6;                                 // 64-token blocks: which query block of the tile I am in
    float c = prm.scale_log2;      // e4m3 variant: times the scales of the query block and of the key block, per block
    float c1 = prm.scale_log2;     // e4m3 with 64-token blocks: the same for the tile's second key block
    uint32_t cnt[2] = {0, 0};      // blocks of parity 0 / 1 completed in earlier rows (barrier phase bases)
    uint32_t rows_done = 0;        // non-empty rows finished
    bool ok = true;

    // this group's half (d columns 64w..64w+63) of a row's Q: global -> registers -> TMEM
    auto load_q = [&](int r, uint32_t* qv) {
#pragma unroll
      for (int e = 0; e < 32; ++e) qv[e] = 0u;
      if (F4 || r >= prm.R) return;                                     // (4-bit variant: the Q tile goes to shared memory by TMA)
      const int bh = r / Nb, qi = (r % Nb) * BS + row;
      if (qi >= prm.N || 64 * w >= prm.d) return;                      // (d = 64: the second group's half of Q is zero)
      const long long eoff = (long long)(bh / prm.H) * prm.sq.b + (long long)(bh % prm.H) * prm.sq.h +
                             (long long)qi * prm.sq.n + 64 * w;           // in elements
      const uint4* src = F8 ? reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(prm.q) + eoff)
                            : reinterpret_cast<const uint4*>(prm.q + eoff);
#pragma unroll
      for (int e = 0; e < (F8 ? 4 : 8); ++e) {                            // 64 elements: 64 or 128 bytes
        const uint4 u = __ldg(src + e);
        qv[4 * e] = u.x; qv[4 * e + 1] = u.y; qv[4 * e + 2] = u.z; qv[4 * e + 3] = u.w;
      }
    };
    auto store_q = [&](const uint32_t* qv, int r) {
      if (F4) {
        // one thread fetches the row's Q codes and scale factors; the barrier completes when every softmax thread
        // has arrived (none of them reads the previous row's Q any more) and the bytes have landed
        if (threadIdx.x == 0) {
          const int bh = r / Nb, I = r % Nb;
          mbar_expect_tx_only(bar_q_ready, 8192 + 1024);
          tma_load_4d(sbase + OFF_Q4, &tm_kp, bar_q_ready, 0, I * BS, bh % prm.H, bh / prm.H);
          bulk_load(sbase + OFF_Q4 + 8192, prm.q_sf + ((long long)bh * prm.Nb + I) * 1024, 1024, bar_q_ready);
        }
        mbar_arrive(bar_q_ready);
        return;
      }
      if (F8) tmem_st16(q_tmem, qv); else tmem_st32(q_tmem, qv);
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar_q_ready);
    };

    // 128-token blocks (bf16 / e4m3 Q): ONE group writes the whole Q of the next row -- the group that does not take
    // the current row's last tile, as soon as that last S has been computed, about a tile before the row ends -- so
    // that the S issuer starts on the next row while this one is still finishing.  The Q tile comes by TMA (a
    // thread-per-row read of Q from global memory costs 32 cache lines per load instruction, and that
    // load/store-unit time stood in the way of the other group's last P store): the first 64 columns of d into
    // the group's own output staging panel (idle between two epilogues), the other 64 into a 16 KB buffer behind
    // the control block, both loads in flight together; each thread then copies its row from shared memory into
    // tensor memory.  `use` counts these copies over the CTA's rows (the first row's is copy 0): the barrier's phase.
    constexpr bool EARLYQ = !F4 && !B64;
    auto copy_q = [&](int r, uint32_t use) -> bool {
      const int bh = r / Nb, I = r % Nb;
      if ((threadIdx.x & 127) == 0) {
        bulk_wait_read0();                                                // my previous output store has read the panel
        mbar_expect_tx(bar_qs, F8 ? TILE / 2 : TILE);
        tma_load_4d(sbase + OFF_O + w * (TILE / 2), &tm_q, bar_qs, 0, I * BS, bh % prm.H, bh / prm.H);
        if (!F8) tma_load_4d(sbase + OFF_QS, &tm_q, bar_qs, 64, I * BS, bh % prm.H, bh / prm.H);
      }
      if (!mbar_wait(bar_qs, use & 1u, abort_flag, prm.status)) return false;
#pragma unroll
      for (int ps = 0; ps < (F8 ? 1 : 2); ++ps) {
        // 128-byte rows, 16-byte chunks swizzled by row % 8
        const uint8_t* prow = smem + (ps == 0 ? OFF_O + w * (TILE / 2) : OFF_QS) + row * 128;
        uint32_t qv[32];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const uint4 u = *reinterpret_cast<const uint4*>(prow + ((e ^ (row & 7)) << 4));
          qv[4 * e] = u.x; qv[4 * e + 1] = u.y; qv[4 * e + 2] = u.z; qv[4 * e + 3] = u.w;
        }
        tmem_st32(tmem_base + lane_addr + COL_Q + 32 * ps, qv);
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar_q_ready);
      return true;
    };

    // The row sequence comes from the queue the K producer fills.  The entry after the current one is
    // read in the epilogue (the producer has published it by then: it runs about two blocks ahead),
    // so the next row's Q and first list entries are at hand when the row changes.
    const bool signs = lane == 0;                             // one lane per warp signs queue entries off
    int r_c = prm.R, n_c = 0, beg_c = 0;
    uint32_t e0_c = 0u, e1_c = 0u;
    if (!fetch_row(0, r_c, n_c, beg_c, e0_c, e1_c, signs)) ok = false;
    if (EARLYQ) {
      if (ok && r_c < prm.R && w == 1) ok = copy_q(r_c, 0u);
    } else if (ok && r_c < prm.R) {
      // first row: its Q goes in right away
      uint32_t qv[32];
      load_q(r_c, qv);
      store_q(qv, r_c);
    }
    for (; ok && r_c < prm.R; ++rows_done) {
      const int r = r_c, n = n_c, lbeg = beg_c;
      uint32_t J = (w == 0) ? e0_c : e1_c;                           // my first list entry of the row
      const int I = r % Nb, bh = r / Nb;
      const int hh = bh % prm.H, bb = bh / prm.H;
      const int qi = I * BS + row;
      const int wl = (n - 1) & 1;                                     // group that takes the row's last block
      const uint32_t last = cnt[wl] + (uint32_t)((n - 1) >> 1);       // phase index of that block
      float m_mine = -INFINITY;      // reference exponent my partial row sum is relative to
      float l = 0.f;                 // partial row sum over this group's blocks
      float qs_row = 1.f, ks_next = 1.f, ks_next1 = 1.f;
      auto load_ks = [&](uint32_t e) {                                // scales of the key block(s) of list entry e
        const float* ks = prm.k_scale + (long long)bh * prm.Nb;
        if (B64) {
          ks_next = __ldg(ks + (int)(e & 0x3fffu));
          ks_next1 = __ldg(ks + (int)((e >> 16) & 0x3fffu));
        } else {
          ks_next = __ldg(ks + (int)e);
        }
      };
      if (F4) c = prm.scale_log2 * __ldg(prm.q_scale + bh) * __ldg(prm.k_scale + bh);     // the two tensor scales
      if (F8) {
        const int qb = B64 ? min(2 * I + qh, prm.Nb - 1) : I;         // my query block
        qs_row = __ldg(prm.q_scale + (long long)bh * prm.Nb + qb) * prm.scale_log2;
        if (w < n) load_ks(J);
      }
      const int n_own = n - ((REM && prm.row_ptr) ? prm.np + prm.n1 : 0);      // entries of the row's own list
      // One tile of the row (KIND 0: a kept key block, 1: a tile of block means, 2: the first-order tile).  The
      // kinds are separate instantiations, so the hot one carries none of the remainder's code; false: a wait ran out.
      auto tile = [&](auto kind_tag, const int j) -> bool {
        constexpr int KIND = decltype(kind_tag)::value;
        const uint32_t mine = cnt[w] + (uint32_t)(j >> 1);            // my barriers' phase index for block j
        const uint32_t prev = cnt[w ^ 1] + (uint32_t)((j - 1) >> 1);  // other group's phase index for block j-1
        // valid keys of the tile's two 64-key halves (64-token blocks: a half whose key block this
        // thread's query block does not keep counts as 0; uniform over a warp)
        int v0, v1;
        constexpr bool pooled = REM && KIND == 1;                     // a tile of block means (the remainder)
        const int pc = (int)(J & 0xffffu);                            // ... and which 128 blocks it holds
        constexpr bool fo = REM && KIND == 2;                         // the first-order tile: P = scaled q, "V^T" = A^T
        if (fo) {
          v0 = B64 ? 64 : BS; v1 = B64 ? 64 : 0;
        } else if (pooled) {
          const int vn = min(BS, prm.Nb - BS * pc);                   // blocks that exist in this tile
          v0 = B64 ? min(64, vn) : vn;
          v1 = B64 ? max(vn - 64, 0) : 0;
        } else if (B64) {
          const int u0 = (int)(J & 0x3fffu), u1 = (int)((J >> 16) & 0x3fffu);
          v0 = ((J >> (14 + qh)) & 1u) ? (u0 == prm.Nb - 1 ? tail_keys : 64) : 0;
          v1 = ((J >> (30 + qh)) & 1u) ? (u1 == prm.Nb - 1 ? tail_keys : 64) : 0;
        } else {
          v0 = ((int)J == prm.Nb - 1) ? tail_keys : BS;      // 128-token blocks: all valid keys counted in v0
          v1 = 0;
        }
        if (F8) { c = qs_row * ks_next; if (B64) c1 = qs_row * ks_next1; }
        if (j + 2 < n) {                                               // one entry ahead
          J = list_block<B64, REM>(prm, lbeg, j + 2, n_own);
          if (F8) load_ks(J);
        }
        if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, j, 0);
        if (!mbar_wait(bar_s_full + 8 * w, mine & 1u, abort_flag, prm.status)) return false;
        if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, j, 1);
        tc_fence_after();
        if (B64 ? (v0 + v1 < BS) : (v0 < BS)) {
          // Keys that do not exist (ragged last key block) become -inf in TMEM before S is read: a short
          // rolled loop, which keeps 128 compare/select pairs out of the hot instruction stream.  A half
          // that is not kept at all (64-token blocks) is left alone here: it is excluded below.
          if (B64) {
            if (v0 > 0) {
#pragma unroll 1
              for (int e = v0; e < 64; ++e) tmem_st1(s_tmem + e, 0xff800000u);
            }
            if (v1 > 0) {
#pragma unroll 1
              for (int e = 64 + v1; e < BS; ++e) tmem_st1(s_tmem + e, 0xff800000u);
            }
          } else {
#pragma unroll 1
            for (int e = v0; e < BS; ++e) tmem_st1(s_tmem + e, 0xff800000u);
          }
          tc_wait_st();
        }
        if (REM && pooled) {
          // The remainder stands for the DROPPED blocks only: the blocks this thread's query block keeps become
          // -inf (one warp-wide TMEM store each; the row's CSR entries are the same for a whole warp), and the
          // ragged last block's mean stands for fewer keys than the others.
          if (RMASK && prm.rem_mask) {
            // (the K producer left the kept blocks of this row as a bit mask: four words for this tile's 128 blocks)
            const volatile uint32_t* mk = reinterpret_cast<const volatile uint32_t*>(smem + OFF_KMASK) +
                                          (rows_done & 7u) * 32 + 4 * pc;
#pragma unroll 1
            for (int kw = 0; kw < 4; ++kw) {
              uint32_t mword = mk[kw];
              while (mword) {
                const int bit = __ffs(mword) - 1;
                mword &= mword - 1u;
                tmem_st1(s_tmem + 32 * kw + bit, 0xff800000u);
              }
            }
          }
          const int rq = B64 ? bh * prm.Nb + min(2 * I + qh, prm.Nb - 1) : r;      // my query block's CSR row
          int cb = 0, ce = 0;                                          // (more than 1024 key blocks: from the CSR itself)
          if (!(RMASK && prm.rem_mask)) { cb = __ldg(prm.row_ptr + rq); ce = __ldg(prm.row_ptr + rq + 1); }
          if (cb < 0 || ce < cb || ce - cb > prm.Nb || ce > nnz_total) ce = cb;      // corrupt pair (reported elsewhere)
#pragma unroll 1
          for (int t0 = cb; t0 < ce; t0 += 32) {                       // 32 entries at a time, one per lane
            const int Jl = t0 + lane < ce ? __ldg(prm.col_idx + t0 + lane) : -1;
            uint32_t hit = __ballot_sync(0xffffffffu, Jl >= 0 && Jl < prm.Nb && (Jl >> 7) == pc);
            while (hit) {
              const int Jk = __shfl_sync(0xffffffffu, Jl, __ffs(hit) - 1);
              hit &= hit - 1;
              tmem_st1(s_tmem + (Jk & 127), 0xff800000u);
            }
          }
          if (tail_keys < KB && ((prm.Nb - 1) >> 7) == pc) {
            tc_wait_st();
            const uint32_t col = s_tmem + ((prm.Nb - 1) & 127);
            const float x = __uint_as_float(tmem_ld1(col));
            tc_wait_ld();
            tmem_st1(col, __float_as_uint(x + prm.tail_bias));          // (-inf stays -inf)
          }
          tc_wait_st();
        }
        uint32_t sv[128];
        if (!(REM && fo)) {                                           // (a first-order tile's S is a dummy: not read)
          tmem_ld32(s_tmem + 0, sv + 0);
          tmem_ld32(s_tmem + 32, sv + 32);
          tc_wait_ld();
          tmem_ld32(s_tmem + 64, sv + 64);
          tmem_ld32(s_tmem + 96, sv + 96);
        }
        float mxa = -INFINITY, mxb = -INFINITY, mxc = -INFINITY, mxd = -INFINITY;
        float mx0, mx1;
        if (!B64) {
          // (the first half's maximum while the second half is still on its way from tensor memory)
#pragma unroll
          for (int e = 0; e < 64; e += 8) {
            mxa = max3(mxa, __uint_as_float(sv[e + 0]), __uint_as_float(sv[e + 1]));
            mxb = max3(mxb, __uint_as_float(sv[e + 2]), __uint_as_float(sv[e + 3]));
            mxc = max3(mxc, __uint_as_float(sv[e + 4]), __uint_as_float(sv[e + 5]));
            mxd = max3(mxd, __uint_as_float(sv[e + 6]), __uint_as_float(sv[e + 7]));
          }
        }
        if (!(REM && fo)) tc_wait_ld();
        tc_fence_before();
        mbar_arrive(bar_s_free + 8 * w);                     // the S issuer may refill this buffer
        if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, j, 2);
        if (B64) {                                           // a, b: keys 0..63; c, d: keys 64..127
#pragma unroll
          for (int e = 0; e < 64; e += 4) {
            mxa = max3(mxa, __uint_as_float(sv[e + 0]), __uint_as_float(sv[e + 1]));
            mxb = max3(mxb, __uint_as_float(sv[e + 2]), __uint_as_float(sv[e + 3]));
            mxc = max3(mxc, __uint_as_float(sv[e + 64]), __uint_as_float(sv[e + 65]));
            mxd = max3(mxd, __uint_as_float(sv[e + 66]), __uint_as_float(sv[e + 67]));
          }
          mx0 = v0 > 0 ? fmaxf(mxa, mxb) : -INFINITY;        // a half this query block does not keep has no say
          mx1 = v1 > 0 ? fmaxf(mxc, mxd) : -INFINITY;
        } else {
#pragma unroll
          for (int e = 64; e < 128; e += 8) {
            mxa = max3(mxa, __uint_as_float(sv[e + 0]), __uint_as_float(sv[e + 1]));
            mxb = max3(mxb, __uint_as_float(sv[e + 2]), __uint_as_float(sv[e + 3]));
            mxc = max3(mxc, __uint_as_float(sv[e + 4]), __uint_as_float(sv[e + 5]));
            mxd = max3(mxd, __uint_as_float(sv[e + 6]), __uint_as_float(sv[e + 7]));
          }
          mx0 = fmaxf(mxa, mxb);
          mx1 = fmaxf(mxc, mxd);
        }
        // (e4m3 with 64-token blocks: each half has its own scale; a half that is not kept stays -inf)
        // (a pooled logit carries + log2(keys per block): a block mean stands for that many keys)
        const float mx = (REM && fo) ? -INFINITY
                       : (B64 && F8) ? fmaxf(v0 > 0 ? mx0 * c : -INFINITY, v1 > 0 ? mx1 * c1 : -INFINITY)
                                     : fmaxf(mx0, mx1) * c + ((REM && pooled) ? prm.log2_block : 0.f);
        // reference exponent left by block j-1 (other group)
        float m_prev = -INFINITY;
        if (j > 0) {
          if (!mbar_wait(bar_ref + 8 * (w ^ 1), prev & 1u, abort_flag, prm.status)) return false;
          m_prev = ref[(w ^ 1) * 128 + row];
        }
        if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, j, 3);
        // lazy rule: raise the reference only when the row maximum outgrows it by more than 2^LAZY_LOG2
        const float m_new = (mx > m_prev + LAZY_LOG2) ? mx : m_prev;
        ref[w * 128 + row] = m_new;
        mbar_arrive(bar_ref + 8 * w);
        if (m_new != m_mine) { l *= ex2(m_mine - m_new); m_mine = m_new; }      // first block: 0 * 2^-inf
        bool pv_waited = false;
        if (j > 0 && __any_sync(0xffffffffu, m_new != m_prev)) {
          // rescale this row of O once P V(j-1) has completed (O is then quiescent: P V(j) waits for us)
          if (!mbar_wait(bar_pv_done + 8 * (w ^ 1), prev & 1u, abort_flag, prm.status)) return false;
          pv_waited = true;
          tc_fence_after();
          const float alpha = ex2(m_prev - m_new);
#pragma unroll 1
          for (int cc = 0; cc < D; cc += 16) {
            uint32_t ov[16];
            tmem_ld16(o_tmem + cc, ov);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * alpha);
            tmem_st16(o_tmem + cc, ov);
          }
          tc_wait_st();
        }
        // P = 2^(S*c - m); the packed bf16 pairs overwrite sv[0..63]
        // (64-token blocks: -inf instead of -m for a half that is not kept, or while the row has seen no
        // kept key yet, makes those P exactly 0 at no cost)
        float nm = -m_new, nmh1 = -m_new;
        if (REM && pooled) { nm += prm.log2_block; nmh1 = nm; }
        if (B64) {
          if (m_new == -INFINITY || v0 == 0) nm = -INFINITY;
          if (m_new == -INFINITY || v1 == 0) nmh1 = -INFINITY;
        }
        const uint64_t c2 = pack2(c, c), nm2 = pack2(nm, nm), nm2h1 = B64 ? pack2(nmh1, nmh1) : nm2;
        const uint64_t c2h1 = (B64 && F8) ? pack2(c1, c1) : c2;
        uint64_t sum2 = pack2(0.f, 0.f);
        if (REM && fo) {
          // P'[i][c] = scale * q_i[c] * exp(mu - m): the row's own query values, for the rows of the query block this
          // tile belongs to (64-token blocks: the other half of the tile row gets zeros); nothing joins the row sum
          const int qb = B64 ? min(2 * I + qh, prm.Nb - 1) : I;
          const bool mine_rows = (qi < prm.N) && (!B64 || qh == (int)(J & 1u)) && m_new != -INFINITY;
          const float f = mine_rows ? prm.scale_log2 * 0.6931471805599453f *
                                          ex2(__ldg(prm.mu + (long long)bh * prm.Nb + qb) * 1.4426950408889634f - m_new)
                                    : 0.f;
          const uint4* src = reinterpret_cast<const uint4*>(prm.q + (long long)bb * prm.sq.b + (long long)hh * prm.sq.h +
                                                            (long long)min(qi, prm.N - 1) * prm.sq.n);
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const uint4 u = __ldg(src + e);
            const uint32_t wd[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int t = 0; t < 4; ++t) sv[4 * e + t] = pack_bf16(bf16lo(wd[t]) * f, bf16hi(wd[t]) * f);
          }
        } else if (!(prm.debug & 1)) {
#pragma unroll
          for (int e = 0; e < 128; e += 2) {
            float x0, x1;
            unpack2(fma2(pack2(__uint_as_float(sv[e]), __uint_as_float(sv[e + 1])), e < 64 ? c2 : c2h1, e < 64 ? nm2 : nm2h1), x0, x1);
            const float p0 = ex2(x0), p1 = ex2(x1);
            sum2 = add2(sum2, pack2(p0, p1));
            sv[e / 2] = pack_bf16(p0, p1);
          }
        }
        {
          float sum_a, sum_b;
          unpack2(sum2, sum_a, sum_b);
          l += sum_a + sum_b;
        }
        if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, j, 4);
        // the P columns are free once P V(j-1) has completed (block 0: the previous row's last P V
        // was waited for in that row's epilogue)
        if (j > 0 && !pv_waited &&
            !mbar_wait(bar_pv_done + 8 * (w ^ 1), prev & 1u, abort_flag, prm.status)) return false;
        if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, j, 5);
        tc_fence_after();
        tmem_st32(p_tmem, sv);
        tmem_st32(p_tmem + 32, sv + 32);
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(bar_p_full + 8 * w);
        if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, j, 6);
        return true;
      };
      for (int j = w; j < n && ok; j += 2) {
        if (!REM || j < n_own) ok = tile(std::integral_constant<int, 0>{}, j);
        else if (j < n_own + prm.np) ok = tile(std::integral_constant<int, 1>{}, j);
        else ok = tile(std::integral_constant<int, 2>{}, j);
      }
      if (!ok) break;
      if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, 255, 7);
      if (EARLYQ && !fetch_row(rows_done + 1u, r_c, n_c, beg_c, e0_c, e1_c, signs)) { ok = false; break; }   // the row after this one, or the end mark
      // ---- epilogue: merge the two groups' row sums, hand the next row's Q to the S issuer,
      // normalise and store (each group half of d)
      if (!EARLYQ && !fetch_row(rows_done + 1u, r_c, n_c, beg_c, e0_c, e1_c, signs)) { ok = false; break; }   // the row after this one, or the end mark
      const int r_next = r_c;                                         // (the queue holds non-empty rows only)
      uint32_t qn[32];
      if (!EARLYQ) load_q(r_next, qn);                                // in flight during the waits below
      if (!mbar_wait(bar_ref + 8 * wl, last & 1u, abort_flag, prm.status)) { ok = false; break; }
      const float m_fin = ref[wl * 128 + row];
      if (m_mine != m_fin) { l *= ex2(m_mine - m_fin); m_mine = m_fin; }        // l = 0 for a group without blocks
      volatile float* lxr = lx + (rows_done & 1u) * 256;
      lxr[w * 128 + row] = l;
      if ((threadIdx.x & 127) == 0) bulk_wait_read0();                // the previous row's store has read the staging panel
      mbar_arrive(bar_xch);
      if (EARLYQ && w != wl) {
        // (after this group's row sums are out, so that the other group's epilogue does not wait for the copy)
        // The row's last S tile (the other group's) has been computed, and with it every S of the row: Q is free.
        // (Its barrier's previous phase completed before the S tile this group has just worked on, or in an earlier row.)
        if (!mbar_wait(bar_s_full + 8 * wl, last & 1u, abort_flag, prm.status)) { ok = false; break; }
        if (r_next < prm.R && !copy_q(r_next, rows_done + 1u)) { ok = false; break; }
        if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, 255, 8);
      }
      if (!mbar_wait(bar_xch, rows_done & 1u, abort_flag, prm.status)) { ok = false; break; }
      // both groups have seen all their S tiles: no MMA reads Q any more
      if (!EARLYQ && r_next < prm.R) store_q(qn, r_next);
      if (!EARLYQ && (threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, 255, 8);
      if (!mbar_wait(bar_pv_done + 8 * wl, last & 1u, abort_flag, prm.status)) { ok = false; break; }
      if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, 255, 9);
      tc_fence_after();
      const float lt = l + lxr[(w ^ 1) * 128 + row];
      // (64-token blocks: a query block with an empty list beside one with work has lt = 0 -> zeros, lse = -inf)
      const float inv = (!B64 || lt > 0.f) ? 1.0f / lt : 0.f;
      {
        uint32_t ov[64];
        tmem_ld32(o_tmem + (D / 2) * w, ov);
        tmem_ld32(o_tmem + (D / 2) * w + 32, ov + 32);
        tc_wait_ld();
        tc_fence_before();
        mbar_arrive(bar_o_free);                                      // the next row may overwrite O
        // normalised bf16 row -> this group's staging panel (128-byte swizzle), then one tile store;
        // rows beyond N are clipped by the tensor map
        uint8_t* stg = smem + OFF_O + w * (TILE / 2) + row * 128;
#pragma unroll
        for (int e = 0; e < 64; e += 8) {
          uint4 v4;
          v4.x = pack_bf16(__uint_as_float(ov[e + 0]) * inv, __uint_as_float(ov[e + 1]) * inv);
          v4.y = pack_bf16(__uint_as_float(ov[e + 2]) * inv, __uint_as_float(ov[e + 3]) * inv);
          v4.z = pack_bf16(__uint_as_float(ov[e + 4]) * inv, __uint_as_float(ov[e + 5]) * inv);
          v4.w = pack_bf16(__uint_as_float(ov[e + 6]) * inv, __uint_as_float(ov[e + 7]) * inv);
          *reinterpret_cast<uint4*>(stg + (((e >> 3) ^ (row & 7)) << 4)) = v4;
        }
        fence_async_smem();
        mbar_arrive(bar_ost + 8 * w);
        if ((threadIdx.x & 127) == 0) {
          // (a wait that runs out has raised the abort flag; the other threads leave at their next wait)
          if (mbar_wait(bar_ost + 8 * w, rows_done & 1u, abort_flag, prm.status) && (D / 2) * w < prm.d) {
            tma_store_4d(&tm_o, sbase + OFF_O + w * (TILE / 2), (D / 2) * w, I * BS, hh, bb);
            bulk_commit();
          }
        }
        if (qi < prm.N && prm.lse && w == 0) prm.lse[(long long)bh * prm.N + qi] = (m_fin + log2f(lt)) * 0.6931471805599453f;
      }
      if ((threadIdx.x & 127) == 0) SVA_STAMP(w, rows_done, 255, 10);
      cnt[0] += (uint32_t)((n + 1) >> 1);
      cnt[1] += (uint32_t)(n >> 1);
    }
    if ((threadIdx.x & 127) == 0) bulk_wait0();                       // my output stores have completed
  }

  // ---------------------------------------------------------------- tear-down
  if (prm.prof && threadIdx.x == 0)
    atomicMax(reinterpret_cast<unsigned long long*>(prm.prof + 319), (unsigned long long)(clock64() - t_cta0));
#ifdef SVA_TIMELINE
  __syncthreads();
  if (prm.prof && blockIdx.x == 0) for (int i_ = threadIdx.x; i_ < 1400; i_ += THREADS) prm.prof[512 + i_] = (long long)stamp_buf[i_];
#endif
  if (*abort_flag) {
    // give copies and MMAs still in flight time to land before shared memory and TMEM go away
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------ V^T
// V [B,H,N,d] (strided) -> tiled transposed copy: for every (b,h) and key block J (kb = 128 or 64
// keys) one contiguous tile [d = 128 rows][kb keys], keys >= N zero.  A 128-key tile is then one
// contiguous TMA box pair, exactly like a K tile; a 64-key tile is one box (one panel of a tile).
__global__ void __launch_bounds__(256)
transpose_v_kernel(const __nv_bfloat16* __restrict__ v, Strides sv, __nv_bfloat16* __restrict__ vt, int H, int N,
                   int Nb, int d, int kb, int32_t* __restrict__ row_counter) {
  // d = 64: the tile still has 128 d-rows; the CTAs of the upper half (d0 >= d) write zeros
  // the attention kernel that follows draws its rows from this counter
  if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) {
    row_counter[0] = 0;     // next row to hand out
    row_counter[1] = 0;     // CTAs that have finished drawing
  }
  __shared__ __nv_bfloat16 tile[64][66];            // [d][key], padded
  const int n0 = blockIdx.x * 64, d0 = blockIdx.y * 64, bh = blockIdx.z;
  const int b = bh / H, h = bh % H;
  const __nv_bfloat16* src = v + (long long)b * sv.b + (long long)h * sv.h;
  {
    const int c8 = threadIdx.x & 7;                 // 8 d-values (16 bytes)
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
      const int key = (threadIdx.x >> 3) + 32 * pass;
      uint4 u = make_uint4(0, 0, 0, 0);
      if (n0 + key < N && d0 < d) u = __ldg(reinterpret_cast<const uint4*>(src + (long long)(n0 + key) * sv.n + d0) + c8);
      const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&u);
#pragma unroll
      for (int q = 0; q < 8; ++q) tile[c8 * 8 + q][key] = e[q];
    }
  }
  __syncthreads();
  {
    const int k8 = threadIdx.x & 7;                 // 8 keys (16 bytes)
    const int J = n0 / kb, kin = (n0 % kb) + k8 * 8;
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
      const int dd = (threadIdx.x >> 3) + 32 * pass;
      __align__(16) __nv_bfloat16 e[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) e[q] = tile[dd][k8 * 8 + q];
      *reinterpret_cast<uint4*>(vt + (((long long)bh * Nb + J) * ts::D + d0 + dd) * kb + kin) = *reinterpret_cast<uint4*>(e);
    }
  }
}

// ------------------------------------------------------------------ 64-token blocks: tile lists
// The MMA tile is 128 x 128, so with 64-token blocks one tile row is two adjacent query blocks (A, B)
// and one tile two key blocks.  Per tile row this kernel merges the two CSR rows into the ascending
// union of their key blocks, pairs the union up into tiles and notes for every key block which of the
// two query blocks keeps it (the softmax excludes the other).  One warp per tile row: membership
// bitmaps in shared memory, then every lane enumerates the bits of its word.  Entries are 16 bits
// {key block (14), kept by A, kept by B}; tile j of the row is the 32-bit word at start + j.  The
// start needs no scan: ceil((entries before the tile row + its index) / 2) leaves room for every earlier
// row's ceil(|union| / 2) tiles.
constexpr int PAIR_WARPS = 8;
__global__ void __launch_bounds__(PAIR_WARPS * 32)
pair_lists_kernel(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col_idx, int Nb, int Nt, int R2,
                  int32_t* __restrict__ tile_cnt, int32_t* __restrict__ tile_beg, uint32_t* __restrict__ tile_desc,
                  long long cap, int32_t* __restrict__ status) {
  __shared__ uint32_t bm[PAIR_WARPS][2][32];
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * PAIR_WARPS + w;
  if (t >= R2) return;
  const int bh = t / Nt, I2 = t % Nt;
  const int rA = bh * Nb + 2 * I2;
  const bool hasB = 2 * I2 + 1 < Nb;
  bm[w][0][lane] = 0u;
  bm[w][1][lane] = 0u;
  __syncwarp();
  const int begA = __ldg(row_ptr + rA), endA = __ldg(row_ptr + rA + 1);
  const int endB = hasB ? __ldg(row_ptr + rA + 2) : endA;
  const int nnz_bound = __ldg(row_ptr + (R2 / Nt) * Nb);      // row_ptr[R]: the entries the CSR says it has
  const bool bad = begA < 0 || endA < begA || endB < endA || endA - begA > Nb || endB - endA > Nb || endB > nnz_bound;
  bool bad_idx = false;
  if (!bad) {
    for (int e = begA + lane; e < endB; e += 32) {
      const int J = __ldg(col_idx + e);
      if (J < 0 || J >= Nb) { bad_idx = true; continue; }
      atomicOr(&bm[w][e < endA ? 0 : 1][J >> 5], 1u << (J & 31));
    }
  }
  if ((bad || bad_idx) && status) atomicOr(status, SVA_DEV_BAD_INDEX);
  __syncwarp();
  const uint32_t a = bm[w][0][lane], b = bm[w][1][lane];
  uint32_t u = a | b;
  int incl = __popc(u);
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += x;
  }
  const int total = __shfl_sync(0xffffffffu, incl, 31);
  long long start = ((long long)(bad ? 0 : begA) + t + 1) / 2;
  int ntile = (total + 1) / 2;
  if (start + ntile > cap) { ntile = 0; if (lane == 0 && status) atomicOr(status, SVA_DEV_BAD_INDEX); }
  if (ntile > 0) {
    uint16_t* ent = reinterpret_cast<uint16_t*>(tile_desc) + 2 * start;
    int p = incl - __popc(u);
    while (u) {
      const int bit = __ffs(u) - 1;
      u &= u - 1;
      ent[p++] = (uint16_t)((lane * 32 + bit) | (((a >> bit) & 1u) << 14) | (((b >> bit) & 1u) << 15));
    }
    if (lane == 0 && (total & 1)) ent[total] = 0;          // odd union: the last tile's second half is nobody's
  }
  if (lane == 0) {
    tile_cnt[t] = ntile;
    tile_beg[t] = (int32_t)start;
  }
}

// ------------------------------------------------------------------ remainder: block means of K and V
// One CTA per (block J, head, tensor): the mean over the existing tokens of the block, fp32 accumulation in a
// fixed order, rounded to bf16.  K means go to kp [B*H][Nbp][128] (rows >= Nb stay zero: the launcher clears the
// buffer), V means transposed to vtp [B*H][np][128 d][128 blocks], the layout of a V^T tile.
__global__ void __launch_bounds__(256)
pool_kv_kernel(const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, Strides sk, Strides sv,
               int H, int N, int block, int Nb, int Nbp, __nv_bfloat16* __restrict__ kp,
               __nv_bfloat16* __restrict__ vtp, int v_rows) {
  __shared__ float part[16][ts::D + 1];
  const int J = blockIdx.x, bh = blockIdx.y, which = blockIdx.z;
  const int b = bh / H, h = bh % H;
  const Strides s = which ? sv : sk;
  const __nv_bfloat16* base = (which ? v : k) + (long long)b * s.b + (long long)h * s.h;
  const int lo = J * block, cnt = min(block, N - lo);
  const int vec = threadIdx.x & 15, grp = threadIdx.x >> 4;          // 16 vectors of 8 elements per row, 16 rows at a time
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;
  for (int t = grp; t < cnt; t += 16) {
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(base + (long long)(lo + t) * s.n) + vec);
    const uint32_t wd[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) { acc[2 * e] += bf16lo(wd[e]); acc[2 * e + 1] += bf16hi(wd[e]); }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) part[grp][vec * 8 + e] = acc[e];
  __syncthreads();
  if (threadIdx.x < ts::D) {
    float sum = 0.f;
#pragma unroll
    for (int g = 0; g < 16; ++g) sum += part[g][threadIdx.x];
    const __nv_bfloat16 mean = __float2bfloat16_rn(sum / (float)cnt);
    if (which == 0 || v_rows)                                 // (v_rows: the means of V laid out like those of K)
      (which ? vtp : kp)[((long long)bh * Nbp + J) * ts::D + threadIdx.x] = mean;
    else
      vtp[(((long long)bh * (Nbp >> 7) + (J >> 7)) * ts::D + threadIdx.x) * BS + (J & 127)] = mean;
  }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*encode_fn_t)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                CUtensorMapFloatOOBfill);

static encode_fn_t get_encode_ts() {
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

// 4-D map (inner, rows, H, B) of bf16 (or bytes) with byte strides; box = 128 bytes x box_rows, 128-byte swizzle.
// (box_bytes = 64: rows of 64 bytes with the 64-byte swizzle, the packed 4-bit tiles)
static int make_map_ts(CUtensorMap* map, const void* ptr, cuuint64_t inner, cuuint64_t rows, int H, int B,
                       cuuint64_t row_stride, cuuint64_t h_stride, cuuint64_t b_stride, int box_rows,
                       int elem_bytes = 2, int box_bytes = 128) {
  encode_fn_t enc = get_encode_ts();
  if (!enc) return SVA_ERR_CUDA;
  cuuint64_t dims[4] = {inner, rows, (cuuint64_t)H, (cuuint64_t)B};
  cuuint64_t strides[3] = {row_stride, h_stride, b_stride};
  // a size-1 dimension may carry any stride; give it a legal one
  if (H == 1) strides[1] = strides[0] * rows;
  if (B == 1) strides[2] = strides[1] * (cuuint64_t)H;
  for (int i = 0; i < 3; ++i)
    if (strides[i] % 16 != 0 || strides[i] == 0) return SVA_ERR_ALIGNMENT;
  cuuint32_t box[4] = {(cuuint32_t)(box_bytes / elem_bytes), (cuuint32_t)box_rows, 1, 1};   // 128 (or 64) bytes per row
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult rc = enc(map, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, box_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? SVA_OK : SVA_ERR_CUDA;
}

static long long* g_prof_ts = nullptr;
static int g_debug_ts = 0;

// Per-device constants looked up once (the SM count, and the shared-memory opt-in of each kernel variant):
// a cache, not state -- every call would find the same values.
static constexpr int TS_MAX_DEVICES = 64;
static std::mutex g_ts_mutex;
static int g_ts_sms[TS_MAX_DEVICES];
static bool g_ts_attr[TS_MAX_DEVICES][16];

template <bool B64, bool F8, bool REM = false, bool F4 = false, bool VMN = false>
static int launch_ts(int rows, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& to,
                     const CUtensorMap& tkp, const CUtensorMap& tvp, const CUtensorMap& tat, const CUtensorMap& tq,
                     const TsParams& prm, cudaStream_t st) {
  auto kern = attn_ts_kernel<B64, F8, REM, F4, VMN>;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= TS_MAX_DEVICES) return SVA_ERR_CUDA;
  {
    std::lock_guard<std::mutex> lock(g_ts_mutex);
    constexpr int variant = F4 ? 8 : (VMN ? 9 : 0) + (REM ? 4 : 0) + (B64 ? 2 : 0) + (F8 ? 1 : 0);
    if (!g_ts_attr[dev][variant]) {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ts::SMEM_BYTES) != cudaSuccess)
        return SVA_ERR_CUDA;
      g_ts_attr[dev][variant] = true;
    }
    if (g_ts_sms[dev] <= 0 &&
        (cudaDeviceGetAttribute(&g_ts_sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || g_ts_sms[dev] <= 0))
      return SVA_ERR_CUDA;
    sms = g_ts_sms[dev];
  }
  const int grid = rows < sms ? rows : sms;        // persistent: one CTA per SM, rows drawn from a counter
  kern<<<grid, ts::THREADS, ts::SMEM_BYTES, st>>>(tk, tv, to, tkp, tvp, tat, tq, prm);
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

// Workspace layout: transposed V tiles | row counter (256 bytes) | 64-token blocks only: tile_cnt[R2],
// tile_beg[R2], tile_desc[cap] with R2 = B*H*ceil(Nb/2) tile rows and cap the bound for a dense CSR.
struct TsLayout {
  size_t vt_bytes, counter_off, cnt_off, beg_off, desc_off, total;
  size_t kp_off, vtp_off, pooled_bytes, total_rem;      // remainder: bf16 block means of K, and of V transposed
  int np, Nbp;
  long long cap;
  int R2, Nt;
};
// (no_vt: V is read where it lies -- no transposed copy, the rest moves to the front)
static TsLayout ts_layout(const Dims& m, bool no_vt = false) {
  TsLayout L;
  L.vt_bytes = no_vt ? 0 : (size_t)m.B * m.H * m.Nb * m.block * ts::D * 2;      // (d = 64: tiles are padded to 128 d-rows)
  L.counter_off = L.vt_bytes;
  L.Nt = m.block == 64 ? (m.Nb + 1) / 2 : m.Nb;
  L.R2 = m.B * m.H * L.Nt;
  L.cnt_off = L.beg_off = L.desc_off = L.counter_off + 256;
  L.cap = 0;
  L.total = L.counter_off + 256;
  if (m.block == 64) {
    L.beg_off = L.cnt_off + (((size_t)L.R2 * 4 + 255) & ~(size_t)255);
    L.desc_off = L.beg_off + (((size_t)L.R2 * 4 + 255) & ~(size_t)255);
    L.cap = ((long long)m.R * m.Nb + L.R2) / 2 + 2;
    L.total = L.desc_off + (((size_t)L.cap * 4 + 255) & ~(size_t)255);
  }
  L.np = (m.Nb + BS - 1) / BS;
  L.Nbp = L.np * BS;
  L.pooled_bytes = (size_t)m.B * m.H * L.Nbp * ts::D * 2;
  L.kp_off = L.total;
  L.vtp_off = L.kp_off + L.pooled_bytes;
  L.total_rem = L.vtp_off + L.pooled_bytes;
  return L;
}

bool attn_ts_serves(const Dims& m) {
  return (m.d == 128 || m.d == 64) && m.Nb <= 16383 && (m.block == BS || m.block == 64);
}

// The remainder variant: bf16 Q/K, d = 128, a CSR (the dense form drops nothing).
bool attn_ts_remainder_serves(const Dims& m) { return attn_ts_serves(m) && m.d == ts::D && !m.fp8; }
size_t remainder1_bytes(const Dims& m);
int launch_remainder1(const Dims& m, const sva_problem_t* p, const void* k, const void* v, const float* scores,
                      const int32_t* row_ptr, const int32_t* col_idx, void* buf, const __nv_bfloat16** at_out,
                      const float** mu_out, int32_t* status, cudaStream_t st, bool natural);
// (order 1 adds the buffers of the first-order term behind those of order 0)
size_t attn_ts_remainder_workspace_bytes(const Dims& m, int order) {
  if (!attn_ts_remainder_serves(m)) return 0;
  return ts_layout(m, !(g_debug_ts & 32)).total_rem + (order >= 1 ? remainder1_bytes(m) : 0);
}

// What the one-call entry points need: they read V where it lies, so only the row counters (and the tile lists of
// 64-token blocks) remain.  (The transposed copy in the one-call form is a measurement aid: debug bit 5, which then
// needs the workspace of the two-step form.)
size_t attn_ts_one_call_workspace_bytes(const Dims& m) {
  if (!attn_ts_serves(m)) return 0;
  if (g_debug_ts & 32) return attn_ts_workspace_bytes(m);
  size_t bytes = ts_layout(m, true).total;
  if (m.block == 64 && !m.fp8) {            // the dense entry point runs 64-token blocks as 128-token blocks
    Dims d = m;
    d.block = BS; d.Nb = (m.N + BS - 1) / BS; d.R = m.B * m.H * d.Nb;
    const size_t b2 = ts_layout(d, true).total;
    if (b2 > bytes) bytes = b2;
  }
  return bytes;
}

size_t attn_ts_workspace_bytes(const Dims& m) {
  if (!attn_ts_serves(m)) return 0;
  size_t bytes = ts_layout(m).total;
  if (m.block == 64) {                      // the dense entry point runs 64-token blocks as 128-token blocks
    Dims d = m;
    d.block = BS; d.Nb = (m.N + BS - 1) / BS; d.R = m.B * m.H * d.Nb;
    const size_t b2 = ts_layout(d).total;
    if (b2 > bytes) bytes = b2;
  }
  return bytes;
}

static int check_ts_workspace(const Dims& m, const void* ws, size_t ws_bytes, bool one_call = false) {
  if (!attn_ts_serves(m)) return SVA_ERR_UNSUPPORTED;
  if (!ws || ws_bytes < (one_call ? attn_ts_one_call_workspace_bytes(m) : attn_ts_workspace_bytes(m))) return SVA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return SVA_ERR_ALIGNMENT;
  return SVA_OK;
}

// V -> tiled transposed copy in the workspace, row counter of the scheduler = 0.
int launch_prepare_v_ts(const Dims& m, const sva_problem_t* p, const void* v, void* ws, size_t ws_bytes,
                        cudaStream_t st) {
  int rc = check_ts_workspace(m, ws, ws_bytes);
  if (rc) return rc;
  const TsLayout L = ts_layout(m);
  const Strides sv = make_strides(p->v_stride);
  dim3 tg((m.Nb * m.block + 63) / 64, ts::D / 64, m.B * m.H);    // every key slot of every tile, also those beyond N (zeros)
  transpose_v_kernel<<<tg, 256, 0, st>>>((const __nv_bfloat16*)v, sv, (__nv_bfloat16*)ws, m.H, m.N, m.Nb, m.d, m.block,
                                         reinterpret_cast<int32_t*>(static_cast<uint8_t*>(ws) + L.counter_off));
  return cudaGetLastError() == cudaSuccess ? SVA_OK : SVA_ERR_CUDA;
}

// v == nullptr: the workspace has been prepared by launch_prepare_v_ts (once per attention call).
// remainder_order < 0: exact attention over the kept blocks only.  0: plus the block-mean remainder of the
// dropped blocks (needs v, a CSR and the larger workspace of attn_ts_remainder_workspace_bytes).  1: plus the
// first-order term (needs the routing's score matrix as well).
int launch_attn_ts(const Dims& m_in, const sva_problem_t* p, const void* q, const void* k, const void* v,
                   const float* q_scale, const float* k_scale, const int32_t* row_ptr, const int32_t* col_idx, void* o, float* lse, int32_t* status,
                   void* ws, size_t ws_bytes, cudaStream_t st, int remainder_order, const float* block_scores) {
  int rc = check_ts_workspace(m_in, ws, ws_bytes, v != nullptr);
  if (rc) return rc;
  const bool rem = remainder_order >= 0;
  if (rem) {
    if (remainder_order > 1 || !attn_ts_remainder_serves(m_in) || !row_ptr || !v) return SVA_ERR_UNSUPPORTED;
    if (remainder_order == 1 && !block_scores) return SVA_ERR_INVALID_ARG;
    if (ws_bytes < attn_ts_remainder_workspace_bytes(m_in, remainder_order)) return SVA_ERR_WORKSPACE;
  }
  // dense attention does not depend on the block size: 64-token blocks run as 128-token blocks
  Dims m = m_in;
  if (m.block == 64 && row_ptr == nullptr && !m.fp8) {     // (e4m3 scales are per 64-token block: that stays as it is)
    m.block = BS;
    m.Nb = (m.N + BS - 1) / BS;
    m.R = m.B * m.H * m.Nb;
  }
  const bool b64 = m.block == 64;
  // With V at hand it is read where it lies (an MN-major B operand): no transposed copy, no workspace for it, and
  // under the power cap the step is faster without the copy's HBM traffic although the kernel needs 1 % more cycles.
  // (The two-step form keeps the copy, and so does the remainder; bit 5 of the debug mode forces it here, to measure.)
  const bool vmn = v != nullptr && !(g_debug_ts & 32);
  const TsLayout L = ts_layout(m, vmn);
  uint8_t* wsb = static_cast<uint8_t*>(ws);
  const Strides sk = make_strides(p->k_stride);
  const Strides so = make_strides(p->o_stride);
  CUtensorMap tk, tv, to, tkp, tvp, tat;
  const float* mu_dev = nullptr;
  if ((rc = make_map_ts(&to, o, m.d, m.N, m.H, m.B, (cuuint64_t)so.n * 2, (cuuint64_t)so.h * 2, (cuuint64_t)so.b * 2, BS)) != SVA_OK)
    return rc;
  const int eb = m.fp8 ? 1 : 2;
  if ((rc = make_map_ts(&tk, k, m.d, m.N, m.H, m.B, (cuuint64_t)sk.n * eb, (cuuint64_t)sk.h * eb, (cuuint64_t)sk.b * eb,
                        m.block, eb)) != SVA_OK)
    return rc;
  // transposed V: per (b,h) a [Nb*128 rows][block keys] matrix, key block J = rows J*128 .. J*128+127
  const cuuint64_t vrows = (cuuint64_t)m.Nb * ts::D;
  if ((rc = make_map_ts(&tv, ws, m.block, vrows, m.H, m.B, (cuuint64_t)m.block * 2, vrows * m.block * 2,
                        vrows * m.block * 2 * m.H, BS)) != SVA_OK)
    return rc;
  tkp = tk; tvp = tv; tat = tv;  // (placeholders when there is no remainder: the kernel never touches them)
  // Q as 128-row tiles, like K (128-token blocks: a row's Q reaches the kernel by TMA; otherwise unused)
  CUtensorMap tq = tk;
  if (!b64) {
    const Strides sq = make_strides(p->q_stride);
    if ((rc = make_map_ts(&tq, q, m.d, m.N, m.H, m.B, (cuuint64_t)sq.n * eb, (cuuint64_t)sq.h * eb, (cuuint64_t)sq.b * eb,
                          m.block, eb)) != SVA_OK)
      return rc;
  }
  if (rem && remainder_order == 1) {
    // first-order term: C_J, weights, A_I (remainder.cu) into the buffers behind those of order 0
    const __nv_bfloat16* at = nullptr;
    if ((rc = launch_remainder1(m, p, k, v, block_scores, row_ptr, col_idx, wsb + L.total_rem, &at, &mu_dev, status, st, vmn)) != SVA_OK)
      return rc;
    const cuuint64_t arow = (cuuint64_t)m.Nb * BS;               // per head: Nb matrices of 128 rows x 128 bf16
    if ((rc = make_map_ts(&tat, at, BS, arow, m.H, m.B, (cuuint64_t)BS * 2, arow * BS * 2, arow * BS * 2 * m.H, BS)) != SVA_OK)
      return rc;
  }
  if (rem) {
    // block means of K ([Nbp rows][128], rows >= Nb zero) and of V (transposed tiles), then their maps
    __nv_bfloat16* kp = reinterpret_cast<__nv_bfloat16*>(wsb + L.kp_off);
    __nv_bfloat16* vtp = reinterpret_cast<__nv_bfloat16*>(wsb + L.vtp_off);
    if (cudaMemsetAsync(kp, 0, 2 * L.pooled_bytes, st) != cudaSuccess) return SVA_ERR_CUDA;
    pool_kv_kernel<<<dim3(m.Nb, m.B * m.H, 2), 256, 0, st>>>((const __nv_bfloat16*)k, (const __nv_bfloat16*)v, sk,
                                                            make_strides(p->v_stride), m.H, m.N, m.block, m.Nb, L.Nbp, kp, vtp,
                                                            vmn ? 1 : 0);
    if (cudaGetLastError() != cudaSuccess) return SVA_ERR_CUDA;
    const cuuint64_t prow = (cuuint64_t)L.Nbp;
    if ((rc = make_map_ts(&tkp, kp, ts::D, prow, m.H, m.B, (cuuint64_t)ts::D * 2, prow * ts::D * 2,
                          prow * ts::D * 2 * m.H, BS)) != SVA_OK)
      return rc;
    // (V read where it lies: the block means of V as rows, like those of K; else transposed, like a V^T tile)
    if ((rc = make_map_ts(&tvp, vtp, BS, prow, m.H, m.B, (cuuint64_t)BS * 2, prow * BS * 2, prow * BS * 2 * m.H, BS)) != SVA_OK)
      return rc;
  }
  if (vmn) {
    const Strides sv = make_strides(p->v_stride);
    if ((rc = make_map_ts(&tv, v, m.d, m.N, m.H, m.B, (cuuint64_t)sv.n * 2, (cuuint64_t)sv.h * 2, (cuuint64_t)sv.b * 2,
                          m.block)) != SVA_OK)
      return rc;
    if (!rem) tvp = tv;
    if (cudaMemsetAsync(wsb + L.counter_off, 0, 256, st) != cudaSuccess) return SVA_ERR_CUDA;
  } else if (v) {
    // (the transposed copy is laid out for the block size of this launch)
    const Strides sv = make_strides(p->v_stride);
    dim3 tg((m.Nb * m.block + 63) / 64, ts::D / 64, m.B * m.H);    // every key slot of every tile, also those beyond N (zeros)
    transpose_v_kernel<<<tg, 256, 0, st>>>((const __nv_bfloat16*)v, sv, (__nv_bfloat16*)ws, m.H, m.N, m.Nb, m.d, m.block,
                                           reinterpret_cast<int32_t*>(wsb + L.counter_off));
    if (cudaGetLastError() != cudaSuccess) return SVA_ERR_CUDA;
  } else if (m.block != m_in.block) {
    return SVA_ERR_UNSUPPORTED;     // a workspace prepared for 64-token blocks cannot serve the dense path
  }
  TsParams prm;
  prm.q = (const __nv_bfloat16*)q; prm.sq = make_strides(p->q_stride);
  prm.q_scale = q_scale; prm.k_scale = k_scale;
  prm.q_sf = nullptr; prm.k_sf = nullptr;
  prm.row_ptr = row_ptr; prm.col_idx = col_idx;
  prm.o = (__nv_bfloat16*)o; prm.lse = lse; prm.status = status;
  prm.so = make_strides(p->o_stride);
  prm.H = m.H; prm.N = m.N; prm.Nb = m.Nb; prm.Nt = L.Nt; prm.R = L.R2; prm.d = m.d;
  prm.tile_cnt = reinterpret_cast<const int32_t*>(wsb + L.cnt_off);
  prm.tile_beg = reinterpret_cast<const int32_t*>(wsb + L.beg_off);
  prm.tile_desc = reinterpret_cast<const uint32_t*>(wsb + L.desc_off);
  prm.scale_log2 = m.scale * 1.4426950408889634f;
  prm.next_row = reinterpret_cast<int32_t*>(wsb + L.counter_off);
  prm.np = rem ? L.np : 0;
  prm.rem_mask = (rem && !b64 && m.Nb <= 1024 && !(g_debug_ts & 128)) ? 1 : 0;
  prm.n1 = (rem && remainder_order == 1) ? (b64 ? 2 : 1) : 0;
  prm.mu = mu_dev;
  prm.log2_block = log2f((float)m.block);
  {
    const int tail = m.N - (m.Nb - 1) * m.block;
    prm.tail_bias = (log2f((float)tail) - prm.log2_block) / prm.scale_log2;
  }
  prm.prof = g_prof_ts;
  prm.debug = g_debug_ts;
  if (b64) {
    if (row_ptr) {                      // (dense, e4m3 only: the kernel makes up the tile lists itself)
      pair_lists_kernel<<<(L.R2 + PAIR_WARPS - 1) / PAIR_WARPS, PAIR_WARPS * 32, 0, st>>>(
          row_ptr, col_idx, m.Nb, L.Nt, L.R2, reinterpret_cast<int32_t*>(wsb + L.cnt_off),
          reinterpret_cast<int32_t*>(wsb + L.beg_off), reinterpret_cast<uint32_t*>(wsb + L.desc_off), L.cap, status);
      if (cudaGetLastError() != cudaSuccess) return SVA_ERR_CUDA;
    }
    if (rem) return vmn ? launch_ts<true, false, true, false, true>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st)
                        : launch_ts<true, false, true>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st);
    if (m.fp8) return vmn ? launch_ts<true, true, false, false, true>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st)
                          : launch_ts<true, true>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st);
    return vmn ? launch_ts<true, false, false, false, true>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st)
               : launch_ts<true, false>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st);
  }
  if (rem) return vmn ? launch_ts<false, false, true, false, true>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st)
                      : launch_ts<false, false, true>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st);
  if (m.fp8) return vmn ? launch_ts<false, true, false, false, true>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st)
                        : launch_ts<false, true>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st);
  return vmn ? launch_ts<false, false, false, false, true>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st)
             : launch_ts<false, false>(L.R2, tk, tv, to, tkp, tvp, tat, tq, prm, st);
}

// 4-bit Q/K: packed codes [B*H][Nb*128][64], tiled scale factors, one fp32 scale per (b,h); V bf16 as always.
bool attn_ts_fp4_serves(const Dims& m) { return m.d == ts::D && m.block == BS && !m.fp8 && m.Nb <= 16383; }

int launch_attn_ts_fp4(const Dims& m, const sva_problem_t* p, const void* q4, const void* k4, const void* q_sf,
                       const void* k_sf, const float* q_g, const float* k_g, const void* v, const int32_t* row_ptr,
                       const int32_t* col_idx, void* o, float* lse, int32_t* status, void* ws, size_t ws_bytes,
                       cudaStream_t st) {
  if (!attn_ts_fp4_serves(m)) return SVA_ERR_UNSUPPORTED;
  const TsLayout L = ts_layout(m, true);                      // V is read where it lies: the row counters only
  if (!ws || ws_bytes < L.total) return SVA_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return SVA_ERR_ALIGNMENT;
  int rc;
  uint8_t* wsb = static_cast<uint8_t*>(ws);
  const Strides so = make_strides(p->o_stride);
  CUtensorMap tk, tv, to, tq;
  if ((rc = make_map_ts(&to, o, m.d, m.N, m.H, m.B, (cuuint64_t)so.n * 2, (cuuint64_t)so.h * 2, (cuuint64_t)so.b * 2, BS)) != SVA_OK)
    return rc;
  const cuuint64_t crow = (cuuint64_t)m.Nb * BS;              // token rows of the code tensors (padded to whole blocks)
  if ((rc = make_map_ts(&tk, k4, 64, crow, m.H, m.B, 64, crow * 64, crow * 64 * m.H, BS, 1, 64)) != SVA_OK) return rc;
  if ((rc = make_map_ts(&tq, q4, 64, crow, m.H, m.B, 64, crow * 64, crow * 64 * m.H, BS, 1, 64)) != SVA_OK) return rc;
  const Strides sv = make_strides(p->v_stride);
  if ((rc = make_map_ts(&tv, v, m.d, m.N, m.H, m.B, (cuuint64_t)sv.n * 2, (cuuint64_t)sv.h * 2, (cuuint64_t)sv.b * 2,
                        BS)) != SVA_OK)
    return rc;
  if (cudaMemsetAsync(wsb + L.counter_off, 0, 256, st) != cudaSuccess) return SVA_ERR_CUDA;
  TsParams prm = {};
  prm.q = nullptr; prm.sq = Strides{0, 0, 0};
  prm.q_scale = q_g; prm.k_scale = k_g;
  prm.q_sf = static_cast<const uint8_t*>(q_sf); prm.k_sf = static_cast<const uint8_t*>(k_sf);
  prm.row_ptr = row_ptr; prm.col_idx = col_idx;
  prm.o = (__nv_bfloat16*)o; prm.lse = lse; prm.status = status;
  prm.so = so;
  prm.H = m.H; prm.N = m.N; prm.Nb = m.Nb; prm.Nt = L.Nt; prm.R = L.R2; prm.d = m.d;
  prm.tile_cnt = nullptr; prm.tile_beg = nullptr; prm.tile_desc = nullptr;
  prm.scale_log2 = m.scale * 1.4426950408889634f;
  prm.next_row = reinterpret_cast<int32_t*>(wsb + L.counter_off);
  prm.np = 0; prm.rem_mask = 0; prm.n1 = 0; prm.mu = nullptr; prm.log2_block = 7.f; prm.tail_bias = 0.f;
  prm.prof = g_prof_ts;
  prm.debug = g_debug_ts;
  return launch_ts<false, false, false, true, true>(L.R2, tk, tv, to, tq, tv, tv, tq, prm, st);
}

void ts_set_prof_buffer(void* p) { g_prof_ts = (long long*)p; }
void ts_set_debug_mode(int v) { g_debug_ts = v; }
int ts_set_wait_limit(long long cycles) {
  if (cycles <= 0) cycles = WAIT_LIMIT_CYCLES;
  return cudaMemcpyToSymbol(g_wait_limit, &cycles, sizeof(cycles)) == cudaSuccess ? 0 : 1;
}

}  // namespace sva
