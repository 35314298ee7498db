// One persistent, warp-specialised tcgen05 contraction kernel, instantiated with
// six epilogues:
//   MODE_LSE    z = H.W^T tile by tile; per-row running (max, sum-exp) and target logit
//   MODE_GRAD   z recomputed; g = c*(onehot - softmax) written as a bf16 row chunk
//   MODE_DH     dH = g . W      (contraction over the vocabulary), optional per-row scale
//   MODE_DW     dW (+)= g^T . H (contraction over the rows of the range)
//   MODE_LSE_E  z tile by tile; e = exp(z - zref_row) staged as bf16 for a range of whole
//               sequences, per-row sum of e and target logit (no recompute in the backward)
//   MODE_DEBUG  plain C = A.B for bring-up of the four operand-major combinations
//
// The kernel runs as pairs of CTAs (clusters of two, one pair per two SMs) that share one
// tile per step through tcgen05.mma.cta_group::2: each CTA loads its own 128 rows of A and
// 128 of every 256 columns of B (so every operand byte is fetched from L2 by one SM only,
// without multicast), the leader CTA's UMMA thread issues for both, and each CTA's TMEM
// receives its 128 rows of the accumulators.
// Warp 0 issues TMA loads, warp 1 owns TMEM (and, in the leader, issues the UMMAs), the
// remaining warps are the epilogue: four (one TMEM lane quadrant each) or, in the vocabulary
// sweeps, eight (two per quadrant, each taking half of an accumulator's columns).
//
// Two tile shapes (template parameter NACC):
//   NACC = 1  256 x 256 pair tile, six shared-memory stages of 32 KB per CTA, the two
//             256-column fp32 accumulators in TMEM alternate so that the epilogue of tile j
//             overlaps the main loop of tile j+1.  Only the bring-up GEMM uses it now.
//   NACC = 2  256 x 512 pair tile: both accumulators belong to one tile and every A slab
//             feeds two UMMAs, so a third less operand traffic from L2 per flop and half as
//             many re-reads of the streamed operand from HBM; four stages of 48 KB.  The
//             accumulators do not alternate, so the epilogue is exposed except for what the
//             half-accumulator order hides: the epilogue drains accumulator 0 first and
//             releases it, and the UMMA thread starts the next tile with accumulator 0's
//             share of the first four K-steps while accumulator 1 is still being drained.
//             In the vocabulary sweeps the end of a tile is skewed the same way: the last four
//             K-steps are issued for accumulator 0 first, which goes to the epilogue on its own
//             barrier while accumulator 1's share of those K-steps still runs.
//             dH (K = V) and dW (K = rows of the range) have long K loops and four epilogue
//             warps; dW leaves through TMA reduce-add.  The vocabulary sweeps (short K = d,
//             an exponential per element, bf16 stores in two of the three) have eight.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "sm100_ptx.cuh"
#include "sweep_schedule.cuh"

namespace oapl {

enum { MODE_LSE = 0, MODE_GRAD = 1, MODE_DH = 2, MODE_DW = 3, MODE_DEBUG = 4, MODE_LSE_E = 5 };

constexpr int kBM = 128;      // rows of A / of the accumulator per CTA
constexpr int kTileM = 256;   // rows per CTA pair
constexpr int kBN = 256;      // accumulator columns (per pair and per CTA)
constexpr int kHalfN = 128;   // columns of B each CTA loads
constexpr int kBK = 64;
constexpr int kABytes = kBM * kBK * 2;     // 16 KB
constexpr int kBBytes = kHalfN * kBK * 2;  // 16 KB
constexpr int kOutBytes = kBM * 64 * 2;  // one 128 x 64 bf16 output piece (16 KB), two of them
constexpr int kTmemCols = 512;

// Shared-memory plan of the two tile shapes.
template <int NACC>
struct TileCfg {
  static constexpr int kStages = NACC == 2 ? 4 : 6;
  static constexpr int kStageBytes = kABytes + NACC * kBBytes;
  static constexpr int kOutTotal = 0;
  static constexpr int kTileN = NACC * kBN;  // columns of one pair tile
  static constexpr size_t kSmemBytes =
      size_t(kStages) * kStageBytes + kOutTotal + 1024 /*align*/ + 256 /*barriers*/;
};

// Launch shape of one instantiation.
template <int MODE, int NACC>
struct KernelCfg {
  // sweeps that store a bf16 value per element: staged exponentials (MODE_LSE_E) or logit gradients (MODE_GRAD)
  static constexpr bool kWideSweep = ((MODE == 5 || MODE == 1) && NACC == 2);
  static constexpr bool kWideLse = (MODE == 0 /*MODE_LSE*/ && NACC == 2);  // online log-sum-exp, no output tile
  static constexpr bool kReduceOut = (MODE == 3 /*MODE_DW*/ && NACC == 2);  // fp32 tile added by TMA
  static constexpr int kEpiWarps = (kWideSweep || kWideLse) ? 8 : 4;
  static constexpr int kThreads = 64 + 32 * kEpiWarps;
  // bf16 output pieces staged for TMA stores: two alternating 32 x 32 pieces (2 KB each) for each
  // of the eight epilogue warps of a sweep
  // the dW tiles: two alternating 128 x 32 fp32 pieces
  static constexpr int kOutTotal =
      kWideSweep ? 4 * (kOutBytes / 2)
                 : (kReduceOut ? 2 * kOutBytes : (kWideLse ? 2048 /*sums of one group*/ : TileCfg<NACC>::kOutTotal));
  static constexpr size_t kSmemBytes = size_t(TileCfg<NACC>::kStages) * TileCfg<NACC>::kStageBytes +
                                       kOutTotal + 1024 /*align*/ + 256 /*barriers*/;
};
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kErrTimeout = -8;  // OAPL_ERR_DEVICE_TIMEOUT
constexpr int kFwdTag = 0x0A91;  // written by the loss kernel when a forward has completed

struct GemmParams {
  const int* n_live_ptr;  // device: number of live (compacted) rows; null in debug mode
  const int* tag_ptr;     // device: forward-completed tag; when set and wrong, no row is live
  const int* range_ptr;   // device: {row_begin, row_end} of this launch; null = use the two below
  int row_begin;          // first compacted row of this call's row range
  int row_cap;            // capacity of the row range (whole problem, or one chunk)
  int R, C;               // sweep schedule: R row blocks x C vocabulary splits per wave
  int d, V;
  int ldg;                // leading dimension of the staged bf16 chunk (elements)
  // sweep outputs: per (row, split) partials, kMaxSplits slots per row
  float* pm;
  float* pl;
  float* pz;
  float* ps;  // sum of exp(z - ref) * z, for the policy-entropy statistic
  // per compacted row
  const int* tgt_c;
  const int* seq_c;
  const float* lse;
  const float* zref;      // MODE_LSE_E: per-row reference subtracted before the exponential
  const float* rowscale;  // MODE_DH: optional per-row factor applied to the output
  const float* coef;      // per sequence
  const int* live_rows;
  __nv_bfloat16* dH;  // [N, d]
  float* dW;          // [V, d]
  // MODE_DEBUG
  float* Cdbg;
  int M, N, K;
  int* err;  // device status word
  // optional timing: {SM cycles, nanoseconds} of CTA 0, added up per launch (null = off)
  unsigned long long* clk;
  // Lock-step of the CTA pairs (null / 0 = off): every sync_every K-steps the pairs meet at a
  // counter in global memory, so that pairs reading the same operand slabs stay within the
  // time those slabs live in L2.  The counter must be zero at launch.
  unsigned int* sync_ctr;
  int sync_every;
  // Vocabulary sweeps with 256 x 512 tiles: the last acc_skew K-steps of a tile are issued for
  // accumulator 0 first, which is then handed to the epilogue while accumulator 1's share of those
  // K-steps still runs (0 = both accumulators complete together; at most the stage count).
  int acc_skew;
  // Limit of every pipeline wait in SM cycles (0 = kWaitCycles, about 3 s).
  long long wait_cycles;
  // MODE_DEBUG only, for the test of the give-up path: the producers of every pair leave out
  // the loads of pipeline step number test_skip_step - 1 (0 = none), so the consumers' wait
  // for that step runs out.
  int test_skip_step;
};

// Largest number of K-steps any CTA pair of this launch executes (all pairs compute the same
// value): it fixes how many lock-step meetings a pair that runs out of tiles early must still
// be counted for.
template <int MODE, int NACC>
__device__ __forceinline__ long long max_ksteps_per_pair(const GemmParams& p, int row_begin, int row_end) {
  constexpr int kTN = NACC * kBN;
  const int rows = row_end - row_begin;
  const int npairs = gridDim.x >> 1;
  if (MODE == MODE_LSE || MODE == MODE_GRAD || MODE == MODE_LSE_E) {
    if (rows <= 0) return 0;
    const int VT = (p.V + kTN - 1) / kTN;
    const int nrb = (rows + kTileM - 1) / kTileM;
    const SweepShape sh = sweep_shape(nrb, p.R, p.C, VT);
    long long tiles = (long long)sh.nfull * ((VT + p.C - 1) / p.C);
    if (sh.rem) tiles += (VT + sh.Ct - 1) / sh.Ct;
    return tiles * (p.d / kBK);
  }
  long long tiles, nk;
  if (MODE == MODE_DH) {
    if (rows <= 0) return 0;
    tiles = (long long)((rows + kTileM - 1) / kTileM) * ((p.d + kTN - 1) / kTN);
    nk = (p.V + kBK - 1) / kBK;
  } else if (MODE == MODE_DW) {
    if (rows <= 0) return 0;
    tiles = (long long)((p.V + kTileM - 1) / kTileM) * ((p.d + kTN - 1) / kTN);
    nk = (rows + kBK - 1) / kBK;
  } else {
    tiles = (long long)((p.M + kTileM - 1) / kTileM) * ((p.N + kTN - 1) / kTN);
    nk = p.K / kBK;
  }
  return ((tiles + npairs - 1) / npairs) * nk;
}

// One meeting of the lock-step: count this pair in and wait (bounded) until all pairs of the
// launch have been counted `epoch` times.  Returns false when the wait gave up: the caller then
// stops meeting (the others give up once as well); results do not depend on the meetings.
__device__ __forceinline__ bool lockstep_meet(unsigned int* ctr, unsigned int target) {
  atomicAdd(ctr, 1u);
  volatile unsigned int* v = ctr;
  if (*v >= target) return true;
  const unsigned long long t0 = global_timer_ns();
  while (*v < target) {
    if (global_timer_ns() - t0 > 200000ull) return false;  // 200 us
  }
  return true;
}

struct Tile {
  int m0, n0;    // tile origin (A's M coordinate, B's N coordinate)
  int ka0, kb0;  // K origin for the A and B tensor maps
  int nk;        // K steps of 64
  int nh;        // 256-column accumulators in use (2 only for a wide tile that is not cut by the edge)
  int first, last, split;
};

// Tile number pid + j * npairs of an MB x NB grid of 256-row tiles, NACC * 256 columns wide, handed
// out round-robin.  When the last, partial round holds r tiles and 2 r <= npairs, that round hands
// them out as 2 r half-width tiles (one accumulator each), so it takes half as long.
template <int NACC>
__device__ __forceinline__ bool grid_tile(int MB, int NB, int ncols, int pid, int npairs, int j, int& mb,
                                          int& n0, int& nh) {
  constexpr int kTN = NACC * kBN;
  const int total = MB * NB;
  const int full = (total / npairs) * npairs, r = total - full;
  const int tix = pid + j * npairs;
  if (NACC == 2 && tix >= full && r > 0 && 2 * r <= npairs) {
    const int q = tix - full;
    if (q >= 2 * r) return false;
    const int tt = full + (q >> 1);
    mb = tt / NB;
    n0 = (tt % NB) * kTN + (q & 1) * kBN;
    nh = 1;
    return n0 < ncols;
  }
  if (tix >= total) return false;
  mb = tix / NB;
  n0 = (tix % NB) * kTN;
  nh = (NACC == 2 && n0 + kBN < ncols) ? 2 : 1;
  return true;
}

// Tile j of this CTA pair for rows [row_begin, row_end) of the compacted row space.
// m0 is the pair's first row; CTA `rank` of the pair owns rows m0 + 128*rank ....
template <int MODE, int NACC>
__device__ __forceinline__ bool get_tile(const GemmParams& p, int row_begin, int row_end, int j,
                                         Tile& t) {
  constexpr int kTN = NACC * kBN;
  t.first = t.last = 1;
  t.split = 0;
  t.nh = 1;
  const int rows = row_end - row_begin;
  const int pid = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  if (MODE == MODE_LSE || MODE == MODE_GRAD || MODE == MODE_LSE_E) {
    if (rows <= 0) return false;
    const int VT = (p.V + kTN - 1) / kTN;
    const int nrb = (rows + kTileM - 1) / kTileM;
    const SweepShape sh = sweep_shape(nrb, p.R, p.C, VT);
    // complete waves: this CTA is (row block rbi, split s) of every wave
    const int rbi = pid % p.R, s = pid / p.R;
    int vt0 = (int)((long long)VT * s / p.C), vt1 = (int)((long long)VT * (s + 1) / p.C);
    int per = (s < p.C) ? vt1 - vt0 : 0;
    const int main_tiles = sh.nfull * per;
    int rbk, off;
    if (j < main_tiles) {
      const int wave = j / per;
      off = j - wave * per;
      rbk = wave * p.R + rbi;
      t.split = s;
    } else {
      // tail wave: rem row blocks x Ct splits
      if (sh.rem == 0) return false;
      const int rbt = pid % sh.rem, st = pid / sh.rem;
      if (st >= sh.Ct) return false;
      vt0 = (int)((long long)VT * st / sh.Ct);
      vt1 = (int)((long long)VT * (st + 1) / sh.Ct);
      per = vt1 - vt0;
      off = j - main_tiles;
      if (off >= per) return false;
      rbk = sh.nfull * p.R + rbt;
      t.split = st;
    }
    t.m0 = row_begin + rbk * kTileM;
    t.n0 = (vt0 + off) * kTN;
    t.nh = (NACC == 2 && t.n0 + kBN < p.V) ? 2 : 1;
    t.ka0 = t.kb0 = 0;
    t.nk = p.d / kBK;
    t.first = (off == 0);
    t.last = (off == per - 1);
    return true;
  } else if (MODE == MODE_DH) {
    if (rows <= 0) return false;
    const int MB = (rows + kTileM - 1) / kTileM, NB = (p.d + kTN - 1) / kTN;
    int mb;
    if (!grid_tile<NACC>(MB, NB, p.d, pid, npairs, j, mb, t.n0, t.nh)) return false;
    t.m0 = mb * kTileM;  // row inside the staged chunk
    t.ka0 = t.kb0 = 0;
    t.nk = (p.V + kBK - 1) / kBK;
    return true;
  } else if (MODE == MODE_DW) {
    if (rows <= 0) return false;
    const int MB = (p.V + kTileM - 1) / kTileM, NB = (p.d + kTN - 1) / kTN;
    int mb;
    if (!grid_tile<NACC>(MB, NB, p.d, pid, npairs, j, mb, t.n0, t.nh)) return false;
    t.m0 = mb * kTileM;  // vocabulary row
    t.ka0 = 0;           // staged chunk rows are range-relative
    t.kb0 = row_begin;   // compacted H rows are absolute
    t.nk = (rows + kBK - 1) / kBK;
    return true;
  } else {
    const int MB = (p.M + kTileM - 1) / kTileM, NB = (p.N + kTN - 1) / kTN;
    int mb;
    if (!grid_tile<NACC>(MB, NB, p.N, pid, npairs, j, mb, t.n0, t.nh)) return false;
    t.m0 = mb * kTileM;
    t.ka0 = t.kb0 = 0;
    t.nk = p.K / kBK;
    return true;
  }
}

// Column offset, inside a 256 x 512 tile, of 32-column chunk c of epilogue group g: the group's
// 128 columns of accumulator c / 4.
__device__ __forceinline__ int chunk_off_of(int c, int g) { return (c >> 2) * 256 + g * 128 + (c & 3) * 32; }

// Write one thread's 64 bf16 values (32 packed words) as row r of a 128 x 64 piece in the
// 128-byte-swizzled layout the TMA store expects (16-byte chunk j of row r sits at chunk
// j ^ (r & 7)); consecutive rows hit different banks.
__device__ __forceinline__ void stage_row_sw128(uint8_t* piece, int r, const uint32_t (&w)[32]) {
  uint4* rowp = reinterpret_cast<uint4*>(piece + r * 128);
#pragma unroll
  for (int jc = 0; jc < 8; ++jc)
    rowp[jc ^ (r & 7)] = make_uint4(w[4 * jc], w[4 * jc + 1], w[4 * jc + 2], w[4 * jc + 3]);
}

// The same for 32 bf16 values (16 words) as row r of a 128 x 32 piece in the 64-byte-swizzled
// layout (16-byte chunk j of row r sits at chunk j ^ ((r >> 1) & 3)).
__device__ __forceinline__ void stage_row_sw64(uint8_t* piece, int r, const uint32_t* w) {
  uint4* rowp = reinterpret_cast<uint4*>(piece + r * 64);
#pragma unroll
  for (int jc = 0; jc < 4; ++jc)
    rowp[jc ^ ((r >> 1) & 3)] = make_uint4(w[4 * jc], w[4 * jc + 1], w[4 * jc + 2], w[4 * jc + 3]);
}

// AND-reduction of a predicate over the 128 epilogue threads (named barrier 1), so that
// the decision to leave the tile loop is taken by all of them together.
template <int NTHREADS>
__device__ __forceinline__ bool epilogue_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)ok), "n"(NTHREADS)
      : "memory");
  return r != 0;
}
// Named barrier 1 over the 256 threads of the eight-warp epilogue.
__device__ __forceinline__ void epilogue_bar_all256() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

template <int MODE, int A_MN, int B_MN, int NACC>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__((KernelCfg<MODE, NACC>::kThreads), 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmC, const GemmParams p) {
  using Cfg = TileCfg<NACC>;
  using KC = KernelCfg<MODE, NACC>;
  constexpr int kStages = Cfg::kStages, kStageBytes = Cfg::kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;  // 128-byte swizzle atoms need 1024-byte alignment
  uint8_t* smem = smem_raw + (base - raw);
  uint8_t* out_smem = smem + kStages * kStageBytes;  // two 16 KB output pieces (bf16-storing modes)
  uint64_t* bars = reinterpret_cast<uint64_t*>(out_smem + KC::kOutTotal);
  const uint32_t bar0 = base + kStages * kStageBytes + KC::kOutTotal;
  // barrier slots: full[kStages], empty[kStages], tmem_full[2], tmem_empty[2].
  // NACC = 1: accumulator b = j & 1 of tile j uses tmem_full[b] / tmem_empty[b].
  // NACC = 2: tmem_full[0] covers both halves of a tile, tmem_empty[h] releases half h.
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kStages + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * kStages + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * kStages + 2 + b); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 2 * kStages + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * kStages + 5);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader of the pair
  long long clk0 = 0;
  unsigned long long ns0 = 0;
  if (p.clk && blockIdx.x == 0 && threadIdx.x == 0) {
    clk0 = clock64();
    ns0 = global_timer_ns();
  }
  int row_begin = 0, row_end = 0;
  if (MODE != MODE_DEBUG) {
    int n_live = *p.n_live_ptr;
    if (p.tag_ptr && *p.tag_ptr != kFwdTag) n_live = 0;
    if (p.range_ptr) {
      row_begin = p.range_ptr[0];
      row_end = p.range_ptr[1];
    } else {
      row_begin = p.row_begin;
      row_end = p.row_begin + p.row_cap;
    }
    if (row_end > n_live) row_end = n_live;
    // an empty row range (a range slot past the last planned range, a chunk past the live rows):
    // every thread of both CTAs sees the same bounds and leaves before any barrier, TMEM or
    // cluster set-up
    if (row_end <= row_begin) return;
  }
  const long long wlim = p.wait_cycles > 0 ? p.wait_cycles : kWaitCycles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(tfull_bar(b), 1);
      mbar_init(tempty_bar(b), 2 * KC::kEpiWarps);  // leader's copy is used: the epilogue warps of both CTAs
    }
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  if (warp == 1) tmem_alloc(smem_u32((const void*)tmem_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers exist before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      Tile t;
      bool ok = true;
      // the leader CTA's producer keeps the pair in step with the other pairs (its partner
      // follows through the shared pipeline barriers)
      bool meet = p.sync_ctr != nullptr && p.sync_every > 0 && rank == 0;
      const uint64_t pol_keep = l2_policy_evict_last();
      const uint64_t pol_stream_in = l2_policy_evict_first();
      const unsigned int npairs = gridDim.x >> 1;
      unsigned int epochs = 0;
      for (int j = 0; ok && get_tile<MODE, NACC>(p, row_begin, row_end, j, t); ++j) {
        for (int kb = 0; kb < t.nk; ++kb, ++it) {
          if (meet && it % (uint32_t)p.sync_every == 0) {
            ++epochs;
            meet = lockstep_meet(p.sync_ctr, epochs * npairs);
          }
          if (MODE == MODE_DEBUG && p.test_skip_step && it + 1 == (uint32_t)p.test_skip_step) continue;
          const int s = it % kStages;
          if (!mbar_wait(empty_bar(s), ((it / kStages) & 1u) ^ 1u, abort_flag, wlim)) {
            ok = false;
            break;
          }
          const uint32_t sa = base + s * kStageBytes;
          // the leader's barrier collects the bytes of both CTAs' loads
          const uint32_t fb = mapa_shared(full_bar(s), 0);
          if (rank == 0) mbar_expect_tx(full_bar(s), 2 * (kABytes + t.nh * kBBytes));
          const int ka = t.ka0 + kb * kBK, kbb = t.kb0 + kb * kBK;
          const int am = t.m0 + (int)rank * kBM;
          if (A_MN) {
#pragma unroll
            for (int b = 0; b < kBM / 64; ++b) tma_load_2d(sa + b * 8192, &tmA, fb, am + 64 * b, ka);
          } else if (KC::kWideSweep || KC::kWideLse) {
            // the pair's H block is read again for every vocabulary tile: keep it in L2
            tma_load_2d_hint(sa, &tmA, fb, ka, am, pol_keep);
          } else {
            tma_load_2d(sa, &tmA, fb, ka, am);
          }
#pragma unroll
          for (int h = 0; h < NACC; ++h) {
            if (h < t.nh) {
              // this CTA's 128 of the 256 columns of accumulator h
              const uint32_t sb = sa + kABytes + h * kBBytes;
              const int bn = t.n0 + h * kBN + (int)rank * kHalfN;
              if (B_MN) {
#pragma unroll
                for (int b = 0; b < kHalfN / 64; ++b)
                  tma_load_2d(sb + b * 8192, &tmB, fb, bn + 64 * b, kbb);
              } else if (KC::kWideSweep || KC::kWideLse) {
                // W streams through once per wave: it should not push the H blocks out of L2
                tma_load_2d_hint(sb, &tmB, fb, kbb, bn, pol_stream_in);
              } else {
                tma_load_2d(sb, &tmB, fb, kbb, bn);
              }
            }
          }
        }
      }
      if (meet) {
        // out of tiles: be counted for the meetings the longest-running pair still holds
        const long long mx = max_ksteps_per_pair<MODE, NACC>(p, row_begin, row_end);
        const long long total = (mx + p.sync_every - 1) / p.sync_every;
        if (total > (long long)epochs) atomicAdd(p.sync_ctr, (unsigned int)(total - epochs));
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ UMMA issuer (leader CTA only)
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(kTileM, kBN, A_MN, B_MN);
      uint32_t it = 0;
      Tile t;
      bool ok = true;
      for (int j = 0; ok && get_tile<MODE, NACC>(p, row_begin, row_end, j, t); ++j) {
        uint32_t d_tmem;
        if (NACC == 1) {
          const int buf = j & 1;
          if (!mbar_wait(tempty_bar(buf), ((j >> 1) & 1u) ^ 1u, abort_flag, wlim)) break;
          d_tmem = tmem_base + buf * kBN;
        } else {
          d_tmem = tmem_base;
        }
        int kb_start = 0;
        if (NACC == 2) {
          // Accumulator 0 is released by the epilogue before accumulator 1: start with
          // accumulator 0's UMMAs of the first `pre` K-steps (their stages are already loaded),
          // then wait for accumulator 1 and catch up on the same stages.
          const int pre = t.nk < kStages ? t.nk : kStages;
          if (!mbar_wait(tempty_bar(0), (j & 1u) ^ 1u, abort_flag, wlim)) break;
          tc_fence_after();
          for (int kb = 0; ok && kb < pre; ++kb) {
            const uint32_t itk = it + kb;
            const int s = itk % kStages;
            if (!mbar_wait(full_bar(s), (itk / kStages) & 1u, abort_flag, wlim)) {
              ok = false;
              break;
            }
            tc_fence_after();
            const uint32_t sa = base + s * kStageBytes, sb = sa + kABytes;
#pragma unroll
            for (int kk = 0; kk < kBK / 16; ++kk) {
              const uint64_t da = A_MN ? smem_desc_sw128(sa + kk * 2048, 8192, 1024)
                                       : smem_desc_sw128(sa + kk * 32, 16, 1024);
              const uint64_t db = B_MN ? smem_desc_sw128(sb + kk * 2048, 8192, 1024)
                                       : smem_desc_sw128(sb + kk * 32, 16, 1024);
              umma_bf16(d_tmem, da, db, idesc, (kb | kk) ? 1u : 0u);
            }
            if (t.nh == 1) umma_commit_pair(empty_bar(s));
          }
          if (!ok) break;
          if (!mbar_wait(tempty_bar(1), (j & 1u) ^ 1u, abort_flag, wlim)) break;
          tc_fence_after();
          if (t.nh == 2) {
            for (int kb = 0; kb < pre; ++kb) {
              const int s = (it + kb) % kStages;
              const uint32_t sa = base + s * kStageBytes, sb = sa + kABytes + kBBytes;
#pragma unroll
              for (int kk = 0; kk < kBK / 16; ++kk) {
                const uint64_t da = A_MN ? smem_desc_sw128(sa + kk * 2048, 8192, 1024)
                                         : smem_desc_sw128(sa + kk * 32, 16, 1024);
                const uint64_t db = B_MN ? smem_desc_sw128(sb + kk * 2048, 8192, 1024)
                                         : smem_desc_sw128(sb + kk * 32, 16, 1024);
                umma_bf16(d_tmem + kBN, da, db, idesc, (kb | kk) ? 1u : 0u);
              }
              umma_commit_pair(empty_bar(s));  // both accumulators' UMMAs have read the stage
            }
          }
          it += pre;
          kb_start = pre;
        } else {
          tc_fence_after();
        }
        // the last `post` K-steps of a sweep tile: accumulator 0 first (see GemmParams::acc_skew)
        int post = 0;
        if (NACC == 2 && (KC::kWideSweep || KC::kWideLse) && t.nh == 2) {
          post = p.acc_skew < kStages ? p.acc_skew : kStages;
          if (post > t.nk - kb_start) post = t.nk - kb_start;
          if (post < 0) post = 0;
        }
        const int kb_end = t.nk - post;
        for (int kb = kb_start; kb < kb_end; ++kb, ++it) {
          const int s = it % kStages;
          if (!mbar_wait(full_bar(s), (it / kStages) & 1u, abort_flag, wlim)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t sa = base + s * kStageBytes;
#pragma unroll
          for (int kk = 0; kk < kBK / 16; ++kk) {
            const uint64_t da = A_MN ? smem_desc_sw128(sa + kk * 2048, 8192, 1024)
                                     : smem_desc_sw128(sa + kk * 32, 16, 1024);
#pragma unroll
            for (int h = 0; h < NACC; ++h) {
              if (h < t.nh) {
                const uint32_t sb = sa + kABytes + h * kBBytes;
                const uint64_t db = B_MN ? smem_desc_sw128(sb + kk * 2048, 8192, 1024)
                                         : smem_desc_sw128(sb + kk * 32, 16, 1024);
                umma_bf16(d_tmem + h * kBN, da, db, idesc, (kb | kk) ? 1u : 0u);
              }
            }
          }
          umma_commit_pair(empty_bar(s));  // both CTAs' stage reusable once these UMMAs have read it
        }
        if (!ok) break;
        if (NACC == 2 && post > 0) {
          for (int q = 0; ok && q < post; ++q) {
            const uint32_t itk = it + q;
            const int s = itk % kStages;
            if (!mbar_wait(full_bar(s), (itk / kStages) & 1u, abort_flag, wlim)) {
              ok = false;
              break;
            }
            tc_fence_after();
            const uint32_t sa = base + s * kStageBytes, sb = sa + kABytes;
#pragma unroll
            for (int kk = 0; kk < kBK / 16; ++kk)
              umma_bf16(d_tmem, smem_desc_sw128(sa + kk * 32, 16, 1024), smem_desc_sw128(sb + kk * 32, 16, 1024),
                        idesc, 1u);
          }
          if (!ok) break;
          umma_commit_pair(tfull_bar(0));  // accumulator 0 complete in both CTAs
          for (int q = 0; q < post; ++q) {
            const int s = (it + q) % kStages;
            const uint32_t sa = base + s * kStageBytes, sb = sa + kABytes + kBBytes;
#pragma unroll
            for (int kk = 0; kk < kBK / 16; ++kk)
              umma_bf16(d_tmem + kBN, smem_desc_sw128(sa + kk * 32, 16, 1024),
                        smem_desc_sw128(sb + kk * 32, 16, 1024), idesc, 1u);
            umma_commit_pair(empty_bar(s));
          }
          it += post;
          umma_commit_pair(tfull_bar(1));  // accumulator 1 complete
        } else if (NACC == 2 && (KC::kWideSweep || KC::kWideLse)) {
          umma_commit_pair(tfull_bar(0));
          umma_commit_pair(tfull_bar(1));
        } else {
          // accumulator(s) complete in both CTAs
          umma_commit_pair(tfull_bar(NACC == 1 ? (j & 1) : 0));
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int quad = warp & 3;  // TMEM lanes [32*quad, 32*quad+32)
    const int r_in_tile = quad * 32 + lane;
    // eight-warp epilogue: warps 2..5 are group 0, warps 6..9 group 1; each group takes half of
    // an accumulator's columns (four-warp epilogue: one group)
    const int group = (warp - 2) >> 2;
    const bool issuer = ((warp - 2) & 3) == 0 && lane == 0;  // issues its group's TMA stores
    // running state of this thread's row across the tiles of a sweep
    float run_m2 = -INFINITY, run_l = 0.f, run_z = 0.f, run_s = 0.f;
    Tile t;
    for (int j = 0; get_tile<MODE, NACC>(p, row_begin, row_end, j, t); ++j) {
      const int buf = NACC == 1 ? (j & 1) : 0;
      // MODE_LSE/GRAD/LSE_E: compacted row; DH: row inside the staged chunk; DW: vocabulary row
      const int row = t.m0 + (int)rank * kBM + r_in_tile;
      int tgt = -1;
      float cf = 0.f, ref2 = 0.f;
      bool valid = true;
      if (MODE == MODE_LSE || MODE == MODE_LSE_E) {
        valid = row < row_end;
        tgt = valid ? p.tgt_c[row] : -1;
        if (MODE == MODE_LSE_E && valid) ref2 = p.zref[row] * kLog2e;
        if (t.first) { run_m2 = -INFINITY; run_l = 0.f; run_z = 0.f; run_s = 0.f; }
      } else if (MODE == MODE_GRAD) {
        valid = row < row_end;
        if (valid) {
          tgt = p.tgt_c[row];
          cf = p.coef[p.seq_c[row]];
          ref2 = p.lse[row] * kLog2e;
        }
      }
      const bool got = mbar_wait(tfull_bar(buf), (NACC == 1 ? (j >> 1) : j) & 1u, abort_flag, wlim);
      if (!epilogue_all<32 * KC::kEpiWarps>(got)) break;
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t(quad * 32) << 16) + buf * kBN;

      if (KC::kWideLse) {
        // Online log-sum-exp over this group's 128 columns of each accumulator, 32 at a time with
        // the next 32 already on their way from TMEM; nothing is stored per element.
        const int nchunks = 4 * t.nh;
        auto lse_chunk = [&](const uint32_t (&r)[32], int c) {
          const int col0 = t.n0 + chunk_off_of(c, group);
          if (!valid || col0 >= p.V) return;
          float v[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
          if (col0 + 32 > p.V) {
            // a large finite negative: its exponential is 0 and 0 * v stays 0 (no NaN)
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (col0 + i >= p.V) v[i] = -3.0e38f;
          }
          float cmax = v[0];
#pragma unroll
          for (int i = 1; i < 32; ++i) cmax = fmaxf(cmax, v[i]);
          const float m2 = fmaxf(run_m2, cmax * kLog2e);
          float acc = 0.f, accs = 0.f;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float e = ex2_approx(fmaf(v[i], kLog2e, -m2));
            acc += e;
            accs = fmaf(e, v[i], accs);
          }
          const float resc = ex2_approx(run_m2 - m2);
          run_l = run_l * resc + acc;
          run_s = run_s * resc + accs;
          run_m2 = m2;
          const int ti = tgt - col0;
          if (ti >= 0 && ti < 32) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i == ti) run_z = v[i];
          }
        };
        // all of this warp's 128 columns of an accumulator go to registers first, so the
        // accumulator is handed back to the UMMA warp before the exponentials are taken
        uint32_t rr[4][32];
        (void)nchunks;
        bool dead = false;
#pragma unroll 1
        for (int h = 0; h < t.nh; ++h) {
          if (h == 1) {
            // accumulator 1 may complete later than accumulator 0 (GemmParams::acc_skew)
            const bool got1 = mbar_wait(tfull_bar(1), j & 1u, abort_flag, wlim);
            if (!epilogue_all<32 * KC::kEpiWarps>(got1)) {
              dead = true;
              break;
            }
            tc_fence_after();
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) tmem_ld32(taddr + chunk_off_of(4 * h + q, group), rr[q]);
          tmem_ld_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar(h), 0));
#pragma unroll
          for (int q = 0; q < 4; ++q) lse_chunk(rr[q], 4 * h + q);
        }
        if (dead) break;
        if (t.nh == 1) {
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar(1), 0));
        }
        if (t.last) {
          // end of this row block's sweep: merge the two groups' (max, sum-exp, sum exp*z, target logit)
          float* xch = reinterpret_cast<float*>(out_smem);
          if (group == 1) {
            xch[r_in_tile * 4 + 0] = run_m2;
            xch[r_in_tile * 4 + 1] = run_l;
            xch[r_in_tile * 4 + 2] = run_s;
            xch[r_in_tile * 4 + 3] = run_z;
          }
          epilogue_bar_all256();
          if (group == 0 && valid) {
            const float m1 = xch[r_in_tile * 4 + 0];
            const float M = fmaxf(run_m2, m1);
            const float w0 = ex2_approx(run_m2 - M), w1 = ex2_approx(m1 - M);
            const size_t o = (size_t)row * kMaxSplits + t.split;
            p.pm[o] = M * kLn2;  // back to natural units
            p.pl[o] = run_l * w0 + xch[r_in_tile * 4 + 1] * w1;
            p.ps[o] = run_s * w0 + xch[r_in_tile * 4 + 2] * w1;
            p.pz[o] = run_z + xch[r_in_tile * 4 + 3];
          }
          epilogue_bar_all256();  // the exchange buffer may be written again
        }
      } else if (KC::kWideSweep) {
        // This group's 128 columns of each accumulator, 32 at a time with the next 32 already
        // on their way from TMEM: exp, sums, bf16.  Every warp sends its own 32 rows x 32 columns
        // through one of its two swizzled 2 KB pieces in shared memory and a TMA store of its own
        // (tmC has 32 x 32 boxes), so the stores need no barrier between warps.  An accumulator
        // is handed back to the UMMA warp as soon as this warp's last load from it has landed.
        constexpr int kWarpPiece = 32 * 64;  // 32 rows of 32 bf16
        uint8_t* const my_pieces = out_smem + (warp - 2) * (2 * kWarpPiece);
        const uint64_t pol_stream = l2_policy_evict_first();
        const int nchunks = 4 * t.nh;
        auto send_chunk = [&](int c, const uint32_t* w16) {
          uint8_t* piece = my_pieces + (c & 1) * kWarpPiece;
          // lane 0 issues this warp's stores: the one two pieces back has drained this buffer
          if (lane == 0) tma_store_wait_read<1>();
          __syncwarp();
          stage_row_sw64(piece, lane, w16);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            // the staged values are not read again before the whole range is written
            tma_store_2d_hint(&tmC, smem_u32(piece), t.n0 + chunk_off_of(c, group),
                              t.m0 - row_begin + (int)rank * kBM + quad * 32, pol_stream);
            tma_store_commit();
          }
        };
        auto chunk_off = [&](int c) { return chunk_off_of(c, group); };
        // exp / sums / packing of one 32-column chunk into 16 words of w
        auto do_chunk = [&](const uint32_t (&r)[32], int c, uint32_t* w16) {
          const int col0 = t.n0 + chunk_off(c);
          if (MODE == MODE_GRAD) {
            // g = c * (onehot - exp(z - lse)); columns past V and rows past the range are 0
            if (valid && col0 < p.V) {
              const int ti = tgt - col0;
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                float g0 = -cf * ex2_approx(fmaf(__uint_as_float(r[i]), kLog2e, -ref2));
                float g1 = -cf * ex2_approx(fmaf(__uint_as_float(r[i + 1]), kLog2e, -ref2));
                if (i == ti) g0 += cf;
                if (i + 1 == ti) g1 += cf;
                if (col0 + i >= p.V) g0 = 0.f;
                if (col0 + i + 1 >= p.V) g1 = 0.f;
                w16[i >> 1] = pack_bf16x2(g0, g1);
              }
            } else {
#pragma unroll
              for (int i = 0; i < 16; ++i) w16[i] = 0u;
            }
            return;
          }
          if (valid && col0 < p.V) {
            const int ti = tgt - col0;
            float acc = 0.f, accs = 0.f;
            if (col0 + 32 <= p.V) {
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const float z0 = __uint_as_float(r[i]), z1 = __uint_as_float(r[i + 1]);
                const float e0 = ex2_approx(fmaf(z0, kLog2e, -ref2));
                const float e1 = ex2_approx(fmaf(z1, kLog2e, -ref2));
                acc += e0 + e1;
                accs = fmaf(e0, z0, fmaf(e1, z1, accs));
                w16[i >> 1] = pack_bf16x2(e0, e1);
              }
            } else {
              // the vocabulary ends inside these 32 columns: columns past V hold z = 0
              // (zero-filled W rows) and their e is cleared
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const float z0 = __uint_as_float(r[i]), z1 = __uint_as_float(r[i + 1]);
                float e0 = ex2_approx(fmaf(z0, kLog2e, -ref2));
                float e1 = ex2_approx(fmaf(z1, kLog2e, -ref2));
                if (col0 + i >= p.V) e0 = 0.f;
                if (col0 + i + 1 >= p.V) e1 = 0.f;
                acc += e0 + e1;
                accs = fmaf(e0, z0, fmaf(e1, z1, accs));
                w16[i >> 1] = pack_bf16x2(e0, e1);
              }
            }
            run_l += acc;
            run_s += accs;
            if (ti >= 0 && ti < 32) {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (i == ti) run_z = __uint_as_float(r[i]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) w16[i] = 0u;
          }
        };
        // All of this warp's 128 columns of an accumulator go to registers first, so the
        // accumulator is handed back to the UMMA warp before the exponentials are taken.
        uint32_t rr[4][32], w[16];
        (void)nchunks;
        bool dead = false;
#pragma unroll 1
        for (int h = 0; h < t.nh; ++h) {
          if (h == 1) {
            // accumulator 1 may complete later than accumulator 0 (GemmParams::acc_skew)
            const bool got1 = mbar_wait(tfull_bar(1), j & 1u, abort_flag, wlim);
            if (!epilogue_all<32 * KC::kEpiWarps>(got1)) {
              dead = true;
              break;
            }
            tc_fence_after();
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) tmem_ld32(taddr + chunk_off(4 * h + q), rr[q]);
          tmem_ld_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar(h), 0));
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            do_chunk(rr[q], 4 * h + q, w);
            send_chunk(4 * h + q, w);
          }
        }
        if (dead) break;
        if (t.nh == 1) {
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar(1), 0));
        }
        if (MODE == MODE_LSE_E && t.last) {
          // end of this row block's sweep: every warp of group 1 hands its rows' sums to the warp
          // of group 0 that holds the same rows (four warps on), through its own first piece
          float* xch = reinterpret_cast<float*>(out_smem + ((warp - 2) | 4) * (2 * kWarpPiece)) + lane * 4;
          if (group == 1) {
            if (lane == 0) tma_store_wait_read<0>();
            __syncwarp();
            xch[0] = run_l;
            xch[1] = run_z;
            xch[2] = run_s;
          }
          epilogue_bar_all256();
          if (group == 0 && valid) {
            const size_t o = (size_t)row * kMaxSplits + t.split;
            p.pl[o] = run_l + xch[0];
            p.pz[o] = run_z + xch[1];
            p.ps[o] = run_s + xch[2];
          }
          epilogue_bar_all256();  // group 1 may stage into its pieces again
        }
      } else if (KC::kReduceOut) {
        // dW += tile: 32 fp32 columns at a time through one of two swizzled 128 x 32 pieces in
        // shared memory and a TMA reduce-add (tmC maps dW), so the old values never travel to
        // the SM.  Every element of dW belongs to one tile of the launch and launches follow
        // one another on the stream, so the sums are formed in a fixed order.  Rows past V and
        // columns past d are clipped by the tensor map.
        const int nchunks = t.nh * (kBN / 32);
        uint32_t ra[32], rb[32];
        // one barrier per piece: before it the issuing thread has seen every earlier reduce
        // finish reading shared memory, so the other buffer may be overwritten next time
        auto send32 = [&](int c, const uint32_t (&r)[32]) {
          uint8_t* piece = out_smem + (c & 1) * kOutBytes;
          stage_row_sw128(piece, r_in_tile, r);
          fence_proxy_async_smem();
          if (issuer) tma_store_wait_read<0>();
          epilogue_bar_sync();
          if (issuer) {
            if (t.n0 + c * 32 < p.d && t.m0 + (int)rank * kBM < p.V)  // box not wholly outside
              tma_reduce_add_2d(&tmC, smem_u32(piece), t.n0 + c * 32, t.m0 + (int)rank * kBM);
            tma_store_commit();
          }
        };
        tmem_ld32(taddr, ra);
#pragma unroll 1
        for (int c = 0; c < nchunks; c += 2) {
          tmem_ld_wait();
          tmem_ld32(taddr + (c + 1) * 32, rb);
          send32(c, ra);
          tmem_ld_wait();
          if (c + 2 < nchunks) tmem_ld32(taddr + (c + 2) * 32, ra);
          if (c + 1 == kBN / 32 - 1 || c + 1 == 2 * (kBN / 32) - 1) {
            // this warp's last load from accumulator (c + 1) / 8 has landed
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar((c + 1) / (kBN / 32)), 0));
          }
          send32(c + 1, rb);
        }
        if (t.nh == 1) {
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar(1), 0));
        }
      } else {
        // dH and the bring-up GEMM: 32 columns at a time, stored straight from registers
#pragma unroll 1
        for (int c = 0; c < t.nh * (kBN / 32); ++c) {
          uint32_t r[32];
          tmem_ld32(taddr + c * 32, r);
          tmem_ld_wait();
          const int col0 = t.n0 + c * 32;
          if (NACC == 2 && c == kBN / 32) {
            // first half drained: the next tile's UMMAs may overwrite it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(tempty_bar(0), 0));
          }
          if (MODE == MODE_DH) {
            const int crow = row_begin + row;
            if (crow < row_end && col0 < p.d) {
              const float sc = p.rowscale ? p.rowscale[crow] : 1.f;
              uint32_t o[16];
#pragma unroll
              for (int i = 0; i < 32; i += 2)
                o[i >> 1] = pack_bf16x2(sc * __uint_as_float(r[i]), sc * __uint_as_float(r[i + 1]));
              uint4* dst = reinterpret_cast<uint4*>(p.dH + (size_t)p.live_rows[crow] * p.d + col0);
#pragma unroll
              for (int q = 0; q < 4; ++q)
                dst[q] = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
            }
          } else {
            if (row < p.M && col0 < p.N) {  // N is a multiple of 8
              float4* dst = reinterpret_cast<float4*>(p.Cdbg + (size_t)row * p.N + col0);
#pragma unroll
              for (int q = 0; q < 8; ++q)
                if (col0 + 4 * q < p.N)
                  dst[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]),
                                       __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
            }
          }
        }
        // accumulator drained: hand the TMEM buffer back to the UMMA warp
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (NACC == 1) {
            mbar_arrive_cluster(mapa_shared(tempty_bar(buf), 0));
          } else {
            if (t.nh == 1) mbar_arrive_cluster(mapa_shared(tempty_bar(0), 0));
            mbar_arrive_cluster(mapa_shared(tempty_bar(1), 0));
          }
        }
      }
    }
    // whoever issued bulk stores or reductions waits for them before the CTA may exit
    if ((KC::kWideSweep && lane == 0) || (KC::kReduceOut && issuer)) tma_store_wait_all();
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      if (p.err) atomicCAS(p.err, 0, kErrTimeout);
      const long long t0 = clock64();  // let loads already in flight land before smem is released
      while (clock64() - t0 < 2000000LL) {
      }
    }
    __syncthreads();
  }
  // neither CTA may release its TMEM or shared memory while the other can still touch them
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  if (p.clk && blockIdx.x == 0 && threadIdx.x == 0) {
    atomicAdd(p.clk, (unsigned long long)(clock64() - clk0));
    atomicAdd(p.clk + 1, global_timer_ns() - ns0);
  }
}

}  // namespace oapl
