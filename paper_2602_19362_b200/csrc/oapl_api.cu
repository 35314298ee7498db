// Host side of the C ABI declared in include/oapl.h: argument validation, the
// workspace carve-up, tensor-map encoding and the launch sequences.
#include <cuda.h>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "../../include/oapl.h"
#include "adamw.cuh"
#include "gemm_sm100.cuh"
#include "small_kernels.cuh"

namespace oapl {

static std::atomic<uint64_t> g_launches{0};
#define OAPL_LAUNCHED() (g_launches.fetch_add(1, std::memory_order_relaxed))

// rows of one g chunk of the two-call backward: 74 row blocks of 256, so that on 74 CTA pairs the
// chunk's dH tiles (74 x d/512) fill whole rounds and its sweep two whole waves of 37 row blocks
constexpr int kChunkRowsDefault = 74 * 256;
// rows of staged e = exp(z - zref) per range in the single-call path (20 GB at V = 152064): the longer
// the ranges, the fewer partial rounds of dH tiles, passes over dW and tail waves of the sweep
constexpr int kStageRowsDefault = 65536;
constexpr int kSyncSlots = 4096;             // lock-step counters in the workspace, one per contraction launch
constexpr int kMaxDevices = 64;              // per-device host-side caches

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Carve {
  size_t state, sync, block_cnt, block_off, live_rows, tgt_c, seq_c, q_c, lp_c, lse, ent_c, pm, pl, pz, ps, cstart,
      cend, seq_D, coef, vhat, seq_logp, Hc, G, zref, alpha, ztc, rowscale, Hs, ranges, coef_row, qo_c,
      seq_obj, seq_clip, total;
  int n_pad, nblk, chunk_rows, ldg;
  int stage_rows, stage_alloc_rows, max_ranges;  // single-call path only
};

static int env_int(const char* name, int dflt) {
  const char* s = getenv(name);
  return (s && *s) ? atoi(s) : dflt;
}

// Named ranges for a timeline profiler around the phases a call enqueues (OAPL_NVTX=1; off by
// default).  They mark host-side enqueue spans; the profiler attributes the launches inside.
struct NvtxRange {
  bool on;
  explicit NvtxRange(const char* name) : on(env_int("OAPL_NVTX", 0) != 0) {
    if (on) nvtxRangePushA(name);
  }
  ~NvtxRange() {
    if (on) nvtxRangePop();
  }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};

static bool carve(const oapl_problem* p, int flags, Carve* c) {
  if (!p || p->N <= 0 || p->d <= 0 || p->V <= 0 || p->S <= 0 || p->P <= 0) return false;
  if (p->d % 64 != 0) return false;
  if (p->N > (int64_t)2000000000 || (int64_t)p->V + 512 > (int64_t)2000000000) return false;
  const size_t n_pad = align_up((size_t)p->N, 256);
  c->n_pad = (int)n_pad;
  c->nblk = (int)((p->N + kScanBlock - 1) / kScanBlock);
  int chunk = env_int("OAPL_CHUNK_ROWS", kChunkRowsDefault);
  chunk = (int)align_up((size_t)(chunk < 256 ? 256 : chunk), 256);
  if ((size_t)chunk > n_pad) chunk = (int)n_pad;
  c->chunk_rows = chunk;
  c->ldg = (int)align_up((size_t)p->V, 512);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off = align_up(off + bytes, 1024);
    return o;
  };
  c->state = take(sizeof(DevState));
  c->sync = take(4 * (size_t)kSyncSlots);
  c->block_cnt = take(4 * (size_t)c->nblk);
  c->block_off = take(4 * (size_t)c->nblk);
  c->live_rows = take(4 * n_pad);
  c->tgt_c = take(4 * n_pad);
  c->seq_c = take(4 * n_pad);
  c->q_c = take(4 * n_pad);
  c->lp_c = take(4 * n_pad);
  c->lse = take(4 * n_pad);
  c->ent_c = take(4 * n_pad);
  c->pm = take(4 * n_pad * kMaxSplits);
  c->pl = take(4 * n_pad * kMaxSplits);
  c->pz = take(4 * n_pad * kMaxSplits);
  c->ps = take(4 * n_pad * kMaxSplits);
  c->cstart = take(4 * (size_t)p->S);
  c->cend = take(4 * (size_t)p->S);
  c->seq_D = take(4 * (size_t)p->S);
  c->coef = take(4 * (size_t)p->S);
  c->vhat = take(4 * (size_t)p->P);
  c->seq_logp = take(4 * (size_t)p->S);
  c->Hc = take(2 * n_pad * (size_t)p->d);
  c->stage_rows = c->stage_alloc_rows = c->max_ranges = 0;
  if (flags & OAPL_FLAG_FUSED) {
    // the chunk region holds e for a range of whole sequences instead of a row chunk of g
    int stage = env_int("OAPL_STAGE_ROWS", kStageRowsDefault);
    stage = (int)align_up((size_t)(stage < 256 ? 256 : stage), 256);
    if ((size_t)stage > n_pad) stage = (int)n_pad;
    c->stage_rows = stage;
    c->stage_alloc_rows = stage + 256;
    // greedy packing of whole sequences: two neighbouring ranges together always hold more than
    // `stage` rows, and every range holds at least one sequence
    {
      const size_t by_rows = 2 * ((n_pad + (size_t)stage - 1) / (size_t)stage) - 1;
      c->max_ranges = (int)(by_rows < (size_t)p->S ? by_rows : (size_t)p->S);
      if (c->max_ranges < 1) c->max_ranges = 1;
    }
    c->G = take(2 * (size_t)c->stage_alloc_rows * (size_t)c->ldg);
    c->zref = take(4 * n_pad);
    c->alpha = take(4 * n_pad);
    c->ztc = take(4 * n_pad);
    c->rowscale = take(4 * n_pad);
    c->Hs = take(2 * (n_pad + 256) * (size_t)p->d);
    c->ranges = take(sizeof(RangeRec) * (size_t)c->max_ranges);
    c->coef_row = take(4 * n_pad);
    c->qo_c = take(4 * n_pad);
    c->seq_obj = take(4 * (size_t)p->S);
    c->seq_clip = take(4 * (size_t)p->S);
  } else {
    c->G = take(2 * (size_t)chunk * (size_t)c->ldg);
    c->zref = c->alpha = c->ztc = c->rowscale = c->Hs = c->ranges = 0;
    c->coef_row = c->qo_c = c->seq_obj = c->seq_clip = 0;
  }
  c->total = off;
  return true;
}

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 matrix [rows, cols] row-major with leading dimension ld (elements); the box
// is box_cols (= 64 elements = one 128-byte swizzle row) by box_rows.
static bool make_map(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                     uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {ld * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same matrix seen through 32-row x 32-column boxes (64-byte rows, 64-byte swizzle): the
// store map of the sweeps that write a bf16 value per element (one box per epilogue warp).
static bool make_map_store32(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint64_t ld) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {ld * 2};
  const cuuint32_t box[2] = {32, 32};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 matrix [rows, cols] row-major seen through 128-row x 32-column boxes (128-byte rows,
// 128-byte swizzle): the reduce-add map of the dW contraction.
static bool make_map_f32(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint64_t ld) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {ld * 4};
  const cuuint32_t box[2] = {32, 128};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int sm_count() {
  static int n[kMaxDevices] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
  if (!n[dev] && cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n[dev] = 0;
  return n[dev];
}

// Sweep schedule: a wave is R row blocks (256 rows, one CTA pair each) x C vocabulary
// splits, R*C <= number of CTA pairs.  C is the smallest power of two that keeps the wave's
// H row blocks within an L2 budget; a short row range is handled by the tail-wave
// re-splitting of the schedule itself.
// The budget: every H block is re-read by its C pairs for each vocabulary tile and has to stay
// in L2 for a whole sweep.  DRAM counters of the sweep on 32 k rows at d = 3584: with 68 MB of
// blocks, each read by two pairs (R = 37, C = 2), half of the re-reads went to DRAM (22 GB read
// against 4 GB needed); the same 68 MB read by one pair per block stayed resident (5.9 GB); 33 MB
// read by four pairs each (R = 18, C = 4) stayed resident too (10 GB against 8).  So blocks with
// several readers get about half of the 126 MB L2.
constexpr int kL2BudgetMB = 48;
static void pick_sweep(int n_sm, int d, int vtiles, int* R, int* C) {
  const int pairs = n_sm / 2;
  int c = env_int("OAPL_SPLITS", 0);
  if (c <= 0) {
    c = 1;
    const size_t budget = (size_t)env_int("OAPL_L2_BUDGET_MB", kL2BudgetMB) << 20;
    while (c < kMaxSplits && (size_t)(pairs / c) * kSweepRows * d * 2 > budget) c *= 2;
  }
  if (c > kMaxSplits) c = kMaxSplits;
  while (c > 1 && c > vtiles) c /= 2;
  int r = pairs / c;
  if (r < 1) r = 1;
  *R = r;
  *C = c;
}

// Lock-step meetings of the CTA pairs of one contraction launch (see GemmParams::sync_ctr):
// counter number `slot` of the workspace, which the caller has zeroed; every `nk_tile`-aligned
// 32 K-steps or so.  OAPL_SYNC_EVERY overrides the interval (0 switches the meetings off).
static void set_lockstep(GemmParams* gp, uint8_t* ws, const Carve& c, int slot, int nk_tile) {
  const int forced = env_int("OAPL_SYNC_EVERY", -1);
  gp->sync_ctr = nullptr;
  gp->sync_every = 0;
  if (forced == 0 || slot < 0 || slot >= kSyncSlots) return;
  int every = forced > 0 ? forced : 32;
  if (nk_tile > 0) every = ((every + nk_tile - 1) / nk_tile) * nk_tile;  // whole tiles of a sweep
  gp->sync_ctr = reinterpret_cast<unsigned int*>(ws + c.sync) + slot;
  gp->sync_every = every;
}

// Optional per-contraction timing (off by default): an event pair around every contraction
// launch on the device the timing was enabled on, summed per kind by oapl_profile_read.
// Launches on any other device run untimed.  Event pairs are created as they are needed, up
// to kProfMaxPairs between two reads; launches beyond that are counted as dropped.
constexpr int kProfMaxPairs = 1 << 16;
constexpr int kProfKinds = 8;
struct ProfPair {
  cudaEvent_t ev[2];
  int kind;
};
struct ProfState {
  int device = -1;               // device the timing is enabled on (-1 = off)
  std::vector<ProfPair> pairs;   // pairs created so far (events belong to `made_on`)
  int made_on = -1;
  int used = 0;                  // pairs in use since the last read
  int dropped = 0;               // launches not recorded since the last read
  unsigned long long* clk_addr = nullptr;  // device address of g_prof_clk on `device`
};
static ProfState g_prof;

// {SM cycles, nanoseconds} of CTA 0 of every contraction launch, summed per kind while
// the timing is enabled; their ratio is the SM clock the kind ran at.
static __device__ unsigned long long g_prof_clk[kProfKinds][2];

// Pure host logic of "is this launch timed": only on the device the timing was enabled on.
static inline bool prof_applies(int enabled_device, int current_device) {
  return enabled_device >= 0 && enabled_device == current_device;
}

static int prof_begin(int kind, int dev, cudaStream_t st) {
  if (!prof_applies(g_prof.device, dev)) return -1;
  if (g_prof.used >= (int)g_prof.pairs.size()) {
    if ((int)g_prof.pairs.size() >= kProfMaxPairs) {
      ++g_prof.dropped;
      return -1;
    }
    ProfPair pr;
    if (cudaEventCreate(&pr.ev[0]) != cudaSuccess) { ++g_prof.dropped; return -1; }
    if (cudaEventCreate(&pr.ev[1]) != cudaSuccess) { cudaEventDestroy(pr.ev[0]); ++g_prof.dropped; return -1; }
    pr.kind = 0;
    g_prof.pairs.push_back(pr);
  }
  const int s = g_prof.used++;
  g_prof.pairs[s].kind = kind;
  cudaEventRecord(g_prof.pairs[s].ev[0], st);
  return s;
}
static void prof_end(int slot, cudaStream_t st) {
  if (slot >= 0) cudaEventRecord(g_prof.pairs[slot].ev[1], st);
}

template <int MODE, int A_MN, int B_MN, int NACC = 1>
static int launch_gemm(const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& c,
                       const GemmParams& gp_in, int grid, cudaStream_t st) {
  GemmParams gp = gp_in;
  gp.acc_skew = env_int("OAPL_ACC_SKEW", TileCfg<NACC>::kStages);
  static bool attr_set[kMaxDevices] = {false};  // the attribute belongs to the function on one device
  auto kern = gemm_kernel<MODE, A_MN, B_MN, NACC>;
  constexpr size_t smem = KernelCfg<MODE, NACC>::kSmemBytes;
  constexpr int threads = KernelCfg<MODE, NACC>::kThreads;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return OAPL_ERR_CUDA;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return OAPL_ERR_CUDA;
    attr_set[dev] = true;
  }
  const int slot = prof_begin(MODE, dev, st);
  if (slot >= 0 && g_prof.clk_addr) {
    GemmParams timed = gp;
    timed.clk = g_prof.clk_addr + 2 * MODE;
    kern<<<grid, threads, smem, st>>>(a, b, c, timed);
  } else {
    kern<<<grid, threads, smem, st>>>(a, b, c, gp);
  }
  OAPL_LAUNCHED();
  prof_end(slot, st);
  return cudaGetLastError() == cudaSuccess ? OAPL_OK : OAPL_ERR_CUDA;
}

static int check_problem(const oapl_problem* p, bool need_loss_inputs) {
  if (!p) return OAPL_ERR_INVALID_ARG;
  if (p->N <= 0 || p->d <= 0 || p->V <= 0 || p->S <= 0 || p->P <= 0) return OAPL_ERR_INVALID_ARG;
  if (p->d % 64 != 0) return OAPL_ERR_UNSUPPORTED_SHAPE;
  if (p->N > (int64_t)2000000000 || (int64_t)p->V + 512 > (int64_t)2000000000)
    return OAPL_ERR_UNSUPPORTED_SHAPE;
  if (!p->H || !p->W || !p->targets || !p->mask || !p->seq_id) return OAPL_ERR_INVALID_ARG;
  if (((uintptr_t)p->H | (uintptr_t)p->W) & 15) return OAPL_ERR_MISALIGNED;
  if (need_loss_inputs) {
    if (!p->group_id || !p->reward || !p->logp_inf) return OAPL_ERR_INVALID_ARG;
    if (!(p->beta_v > 0.f) || !std::isfinite(p->beta_v)) return OAPL_ERR_INVALID_ARG;
    if (!(p->beta_loss > 0.f) || !std::isfinite(p->beta_loss)) return OAPL_ERR_INVALID_ARG;
    if (!std::isfinite(p->loss_scale)) return OAPL_ERR_INVALID_ARG;
  }
  return OAPL_OK;
}

#define CK(call)                                   \
  do {                                             \
    if ((call) != cudaSuccess) return OAPL_ERR_CUDA; \
  } while (0)
#define CKL()                                                  \
  do {                                                         \
    OAPL_LAUNCHED();                                           \
    if (cudaGetLastError() != cudaSuccess) return OAPL_ERR_CUDA; \
  } while (0)

// Live-row compaction shared by every forward: state word, compacted per-row arrays,
// compacted-sequence bounds and the dense copy of the live rows of H.
static int prologue(const oapl_problem* p, const Carve& c, uint8_t* ws, float* token_logp, bool with_q,
                    cudaStream_t st) {
  NvtxRange nvtx("oapl: live-row compaction");
  const int n_sm = sm_count();
  if (n_sm <= 0) return OAPL_ERR_CUDA;
  DevState* state = reinterpret_cast<DevState*>(ws + c.state);
  int* block_cnt = reinterpret_cast<int*>(ws + c.block_cnt);
  int* block_off = reinterpret_cast<int*>(ws + c.block_off);
  int* live_rows = reinterpret_cast<int*>(ws + c.live_rows);
  int* tgt_c = reinterpret_cast<int*>(ws + c.tgt_c);
  int* seq_c = reinterpret_cast<int*>(ws + c.seq_c);
  float* q_c = reinterpret_cast<float*>(ws + c.q_c);
  int* cstart = reinterpret_cast<int*>(ws + c.cstart);
  int* cend = reinterpret_cast<int*>(ws + c.cend);
  __nv_bfloat16* Hc = reinterpret_cast<__nv_bfloat16*>(ws + c.Hc);

  CK(cudaMemsetAsync(state, 0, sizeof(DevState), st));
  CK(cudaMemsetAsync(ws + c.sync, 0, 4 * (size_t)kSyncSlots, st));
  CK(cudaMemsetAsync(cstart, 0, 4 * (size_t)p->S, st));
  CK(cudaMemsetAsync(cend, 0, 4 * (size_t)p->S, st));
  if (token_logp) CK(cudaMemsetAsync(token_logp, 0, 4 * (size_t)p->N, st));

  count_live_kernel<<<c.nblk, kScanBlock, 0, st>>>(p->mask, p->seq_id, p->targets, p->N, p->S, p->V,
                                                   block_cnt, &state->status);
  CKL();
  scan_blocks_kernel<<<1, 1024, 0, st>>>(block_cnt, c.nblk, block_off, state);
  CKL();
  write_live_kernel<<<c.nblk, kScanBlock, 0, st>>>(p->mask, p->seq_id, p->targets,
                                                   with_q ? p->logp_inf : nullptr, p->N, p->S, block_off,
                                                   live_rows, tgt_c, seq_c, q_c);
  CKL();
  seq_bounds_kernel<<<n_sm * 2, 256, 0, st>>>(seq_c, state, cstart, cend);
  CKL();
  gather_rows_kernel<<<n_sm * 8, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(p->H), live_rows,
                                               state, p->d, Hc);
  CKL();
  return OAPL_OK;
}

// Shared forward: compaction, fused logits + online log-sum-exp, merge, per-sequence sums.
static int forward_common(const oapl_problem* p, const Carve& c, uint8_t* ws, float* token_logp,
                          float* seq_logp, bool with_q, cudaStream_t st) {
  const int n_sm = sm_count();
  if (n_sm <= 0) return OAPL_ERR_CUDA;
  int rc0 = prologue(p, c, ws, token_logp, with_q, st);
  if (rc0 != OAPL_OK) return rc0;
  DevState* state = reinterpret_cast<DevState*>(ws + c.state);
  int* live_rows = reinterpret_cast<int*>(ws + c.live_rows);
  int* tgt_c = reinterpret_cast<int*>(ws + c.tgt_c);
  float* q_c = reinterpret_cast<float*>(ws + c.q_c);
  float* lp_c = reinterpret_cast<float*>(ws + c.lp_c);
  float* lse = reinterpret_cast<float*>(ws + c.lse);
  int* cstart = reinterpret_cast<int*>(ws + c.cstart);
  int* cend = reinterpret_cast<int*>(ws + c.cend);
  __nv_bfloat16* Hc = reinterpret_cast<__nv_bfloat16*>(ws + c.Hc);

  CUtensorMap tmA, tmB;
  if (!make_map(&tmA, Hc, (uint64_t)c.n_pad, (uint64_t)p->d, (uint64_t)p->d, 128)) return OAPL_ERR_CUDA;
  if (!make_map(&tmB, p->W, (uint64_t)p->V, (uint64_t)p->d, (uint64_t)p->d, 128)) return OAPL_ERR_CUDA;
  GemmParams gp;
  memset(&gp, 0, sizeof(gp));
  gp.n_live_ptr = &state->n_live;
  gp.row_begin = 0;
  gp.row_cap = c.n_pad;
  const int vtiles = (p->V + 2 * kBN - 1) / (2 * kBN);  // the sweep walks 512-column tiles
  pick_sweep(n_sm, p->d, vtiles, &gp.R, &gp.C);
  gp.d = p->d;
  gp.V = p->V;
  gp.pm = reinterpret_cast<float*>(ws + c.pm);
  gp.pl = reinterpret_cast<float*>(ws + c.pl);
  gp.pz = reinterpret_cast<float*>(ws + c.pz);
  gp.ps = reinterpret_cast<float*>(ws + c.ps);
  gp.tgt_c = tgt_c;
  gp.err = &state->status;
  set_lockstep(&gp, ws, c, 0, p->d / kBK);
  NvtxRange nvtx("oapl: logits + online log-sum-exp, merge, sequence sums");
  int rc = launch_gemm<MODE_LSE, 0, 0, 2>(tmA, tmB, tmA, gp, 2 * gp.R * gp.C, st);
  if (rc != OAPL_OK) return rc;

  merge_lse_kernel<<<n_sm * 2, 256, 0, st>>>(gp.pm, gp.pl, gp.pz, gp.ps, gp.R, gp.C, vtiles, state, live_rows, lse,
                                             lp_c,
                                             reinterpret_cast<float*>(ws + c.ent_c), token_logp);
  CKL();
  seq_sums_kernel<<<p->S, 256, 0, st>>>(lp_c, q_c, cstart, cend, seq_logp,
                                        reinterpret_cast<float*>(ws + c.seq_D), with_q ? 1 : 0, nullptr);
  CKL();
  return OAPL_OK;
}

// What the staged single-call pipeline optimises: Eq. 3 (per-sequence coefficients) or
// the GRPO display of the Background section (per-token coefficients).
struct Objective {
  bool grpo;
  float* vhat;            // OAPL
  float* delta;           // OAPL, may be null
  const float* logp_old;  // GRPO [N]
  const float* adv;       // GRPO [S]
  float clip_eps;         // GRPO
  float* clip_frac;       // GRPO, may be null
};

// Number of range slots the single call enqueues: the largest number of ranges the greedy packing
// of whole sequences into `stage` rows can produce for at most `live` live rows in sequences of at
// most `longest` live rows each (0 = unknown), never more than the capacity of the range table.
//   - two neighbouring ranges together hold more than `stage` rows:  n <= 2 ceil(live/stage) - 1
//   - every range but the last holds more than stage - longest rows: n <= live/(stage-longest+1) + 1
static int range_slots(long long live, long long longest, int stage, int S, int table_capacity) {
  if (live < 1) live = 1;
  long long n = 2 * ((live + stage - 1) / stage) - 1;
  if (longest > 0 && longest <= stage) {
    const long long m = live / (stage - longest + 1) + 1;
    if (m < n) n = m;
  }
  if (n > S) n = S;
  if (n > table_capacity) n = table_capacity;
  if (n < 1) n = 1;
  return (int)n;
}

static int staged_fwd_bwd(const oapl_problem* p, const Objective& ob, float* loss, float* seq_logp,
                          float* token_logp, void* dH, float* dW, int accumulate_dW, uint8_t* w,
                          const Carve& c, const oapl_call_options* opt, cudaStream_t st) {
  const int n_sm = sm_count();
  if (n_sm <= 0) return OAPL_ERR_CUDA;
  long long live_bound = p->N, longest_bound = 0;
  if (opt) {
    if (opt->live_rows_bound > 0 && opt->live_rows_bound < live_bound) live_bound = opt->live_rows_bound;
    longest_bound = opt->max_seq_rows_bound;
  }
  const int slots = range_slots(live_bound, longest_bound, c.stage_rows, p->S, c.max_ranges);
  int rc = prologue(p, c, w, token_logp, true, st);
  if (rc != OAPL_OK) return rc;
  DevState* state = reinterpret_cast<DevState*>(w + c.state);
  int* live_rows = reinterpret_cast<int*>(w + c.live_rows);
  int* tgt_c = reinterpret_cast<int*>(w + c.tgt_c);
  int* seq_c = reinterpret_cast<int*>(w + c.seq_c);
  float* q_c = reinterpret_cast<float*>(w + c.q_c);
  float* lp_c = reinterpret_cast<float*>(w + c.lp_c);
  float* lse = reinterpret_cast<float*>(w + c.lse);
  int* cstart = reinterpret_cast<int*>(w + c.cstart);
  int* cend = reinterpret_cast<int*>(w + c.cend);
  float* seq_D = reinterpret_cast<float*>(w + c.seq_D);
  float* coef = reinterpret_cast<float*>(w + c.coef);
  float* coef_row = reinterpret_cast<float*>(w + c.coef_row);
  float* qo_c = reinterpret_cast<float*>(w + c.qo_c);
  float* seq_obj = reinterpret_cast<float*>(w + c.seq_obj);
  int* seq_clip = reinterpret_cast<int*>(w + c.seq_clip);
  __nv_bfloat16* Hc = reinterpret_cast<__nv_bfloat16*>(w + c.Hc);
  __nv_bfloat16* E = reinterpret_cast<__nv_bfloat16*>(w + c.G);
  __nv_bfloat16* Hs = reinterpret_cast<__nv_bfloat16*>(w + c.Hs);
  float* zref = reinterpret_cast<float*>(w + c.zref);
  float* alpha = reinterpret_cast<float*>(w + c.alpha);
  float* ztc = reinterpret_cast<float*>(w + c.ztc);
  float* rowscale = reinterpret_cast<float*>(w + c.rowscale);
  RangeRec* ranges = reinterpret_cast<RangeRec*>(w + c.ranges);
  const int vtiles = (p->V + 2 * kBN - 1) / (2 * kBN);  // the single-call sweep walks 512-column tiles

  CK(cudaMemsetAsync(seq_D, 0, 4 * (size_t)p->S, st));
  if (seq_logp) CK(cudaMemsetAsync(seq_logp, 0, 4 * (size_t)p->S, st));
  if (!accumulate_dW) CK(cudaMemsetAsync(dW, 0, 4 * (size_t)p->V * (size_t)p->d, st));
  zero_dead_rows_kernel<<<n_sm * 8, 256, 0, st>>>(p->mask, p->N, p->d, static_cast<__nv_bfloat16*>(dH),
                                                  nullptr);
  CKL();
  if (ob.grpo) {
    CK(cudaMemsetAsync(seq_obj, 0, 4 * (size_t)p->S, st));
    CK(cudaMemsetAsync(seq_clip, 0, 4 * (size_t)p->S, st));
    gather_f32_kernel<<<n_sm * 4, 256, 0, st>>>(ob.logp_old, live_rows, state, qo_c);
    CKL();
  } else {
    value_estimate_kernel<<<(p->P + 7) / 8, 256, 0, st>>>(p->reward, p->group_id, p->S, p->P, p->beta_v,
                                                          ob.vhat, &state->status);
    CKL();
  }
  ztgt_kernel<<<n_sm * 8, 256, 0, st>>>(Hc, reinterpret_cast<const __nv_bfloat16*>(p->W), tgt_c, state,
                                        p->d, p->V, zref);
  CKL();
  plan_ranges_kernel<<<1, 32, 0, st>>>(cstart, cend, p->S, c.stage_rows, slots, ranges, state);
  CKL();

  CUtensorMap tmH, tmW, tmEk, tmEst, tmWmn, tmEmn, tmHsmn, tmdW;
  const uint64_t ldg = (uint64_t)c.ldg;
  bool ok = make_map(&tmH, Hc, (uint64_t)c.n_pad, (uint64_t)p->d, (uint64_t)p->d, 128) &&
            make_map(&tmW, p->W, (uint64_t)p->V, (uint64_t)p->d, (uint64_t)p->d, 128) &&
            make_map(&tmEk, E, (uint64_t)c.stage_alloc_rows, ldg, ldg, 128) &&
            make_map_store32(&tmEst, E, (uint64_t)c.stage_alloc_rows, ldg, ldg) &&
            make_map(&tmWmn, p->W, (uint64_t)p->V, (uint64_t)p->d, (uint64_t)p->d, 64) &&
            make_map(&tmEmn, E, (uint64_t)c.stage_alloc_rows, ldg, ldg, 64) &&
            make_map(&tmHsmn, Hs, (uint64_t)c.n_pad + 256, (uint64_t)p->d, (uint64_t)p->d, 64) &&
            make_map_f32(&tmdW, dW, (uint64_t)p->V, (uint64_t)p->d, (uint64_t)p->d);
  if (!ok) return OAPL_ERR_CUDA;

  GemmParams gp;
  memset(&gp, 0, sizeof(gp));
  gp.n_live_ptr = &state->n_live;
  gp.d = p->d;
  gp.V = p->V;
  gp.ldg = c.ldg;
  gp.pl = reinterpret_cast<float*>(w + c.pl);
  gp.pz = reinterpret_cast<float*>(w + c.pz);
  gp.ps = reinterpret_cast<float*>(w + c.ps);
  gp.tgt_c = tgt_c;
  gp.zref = zref;
  gp.live_rows = live_rows;
  gp.dH = static_cast<__nv_bfloat16*>(dH);
  gp.dW = dW;
  gp.err = &state->status;
  pick_sweep(n_sm, p->d, vtiles, &gp.R, &gp.C);

  // The ranges live on the device; the host enqueues the largest number of ranges the packing
  // can produce for the row bounds it was given.  The planner fills the LAST slots, so empty
  // slots come first (their launches return at once) and the last slot always holds the last
  // range: the event after its dW launch marks dW complete while its dH contraction still runs.
  for (int k = 0; k < slots; ++k) {
    NvtxRange nvtx("oapl: range slot (logits + exp, coefficients, dW, dH)");
    const RangeRec* rg = ranges + k;
    gp.range_ptr = &rg->row_begin;
    gp.rowscale = nullptr;
    set_lockstep(&gp, w, c, 3 * k, p->d / kBK);
    rc = launch_gemm<MODE_LSE_E, 0, 0, 2>(tmH, tmW, tmEst, gp, 2 * gp.R * gp.C, st);
    if (rc != OAPL_OK) return rc;
    merge_e_kernel<<<n_sm, 256, 0, st>>>(gp.pl, gp.pz, gp.ps, zref, rg, gp.R, gp.C, vtiles, live_rows, lse, lp_c,
                                         reinterpret_cast<float*>(w + c.ent_c), alpha, ztc, token_logp, state);
    CKL();
    seq_sums_kernel<<<p->S, 256, 0, st>>>(lp_c, q_c, cstart, cend, seq_logp, seq_D, 1, &rg->seq_begin);
    CKL();
    if (ob.grpo) {
      grpo_coef_kernel<<<p->S, 256, 0, st>>>(lp_c, qo_c, q_c, cstart, cend, ob.adv, &rg->seq_begin,
                                             ob.clip_eps, p->loss_scale, coef_row, seq_obj, seq_clip);
      CKL();
    } else {
      coef_range_kernel<<<(p->S + 255) / 256, 256, 0, st>>>(p->reward, p->group_id, ob.vhat, seq_D, rg, p->P,
                                                            p->beta_loss, p->loss_scale, coef);
      CKL();
    }
    scale_patch_kernel<<<n_sm * 8, 256, 0, st>>>(Hc, seq_c, tgt_c, coef, ob.grpo ? coef_row : nullptr, alpha,
                                                 lse, ztc, rg, p->d, p->V, c.ldg, Hs, rowscale, E);
    CKL();
    set_lockstep(&gp, w, c, 3 * k + 1, 0);
    rc = launch_gemm<MODE_DW, 1, 1, 2>(tmEmn, tmHsmn, tmdW, gp, n_sm & ~1, st);
    if (rc != OAPL_OK) return rc;
    if (k == slots - 1 && opt && opt->dW_ready_event)
      CK(cudaEventRecord(static_cast<cudaEvent_t>(opt->dW_ready_event), st));
    gp.rowscale = rowscale;
    set_lockstep(&gp, w, c, 3 * k + 2, 0);
    rc = launch_gemm<MODE_DH, 0, 1, 2>(tmEk, tmWmn, tmEk, gp, n_sm & ~1, st);
    if (rc != OAPL_OK) return rc;
  }
  if (ob.grpo) {
    grpo_loss_kernel<<<1, 256, 0, st>>>(seq_obj, seq_clip, p->S, p->loss_scale, loss, ob.clip_frac, state);
  } else {
    loss_kernel<<<1, 256, 0, st>>>(p->reward, p->group_id, ob.vhat, seq_D, p->S, p->P, p->beta_loss,
                                   p->loss_scale, coef, ob.delta, loss, state);
  }
  CKL();
  return OAPL_OK;
}

}  // namespace oapl

using namespace oapl;

extern "C" {

size_t oapl_workspace_bytes(const oapl_problem* problem, int flags) {
  Carve c;
  if (!carve(problem, flags, &c)) return 0;
  return c.total;
}

const char* oapl_status_string(int status) {
  switch (status) {
    case OAPL_OK: return "ok";
    case OAPL_ERR_INVALID_ARG: return "invalid argument";
    case OAPL_ERR_MISALIGNED: return "pointer not 16-byte aligned";
    case OAPL_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case OAPL_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (d must be a multiple of 64)";
    case OAPL_ERR_BAD_TARGET: return "target outside [0,V) on a live row";
    case OAPL_ERR_BAD_SEQ_ORDER: return "seq_id decreasing or outside [0,S)";
    case OAPL_ERR_NONFINITE_INPUT: return "non-finite reward or group_id outside [0,P)";
    case OAPL_ERR_DEVICE_TIMEOUT: return "device pipeline wait timed out";
    case OAPL_ERR_CUDA: return "CUDA call failed";
    case OAPL_ERR_BAD_STATE: return "backward called without a matching forward";
    case OAPL_ERR_SEQUENCE_TOO_LONG: return "a sequence has more live rows than the staging capacity";
    case OAPL_ERR_OUT_OF_RANGE: return "staged exponentials out of range (logit far above the target's, or non-finite input)";
    case OAPL_ERR_BOUND_EXCEEDED: return "the batch has more live rows (or a longer sequence) than the caller's bounds";
    default: return "unknown status";
  }
}

uint64_t oapl_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int oapl_get_last_status(void* ws, void* stream) {
  if (!ws) return OAPL_ERR_INVALID_ARG;
  DevState h;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&h, ws, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return OAPL_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return OAPL_ERR_CUDA;
  return h.status;
}

int64_t oapl_get_live_rows(void* ws, void* stream) {
  if (!ws) return OAPL_ERR_INVALID_ARG;
  DevState h;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&h, ws, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return OAPL_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return OAPL_ERR_CUDA;
  return h.n_live;
}

int oapl_get_range_count(void* ws, void* stream) {
  if (!ws) return OAPL_ERR_INVALID_ARG;
  DevState h;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&h, ws, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return OAPL_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return OAPL_ERR_CUDA;
  return h.n_ranges;
}

int oapl_value_estimate(const float* reward, const int32_t* group_id, int32_t S, int32_t P,
                        float beta_v, float* vhat, void* stream) {
  if (!reward || !group_id || !vhat || S <= 0 || P <= 0) return OAPL_ERR_INVALID_ARG;
  if (!(beta_v > 0.f) || !std::isfinite(beta_v)) return OAPL_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  value_estimate_kernel<<<(P + 7) / 8, 256, 0, st>>>(reward, group_id, S, P, beta_v, vhat, nullptr);
  CKL();
  return OAPL_OK;
}

int oapl_token_logprobs(const oapl_problem* p, float* token_logp, float* seq_logp, void* ws,
                        size_t ws_bytes, int /*flags*/, void* stream) {
  int rc = check_problem(p, false);
  if (rc != OAPL_OK) return rc;
  if (!token_logp || !ws) return OAPL_ERR_INVALID_ARG;
  if ((uintptr_t)ws & 1023) return OAPL_ERR_MISALIGNED;
  Carve c;
  if (!carve(p, 0, &c)) return OAPL_ERR_INVALID_ARG;
  if (ws_bytes < c.total) return OAPL_ERR_WORKSPACE_TOO_SMALL;
  return forward_common(p, c, static_cast<uint8_t*>(ws), token_logp, seq_logp, false,
                        static_cast<cudaStream_t>(stream));
}

int oapl_loss_fwd(const oapl_problem* p, float* loss, float* seq_logp, float* vhat, float* delta,
                  float* token_logp, void* ws, size_t ws_bytes, int /*flags*/, void* stream) {
  int rc = check_problem(p, true);
  if (rc != OAPL_OK) return rc;
  if (!loss || !seq_logp || !vhat || !ws) return OAPL_ERR_INVALID_ARG;
  if ((uintptr_t)ws & 1023) return OAPL_ERR_MISALIGNED;
  Carve c;
  if (!carve(p, 0, &c)) return OAPL_ERR_INVALID_ARG;
  if (ws_bytes < c.total) return OAPL_ERR_WORKSPACE_TOO_SMALL;
  uint8_t* w = static_cast<uint8_t*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = forward_common(p, c, w, token_logp, seq_logp, true, st);
  if (rc != OAPL_OK) return rc;
  DevState* state = reinterpret_cast<DevState*>(w + c.state);
  value_estimate_kernel<<<(p->P + 7) / 8, 256, 0, st>>>(p->reward, p->group_id, p->S, p->P, p->beta_v,
                                                        vhat, &state->status);
  CKL();
  loss_kernel<<<1, 256, 0, st>>>(p->reward, p->group_id, vhat, reinterpret_cast<float*>(w + c.seq_D),
                                 p->S, p->P, p->beta_loss, p->loss_scale,
                                 reinterpret_cast<float*>(w + c.coef), delta, loss, state);
  CKL();
  return OAPL_OK;
}

int oapl_loss_bwd(const oapl_problem* p, void* dH, float* dW, int accumulate_dW, void* ws,
                  size_t ws_bytes, int /*flags*/, void* stream) {
  int rc = check_problem(p, true);
  if (rc != OAPL_OK) return rc;
  if (!dH || !dW || !ws) return OAPL_ERR_INVALID_ARG;
  if (((uintptr_t)dH | (uintptr_t)dW) & 15) return OAPL_ERR_MISALIGNED;
  if ((uintptr_t)ws & 1023) return OAPL_ERR_MISALIGNED;
  Carve c;
  if (!carve(p, 0, &c)) return OAPL_ERR_INVALID_ARG;
  if (ws_bytes < c.total) return OAPL_ERR_WORKSPACE_TOO_SMALL;
  const int n_sm = sm_count();
  if (n_sm <= 0) return OAPL_ERR_CUDA;
  uint8_t* w = static_cast<uint8_t*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DevState* state = reinterpret_cast<DevState*>(w + c.state);
  __nv_bfloat16* Hc = reinterpret_cast<__nv_bfloat16*>(w + c.Hc);
  __nv_bfloat16* G = reinterpret_cast<__nv_bfloat16*>(w + c.G);

  zero_dead_rows_kernel<<<n_sm * 8, 256, 0, st>>>(p->mask, p->N, p->d, static_cast<__nv_bfloat16*>(dH), state);
  CKL();
  if (!accumulate_dW) CK(cudaMemsetAsync(dW, 0, 4 * (size_t)p->V * (size_t)p->d, st));

  CUtensorMap tmH, tmW, tmGk, tmGst, tmWmn, tmGmn, tmHmn, tmdW;
  const uint64_t ldg = (uint64_t)c.ldg;
  bool ok = make_map(&tmH, Hc, (uint64_t)c.n_pad, (uint64_t)p->d, (uint64_t)p->d, 128) &&
            make_map(&tmW, p->W, (uint64_t)p->V, (uint64_t)p->d, (uint64_t)p->d, 128) &&
            make_map(&tmGk, G, (uint64_t)c.chunk_rows, ldg, ldg, 128) &&
            make_map_store32(&tmGst, G, (uint64_t)c.chunk_rows, ldg, ldg) &&
            make_map(&tmWmn, p->W, (uint64_t)p->V, (uint64_t)p->d, (uint64_t)p->d, 64) &&
            make_map(&tmGmn, G, (uint64_t)c.chunk_rows, ldg, ldg, 64) &&
            make_map(&tmHmn, Hc, (uint64_t)c.n_pad, (uint64_t)p->d, (uint64_t)p->d, 64) &&
            make_map_f32(&tmdW, dW, (uint64_t)p->V, (uint64_t)p->d, (uint64_t)p->d);
  if (!ok) return OAPL_ERR_CUDA;

  GemmParams gp;
  memset(&gp, 0, sizeof(gp));
  gp.n_live_ptr = &state->n_live;
  gp.tag_ptr = &state->fwd_tag;
  gp.row_cap = c.chunk_rows;
  gp.d = p->d;
  gp.V = p->V;
  gp.ldg = c.ldg;
  gp.tgt_c = reinterpret_cast<int*>(w + c.tgt_c);
  gp.seq_c = reinterpret_cast<int*>(w + c.seq_c);
  gp.lse = reinterpret_cast<float*>(w + c.lse);
  gp.coef = reinterpret_cast<float*>(w + c.coef);
  gp.live_rows = reinterpret_cast<int*>(w + c.live_rows);
  gp.dH = static_cast<__nv_bfloat16*>(dH);
  gp.dW = dW;
  // dW is zeroed above unless the caller accumulates; every chunk adds to it
  gp.err = &state->status;
  pick_sweep(n_sm, p->d, (p->V + 2 * kBN - 1) / (2 * kBN), &gp.R, &gp.C);  // 512-column sweep tiles

  // Row chunks of the compacted rows.  The live-row count lives on the device, so the
  // host enqueues every chunk the row count N could need; chunks past the live rows
  // find no tile and return at once.
  CK(cudaMemsetAsync(w + c.sync, 0, 4 * (size_t)kSyncSlots, st));
  int slot = 0;
  for (int r0 = 0; r0 < c.n_pad; r0 += c.chunk_rows) {
    NvtxRange nvtx("oapl: backward row chunk (logit gradient, dH, dW)");
    gp.row_begin = r0;
    set_lockstep(&gp, w, c, slot++, p->d / kBK);
    rc = launch_gemm<MODE_GRAD, 0, 0, 2>(tmH, tmW, tmGst, gp, 2 * gp.R * gp.C, st);
    if (rc != OAPL_OK) return rc;
    set_lockstep(&gp, w, c, slot++, 0);
    rc = launch_gemm<MODE_DH, 0, 1, 2>(tmGk, tmWmn, tmGk, gp, n_sm & ~1, st);
    if (rc != OAPL_OK) return rc;
    set_lockstep(&gp, w, c, slot++, 0);
    rc = launch_gemm<MODE_DW, 1, 1, 2>(tmGmn, tmHmn, tmdW, gp, n_sm & ~1, st);
    if (rc != OAPL_OK) return rc;
  }
  return OAPL_OK;
}

int oapl_loss_fwd_bwd(const oapl_problem* p, float* loss, float* seq_logp, float* vhat, float* delta,
                      float* token_logp, void* dH, float* dW, int accumulate_dW, void* ws,
                      size_t ws_bytes, int flags, void* stream) {
  return oapl_loss_fwd_bwd_ex(p, loss, seq_logp, vhat, delta, token_logp, dH, dW, accumulate_dW, ws, ws_bytes,
                              flags, nullptr, stream);
}

int oapl_loss_fwd_bwd_ex(const oapl_problem* p, float* loss, float* seq_logp, float* vhat, float* delta,
                         float* token_logp, void* dH, float* dW, int accumulate_dW, void* ws,
                         size_t ws_bytes, int flags, const oapl_call_options* options, void* stream) {
  int rc = check_problem(p, true);
  if (rc != OAPL_OK) return rc;
  if (!loss || !seq_logp || !vhat || !dH || !dW || !ws) return OAPL_ERR_INVALID_ARG;
  if (options && (options->live_rows_bound < 0 || options->max_seq_rows_bound < 0)) return OAPL_ERR_INVALID_ARG;
  if (((uintptr_t)dH | (uintptr_t)dW) & 15) return OAPL_ERR_MISALIGNED;
  if ((uintptr_t)ws & 1023) return OAPL_ERR_MISALIGNED;
  Carve c;
  if (!carve(p, flags | OAPL_FLAG_FUSED, &c)) return OAPL_ERR_INVALID_ARG;
  if (ws_bytes < c.total) return OAPL_ERR_WORKSPACE_TOO_SMALL;
  Objective ob;
  memset(&ob, 0, sizeof(ob));
  ob.grpo = false;
  ob.vhat = vhat;
  ob.delta = delta;
  return staged_fwd_bwd(p, ob, loss, seq_logp, token_logp, dH, dW, accumulate_dW, static_cast<uint8_t*>(ws), c,
                        options, static_cast<cudaStream_t>(stream));
}

int oapl_group_advantage(const float* reward, const int32_t* group_id, int32_t S, int32_t P, float eps,
                         float* advantage, void* stream) {
  if (!reward || !group_id || !advantage || S <= 0 || P <= 0) return OAPL_ERR_INVALID_ARG;
  if (!(eps >= 0.f) || !std::isfinite(eps)) return OAPL_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  group_advantage_kernel<<<(P + 7) / 8, 256, 0, st>>>(reward, group_id, S, P, eps, advantage);
  CKL();
  return OAPL_OK;
}

int oapl_grpo_loss_fwd_bwd(const oapl_problem* p, const float* logp_old, const float* advantage,
                           float clip_eps, float* loss, float* seq_logp, float* token_logp, float* clip_frac,
                           void* dH, float* dW, int accumulate_dW, void* ws, size_t ws_bytes, int flags,
                           void* stream) {
  int rc = check_problem(p, false);
  if (rc != OAPL_OK) return rc;
  if (!p->logp_inf || !logp_old || !advantage || !loss || !dH || !dW || !ws) return OAPL_ERR_INVALID_ARG;
  if (!(clip_eps >= 0.f) || !std::isfinite(clip_eps) || !std::isfinite(p->loss_scale)) return OAPL_ERR_INVALID_ARG;
  if (((uintptr_t)dH | (uintptr_t)dW) & 15) return OAPL_ERR_MISALIGNED;
  if ((uintptr_t)ws & 1023) return OAPL_ERR_MISALIGNED;
  Carve c;
  if (!carve(p, flags | OAPL_FLAG_FUSED, &c)) return OAPL_ERR_INVALID_ARG;
  if (ws_bytes < c.total) return OAPL_ERR_WORKSPACE_TOO_SMALL;
  Objective ob;
  memset(&ob, 0, sizeof(ob));
  ob.grpo = true;
  ob.logp_old = logp_old;
  ob.adv = advantage;
  ob.clip_eps = clip_eps;
  ob.clip_frac = clip_frac;
  return staged_fwd_bwd(p, ob, loss, seq_logp, token_logp, dH, dW, accumulate_dW, static_cast<uint8_t*>(ws), c,
                        nullptr, static_cast<cudaStream_t>(stream));
}

size_t oapl_adamw_workspace_bytes(void) { return sizeof(double) * kAdamMaxPartials; }

int oapl_adamw_step(void* W, float* master, const float* dW, float* m, float* v, int64_t n, int64_t step,
                    float lr, float beta1, float beta2, float eps, float weight_decay, float clip_norm,
                    const float* other_sq_norm, float* grad_norm, void* ws, size_t ws_bytes, void* stream) {
  if (!W || !dW || !m || !v || !ws || n <= 0 || step < 1) return OAPL_ERR_INVALID_ARG;
  if (!(lr >= 0.f) || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f) ||
      !(weight_decay >= 0.f) || !std::isfinite(lr) || !std::isfinite(eps) || !std::isfinite(weight_decay) ||
      !std::isfinite(clip_norm))
    return OAPL_ERR_INVALID_ARG;
  if (((uintptr_t)W & 7) || (((uintptr_t)dW | (uintptr_t)m | (uintptr_t)v | (uintptr_t)master) & 15) ||
      ((uintptr_t)ws & 7))
    return OAPL_ERR_MISALIGNED;
  if (ws_bytes < sizeof(double) * kAdamMaxPartials) return OAPL_ERR_WORKSPACE_TOO_SMALL;
  const int n_sm = sm_count();
  if (n_sm <= 0) return OAPL_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  double* partial = static_cast<double*>(ws);
  const size_t work = ((size_t)n / 4 + kAdamThreads - 1) / kAdamThreads;
  int grid = n_sm * 8;
  if ((size_t)grid > work) grid = work ? (int)work : 1;
  if (grid > kAdamMaxPartials) grid = kAdamMaxPartials;
  sqnorm_partial_kernel<<<grid, kAdamThreads, 0, st>>>(dW, (size_t)n, partial);
  CKL();
  AdamParams a;
  a.lr = lr;
  a.beta1 = beta1;
  a.beta2 = beta2;
  a.eps = eps;
  a.weight_decay = weight_decay;
  a.clip_norm = clip_norm;
  a.bias1 = (float)(1.0 - std::pow((double)beta1, (double)step));
  a.bias2 = (float)(1.0 - std::pow((double)beta2, (double)step));
  adamw_kernel<<<grid, kAdamThreads, 0, st>>>(dW, m, v, master, static_cast<__nv_bfloat16*>(W), (size_t)n, partial,
                                              grid, other_sq_norm, a, grad_norm);
  CKL();
  return OAPL_OK;
}

int oapl_entropy(const oapl_problem* p, float* token_entropy, float* seq_entropy, float* mean_entropy,
                 void* ws, size_t ws_bytes, int flags, void* stream) {
  int rc = check_problem(p, false);
  if (rc != OAPL_OK) return rc;
  if (!ws || (!token_entropy && !seq_entropy && !mean_entropy)) return OAPL_ERR_INVALID_ARG;
  if ((uintptr_t)ws & 1023) return OAPL_ERR_MISALIGNED;
  Carve c;
  if (!carve(p, flags, &c)) return OAPL_ERR_INVALID_ARG;
  if (ws_bytes < c.total) return OAPL_ERR_WORKSPACE_TOO_SMALL;
  uint8_t* w = static_cast<uint8_t*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DevState* state = reinterpret_cast<DevState*>(w + c.state);
  const float* ent_c = reinterpret_cast<const float*>(w + c.ent_c);
  if (token_entropy) CK(cudaMemsetAsync(token_entropy, 0, 4 * (size_t)p->N, st));
  entropy_seq_kernel<<<p->S, 256, 0, st>>>(ent_c, reinterpret_cast<const int*>(w + c.cstart),
                                           reinterpret_cast<const int*>(w + c.cend),
                                           reinterpret_cast<const int*>(w + c.live_rows), token_entropy,
                                           seq_entropy, state);
  CKL();
  if (mean_entropy) {
    entropy_mean_kernel<<<1, 1024, 0, st>>>(ent_c, state, mean_entropy);
    CKL();
  }
  return OAPL_OK;
}

int oapl_batch_stats(const oapl_problem* p, const float* vhat, float* stats, void* ws, size_t ws_bytes, int flags,
                     void* stream) {
  int rc = check_problem(p, true);
  if (rc != OAPL_OK) return rc;
  if (!vhat || !stats || !ws) return OAPL_ERR_INVALID_ARG;
  if ((uintptr_t)ws & 1023) return OAPL_ERR_MISALIGNED;
  Carve c;
  if (!carve(p, flags, &c)) return OAPL_ERR_INVALID_ARG;
  if (ws_bytes < c.total) return OAPL_ERR_WORKSPACE_TOO_SMALL;
  uint8_t* w = static_cast<uint8_t*>(ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  batch_stats_kernel<<<1, 256, 0, st>>>(reinterpret_cast<const float*>(w + c.seq_D),
                                        reinterpret_cast<const int*>(w + c.cstart),
                                        reinterpret_cast<const int*>(w + c.cend), p->reward, p->group_id, vhat,
                                        p->S, p->P, reinterpret_cast<DevState*>(w + c.state), stats);
  CKL();
  return OAPL_OK;
}

int oapl_profile_enable(int on) {
  if (!on) {
    g_prof.device = -1;
    g_prof.used = 0;
    g_prof.dropped = 0;
    return OAPL_OK;
  }
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return OAPL_ERR_CUDA;
  if (g_prof.made_on != dev) {
    // events belong to the device they were created on: start over on another device
    if (g_prof.made_on >= 0) {
      int cur = dev;
      if (cudaSetDevice(g_prof.made_on) == cudaSuccess)
        for (auto& pr : g_prof.pairs) { cudaEventDestroy(pr.ev[0]); cudaEventDestroy(pr.ev[1]); }
      cudaSetDevice(cur);
    }
    g_prof.pairs.clear();
    g_prof.made_on = dev;
  }
  void* ptr = nullptr;
  if (cudaGetSymbolAddress(&ptr, g_prof_clk) != cudaSuccess) return OAPL_ERR_CUDA;
  if (cudaMemset(ptr, 0, sizeof(unsigned long long) * kProfKinds * 2) != cudaSuccess) return OAPL_ERR_CUDA;
  g_prof.clk_addr = static_cast<unsigned long long*>(ptr);
  g_prof.device = dev;
  g_prof.used = 0;
  g_prof.dropped = 0;
  return OAPL_OK;
}

int oapl_profile_read_clocks(float* sm_mhz_by_kind, int kinds) {
  if (!sm_mhz_by_kind || kinds <= 0 || kinds > kProfKinds) return OAPL_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return OAPL_ERR_CUDA;
  if (!g_prof.clk_addr || !prof_applies(g_prof.device, dev)) return OAPL_ERR_BAD_STATE;
  unsigned long long h[kProfKinds][2];
  if (cudaDeviceSynchronize() != cudaSuccess) return OAPL_ERR_CUDA;
  if (cudaMemcpy(h, g_prof.clk_addr, sizeof(h), cudaMemcpyDeviceToHost) != cudaSuccess) return OAPL_ERR_CUDA;
  for (int k = 0; k < kinds; ++k)
    sm_mhz_by_kind[k] = h[k][1] ? (float)((double)h[k][0] / (double)h[k][1] * 1e3) : 0.f;
  if (cudaMemset(g_prof.clk_addr, 0, sizeof(h)) != cudaSuccess) return OAPL_ERR_CUDA;
  return OAPL_OK;
}

int oapl_profile_read(float* ms_by_kind, int* launches_by_kind, int kinds, int* launches_dropped) {
  if (!ms_by_kind || !launches_by_kind || kinds <= 0) return OAPL_ERR_INVALID_ARG;
  for (int k = 0; k < kinds; ++k) { ms_by_kind[k] = 0.f; launches_by_kind[k] = 0; }
  if (launches_dropped) *launches_dropped = g_prof.dropped;
  for (int s = 0; s < g_prof.used; ++s) {
    const ProfPair& pr = g_prof.pairs[s];
    float ms = 0.f;
    if (cudaEventSynchronize(pr.ev[1]) != cudaSuccess) return OAPL_ERR_CUDA;
    if (cudaEventElapsedTime(&ms, pr.ev[0], pr.ev[1]) != cudaSuccess) return OAPL_ERR_CUDA;
    if (pr.kind < kinds) { ms_by_kind[pr.kind] += ms; launches_by_kind[pr.kind] += 1; }
  }
  g_prof.used = 0;
  g_prof.dropped = 0;
  return OAPL_OK;
}

int oapl_range_slots(int64_t live_rows_bound, int64_t max_seq_rows_bound, int32_t stage_rows, int32_t S) {
  if (stage_rows < 1 || S < 1 || live_rows_bound < 0 || max_seq_rows_bound < 0) return OAPL_ERR_INVALID_ARG;
  return range_slots(live_rows_bound, max_seq_rows_bound, stage_rows, S, 0x7fffffff);
}

int oapl_profile_applies(int enabled_device, int current_device) {
  return prof_applies(enabled_device, current_device) ? 1 : 0;
}

int oapl_debug_gemm(const void* A, const void* B, float* C, int M, int N, int K, int a_mn, int b_mn,
                    int wide, long long wait_cycles, int skip_step, int* err, void* stream) {
  if (!A || !B || !C || !err || M <= 0 || N <= 0 || K <= 0) return OAPL_ERR_INVALID_ARG;
  if (wait_cycles < 0 || skip_step < 0) return OAPL_ERR_INVALID_ARG;
  // leaving a pipeline step out is only allowed together with a short wait limit (at most 1e8
  // cycles, well under a tenth of a second), so that the launch ends soon
  if (skip_step > 0 && (wait_cycles == 0 || wait_cycles > 100000000LL)) return OAPL_ERR_INVALID_ARG;
  if (K % 64 || M % 8 || N % 8) return OAPL_ERR_UNSUPPORTED_SHAPE;
  const int n_sm = sm_count();
  if (n_sm <= 0) return OAPL_ERR_CUDA;
  CUtensorMap ta, tb;
  bool ok = a_mn ? make_map(&ta, A, (uint64_t)K, (uint64_t)M, (uint64_t)M, 64)
                 : make_map(&ta, A, (uint64_t)M, (uint64_t)K, (uint64_t)K, 128);
  ok = ok && (b_mn ? make_map(&tb, B, (uint64_t)K, (uint64_t)N, (uint64_t)N, 64)
                   : make_map(&tb, B, (uint64_t)N, (uint64_t)K, (uint64_t)K, 128));
  if (!ok) return OAPL_ERR_CUDA;
  GemmParams gp;
  memset(&gp, 0, sizeof(gp));
  gp.Cdbg = C;
  gp.M = M;
  gp.N = N;
  gp.K = K;
  gp.err = err;
  gp.wait_cycles = wait_cycles;
  gp.test_skip_step = skip_step;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    // the CTA pairs meet every 32 K-steps as in the product contractions
    const int forced = env_int("OAPL_SYNC_EVERY", -1);
    if (forced != 0) {
      CK(cudaMemsetAsync(err + 1, 0, sizeof(int), st));
      gp.sync_ctr = reinterpret_cast<unsigned int*>(err + 1);
      gp.sync_every = forced > 0 ? forced : 32;
    }
  }
  const int tile_n = wide ? 2 * kBN : kBN;
  const int tiles = ((M + kTileM - 1) / kTileM) * ((N + tile_n - 1) / tile_n);
  const int grid = 2 * (tiles < n_sm / 2 ? tiles : n_sm / 2);
  if (wide) {
    if (!a_mn && !b_mn) return launch_gemm<MODE_DEBUG, 0, 0, 2>(ta, tb, ta, gp, grid, st);
    if (!a_mn && b_mn) return launch_gemm<MODE_DEBUG, 0, 1, 2>(ta, tb, ta, gp, grid, st);
    if (a_mn && !b_mn) return launch_gemm<MODE_DEBUG, 1, 0, 2>(ta, tb, ta, gp, grid, st);
    return launch_gemm<MODE_DEBUG, 1, 1, 2>(ta, tb, ta, gp, grid, st);
  }
  if (!a_mn && !b_mn) return launch_gemm<MODE_DEBUG, 0, 0>(ta, tb, ta, gp, grid, st);
  if (!a_mn && b_mn) return launch_gemm<MODE_DEBUG, 0, 1>(ta, tb, ta, gp, grid, st);
  if (a_mn && !b_mn) return launch_gemm<MODE_DEBUG, 1, 0>(ta, tb, ta, gp, grid, st);
  return launch_gemm<MODE_DEBUG, 1, 1>(ta, tb, ta, gp, grid, st);
}

// ---------------------------------------------------------------------------------------
// Token log-probabilities without a caller-provided workspace.
//
// Some callers of this library cannot hand it scratch memory because they are not allowed
// to allocate device memory at the point of the call: a plug-in running inside a host
// framework that owns the allocator, a latency-critical serving loop whose memory was fixed
// at start-up, or a region of code where the CUDA allocator must not be entered.  For them
// the scratch of oapl_token_logprobs lives in the fixed device array below (about 4.8 MB,
// resident on every GPU that loads the library until the process exits), which bounds the
// problem size: N <= 2048 rows, d <= 1024, S <= 2048 sequences, any V.
constexpr int kStaticMaxRows = 2048;
constexpr int kStaticMaxD = 1024;
constexpr int kStaticMaxSeq = 2048;
constexpr size_t kStaticScratchBytes =
    1024 /*state*/ + 4 * kSyncSlots /*lock-step counters*/ + 2 * 1024 /*block counts, offsets*/ + 7 * 4 * (size_t)kStaticMaxRows /*per-row arrays*/ +
    4 * 4 * (size_t)kStaticMaxRows * kMaxSplits /*log-sum-exp partials*/ +
    3 * 4 * (size_t)kStaticMaxSeq /*per-sequence arrays*/ +
    2 * (size_t)kStaticMaxRows * kStaticMaxD /*compacted H*/ + 16 * 1024 /*alignment slack*/;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// The array's name is only a host-side handle; kernels need its device address, which is
// looked up once per device (with that device current) and cached.
static unsigned char* g_static_scratch_addr[kMaxDevices] = {nullptr};

static int static_scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return OAPL_ERR_CUDA;
  if (!g_static_scratch_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return OAPL_ERR_CUDA;
    g_static_scratch_addr[dev] = static_cast<unsigned char*>(ptr);
  }
  *out = g_static_scratch_addr[dev];
  return OAPL_OK;
}

int oapl_token_logprobs_static(const oapl_problem* p, float* token_logp, float* seq_logp,
                               int32_t* device_status, void* stream) {
  int rc = check_problem(p, false);
  if (rc != OAPL_OK) return rc;
  if (!token_logp) return OAPL_ERR_INVALID_ARG;
  if (p->N > kStaticMaxRows || p->d > kStaticMaxD || p->S > kStaticMaxSeq) {
    fprintf(stderr,
            "oapl_token_logprobs_static: problem (N=%lld, d=%d, S=%d) exceeds the built-in scratch "
            "(N <= %d, d <= %d, S <= %d); use oapl_token_logprobs with a workspace\n",
            (long long)p->N, p->d, p->S, kStaticMaxRows, kStaticMaxD, kStaticMaxSeq);
    return OAPL_ERR_UNSUPPORTED_SHAPE;
  }
  unsigned char* base = nullptr;
  rc = static_scratch_for_current_device(&base);
  if (rc != OAPL_OK) return rc;

  // Lay the forward's scratch out inside the fixed array (1 KB-aligned pieces).
  Carve c;
  memset(&c, 0, sizeof(c));
  const size_t n_pad = align_up((size_t)p->N, 256);
  c.n_pad = (int)n_pad;
  c.nblk = (int)((p->N + kScanBlock - 1) / kScanBlock);
  c.chunk_rows = (int)n_pad;
  c.ldg = 0;
  size_t off = align_up((size_t)(uintptr_t)base, 1024) - (size_t)(uintptr_t)base;
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off = align_up(off + bytes, 1024);
    return o;
  };
  c.state = take(sizeof(DevState));
  c.sync = take(4 * (size_t)kSyncSlots);
  c.block_cnt = take(4 * (size_t)c.nblk);
  c.block_off = take(4 * (size_t)c.nblk);
  c.live_rows = take(4 * n_pad);
  c.tgt_c = take(4 * n_pad);
  c.seq_c = take(4 * n_pad);
  c.q_c = take(4 * n_pad);
  c.lp_c = take(4 * n_pad);
  c.lse = take(4 * n_pad);
  c.ent_c = take(4 * n_pad);
  c.pm = take(4 * n_pad * kMaxSplits);
  c.pl = take(4 * n_pad * kMaxSplits);
  c.pz = take(4 * n_pad * kMaxSplits);
  c.ps = take(4 * n_pad * kMaxSplits);
  c.cstart = take(4 * (size_t)p->S);
  c.cend = take(4 * (size_t)p->S);
  c.seq_D = take(4 * (size_t)p->S);
  c.Hc = take(2 * n_pad * (size_t)p->d);
  c.total = off;
  if (c.total > kStaticScratchBytes) return OAPL_ERR_UNSUPPORTED_SHAPE;

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // forward_common clears the state word and the per-sequence bounds itself; everything
  // else it reads from the scratch it has written earlier in the same call.
  rc = forward_common(p, c, base, token_logp, seq_logp, false, st);
  if (rc != OAPL_OK) return rc;
  if (device_status)
    CK(cudaMemcpyAsync(device_status, &reinterpret_cast<DevState*>(base + c.state)->status, sizeof(int),
                       cudaMemcpyDeviceToDevice, st));
  return OAPL_OK;
}

}  // extern "C"
