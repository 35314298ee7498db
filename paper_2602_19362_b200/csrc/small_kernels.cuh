// The O(N) and O(S) kernels around the contractions: live-row compaction, merge of
// the per-split log-sum-exp partials, segmented per-sequence sums, Eq. 2 and Eq. 3.
// All reductions run in a fixed order (no floating-point atomics), so results are
// bitwise reproducible from run to run.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sweep_schedule.cuh"

namespace oapl {

constexpr int kScanBlock = 1024;

struct DevState {
  int n_live;    // live rows counted by the last forward
  int status;    // first device-detected error (0 = none)
  int fwd_tag;   // set by the forward, checked by the backward
  int ent_tag;   // set once the forward has left per-row entropies in the workspace
  int n_ranges;  // single call: ranges of whole sequences planned by the last call
};
constexpr int kEntTag = 0x0E27;

__device__ __forceinline__ void set_error(int* status, int code) { atomicCAS(status, 0, code); }

// ---- pass 1: per-block live counts + validation of seq_id / targets ----------
__global__ void count_live_kernel(const uint8_t* __restrict__ mask, const int* __restrict__ seq_id,
                                  const int* __restrict__ targets, long long N, int S, int V,
                                  int* __restrict__ block_cnt, int* status) {
  const long long n = (long long)blockIdx.x * kScanBlock + threadIdx.x;
  int live = 0;
  if (n < N) {
    live = mask[n] != 0;
    const int s = seq_id[n];
    if (s < 0 || s >= S || (n > 0 && s < seq_id[n - 1])) set_error(status, -6);
    if (live) {
      const int t = targets[n];
      if (t < 0 || t >= V) set_error(status, -5);
    }
  }
  const int total = __syncthreads_count(live);
  if (threadIdx.x == 0) block_cnt[blockIdx.x] = total;
}

// ---- pass 2: exclusive scan of the block counts (one CTA, fixed order) --------
__global__ void scan_blocks_kernel(const int* __restrict__ block_cnt, int nblk,
                                   int* __restrict__ block_off, DevState* st) {
  __shared__ int warp_sum[32];
  __shared__ int carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int b0 = 0; b0 < nblk; b0 += blockDim.x) {
    const int i = b0 + threadIdx.x;
    const int v = i < nblk ? block_cnt[i] : 0;
    int x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) warp_sum[warp] = x;
    __syncthreads();
    if (warp == 0) {
      int w = lane < (int)(blockDim.x >> 5) ? warp_sum[lane] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, w, o);
        if (lane >= o) w += y;
      }
      warp_sum[lane] = w;  // inclusive
    }
    __syncthreads();
    const int before = carry + (warp ? warp_sum[warp - 1] : 0) + (x - v);
    if (i < nblk) block_off[i] = before;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry = before + v;
    __syncthreads();
  }
  if (threadIdx.x == 0) st->n_live = carry;
}

// ---- pass 3: write the compacted per-row arrays --------------------------------
__global__ void write_live_kernel(const uint8_t* __restrict__ mask, const int* __restrict__ seq_id,
                                  const int* __restrict__ targets, const float* __restrict__ logp_inf,
                                  long long N, int S, const int* __restrict__ block_off,
                                  int* __restrict__ live_rows, int* __restrict__ tgt_c,
                                  int* __restrict__ seq_c, float* __restrict__ q_c) {
  __shared__ int warp_sum[32];
  const long long n = (long long)blockIdx.x * kScanBlock + threadIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int live = (n < N) && mask[n] != 0;
  const unsigned ballot = __ballot_sync(0xffffffffu, live);
  const int in_warp = __popc(ballot & ((1u << lane) - 1u));
  if (lane == 0) warp_sum[warp] = __popc(ballot);
  __syncthreads();
  if (warp == 0) {
    int w = warp_sum[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += y;
    }
    warp_sum[lane] = w;
  }
  __syncthreads();
  if (live) {
    const int i = block_off[blockIdx.x] + (warp ? warp_sum[warp - 1] : 0) + in_warp;
    live_rows[i] = (int)n;
    tgt_c[i] = targets[n];
    // an out-of-range id has already raised the error word; clamp so that no later
    // kernel indexes outside its per-sequence arrays
    seq_c[i] = min(max(seq_id[n], 0), S - 1);
    q_c[i] = logp_inf ? logp_inf[n] : 0.f;
  }
}

// ---- compacted-sequence boundaries ------------------------------------------------
__global__ void seq_bounds_kernel(const int* __restrict__ seq_c, const DevState* st,
                                  int* __restrict__ cstart, int* __restrict__ cend) {
  const int n_live = st->n_live;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_live; i += gridDim.x * blockDim.x) {
    const int s = seq_c[i];
    if (i == 0 || seq_c[i - 1] != s) cstart[s] = i;
    if (i == n_live - 1 || seq_c[i + 1] != s) cend[s] = i + 1;
  }
}

// ---- gather live rows of H into a dense [round_up(n_live,256), d] matrix ----------
__global__ void gather_rows_kernel(const __nv_bfloat16* __restrict__ H, const int* __restrict__ live_rows,
                                   const DevState* st, int d, __nv_bfloat16* __restrict__ Hc) {
  const int n_live = st->n_live;
  const int n_pad = (n_live + 255) & ~255;
  const int warps_per_block = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  const int vec = d >> 3;  // uint4 per row
  for (int i = blockIdx.x * warps_per_block + (threadIdx.x >> 5); i < n_pad;
       i += gridDim.x * warps_per_block) {
    uint4* dst = reinterpret_cast<uint4*>(Hc + (size_t)i * d);
    if (i < n_live) {
      const uint4* src = reinterpret_cast<const uint4*>(H + (size_t)live_rows[i] * d);
      for (int k = lane; k < vec; k += 32) dst[k] = __ldg(src + k);
    } else {
      for (int k = lane; k < vec; k += 32) dst[k] = make_uint4(0, 0, 0, 0);
    }
  }
}

// ---- zero the dH rows of masked positions -------------------------------------------
__global__ void zero_dead_rows_kernel(const uint8_t* __restrict__ mask, long long N, int d,
                                      __nv_bfloat16* __restrict__ dH, DevState* st) {
  if (st && blockIdx.x == 0 && threadIdx.x == 0 && st->fwd_tag != 0x0A91) set_error(&st->status, -10);
  const int warps_per_block = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  const int vec = d >> 3;
  for (long long n = (long long)blockIdx.x * warps_per_block + (threadIdx.x >> 5); n < N;
       n += (long long)gridDim.x * warps_per_block) {
    if (mask[n] == 0) {
      uint4* dst = reinterpret_cast<uint4*>(dH + (size_t)n * d);
      for (int k = lane; k < vec; k += 32) dst[k] = make_uint4(0, 0, 0, 0);
    }
  }
}

// ---- merge the per-split (max, sum-exp, target-logit) partials ----------------------
// Row i has sweep_splits_of_block(...) partials in slots [i*kMaxSplits, ...).
// Also the row's policy entropy -sum_v p ln p = lse - (sum_v e^{z-M} z) / (sum_v e^{z-M}).
__global__ void merge_lse_kernel(const float* __restrict__ pm, const float* __restrict__ pl,
                                 const float* __restrict__ pz, const float* __restrict__ ps, int R, int C,
                                 int vtiles, DevState* st, const int* __restrict__ live_rows,
                                 float* __restrict__ lse, float* __restrict__ lp_c,
                                 float* __restrict__ ent_c, float* __restrict__ token_logp) {
  const int n_live = st->n_live;
  if (blockIdx.x == 0 && threadIdx.x == 0) st->ent_tag = kEntTag;
  const int nrb = (n_live + kSweepRows - 1) / kSweepRows;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_live; i += gridDim.x * blockDim.x) {
    const int ns = sweep_splits_of_block(i / kSweepRows, nrb, R, C, vtiles);
    const size_t o = (size_t)i * kMaxSplits;
    float M = -INFINITY;
    for (int s = 0; s < ns; ++s) M = fmaxf(M, pm[o + s]);
    float L = 0.f, z = 0.f, sz = 0.f;
    for (int s = 0; s < ns; ++s) {
      const float w = expf(pm[o + s] - M);
      L += pl[o + s] * w;
      sz += ps[o + s] * w;
      z += pz[o + s];
    }
    const float l = M + logf(L);
    lse[i] = l;
    lp_c[i] = z - l;
    ent_c[i] = l - sz / L;
    if (token_logp) token_logp[live_rows[i]] = z - l;
  }
}

// ---- masked per-sequence sums: one CTA per sequence over its compacted rows ---------
__device__ __forceinline__ double warp_sum_d(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
  return x;
}

__global__ void seq_sums_kernel(const float* __restrict__ lp_c, const float* __restrict__ q_c,
                                const int* __restrict__ cstart, const int* __restrict__ cend,
                                float* __restrict__ seq_logp, float* __restrict__ seq_D,
                                int use_q, const int* __restrict__ seq_range) {
  __shared__ double sh[2][8];
  const int s = blockIdx.x;
  if (seq_range && (s < seq_range[0] || s >= seq_range[1])) return;  // whole CTA
  const int b = cstart[s], e = cend[s];
  double a_lp = 0.0, a_df = 0.0;
  // scalar head up to a 16-byte boundary, float4 body, scalar tail
  const int body_b = min(e, (b + 3) & ~3), body_e = max(body_b, e & ~3);
  for (int i = b + threadIdx.x; i < body_b; i += blockDim.x) {
    const float l = lp_c[i];
    a_lp += l;
    if (use_q) a_df += (double)l - (double)q_c[i];
  }
  for (int i = body_b + 4 * threadIdx.x; i < body_e; i += 4 * blockDim.x) {
    const float4 l = *reinterpret_cast<const float4*>(lp_c + i);
    a_lp += ((double)l.x + (double)l.y) + ((double)l.z + (double)l.w);
    if (use_q) {
      const float4 q = *reinterpret_cast<const float4*>(q_c + i);
      a_df += (((double)l.x - (double)q.x) + ((double)l.y - (double)q.y)) +
              (((double)l.z - (double)q.z) + ((double)l.w - (double)q.w));
    }
  }
  for (int i = body_e + threadIdx.x; i < e; i += blockDim.x) {
    const float l = lp_c[i];
    a_lp += l;
    if (use_q) a_df += (double)l - (double)q_c[i];
  }
  a_lp = warp_sum_d(a_lp);
  a_df = warp_sum_d(a_df);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { sh[0][warp] = a_lp; sh[1][warp] = a_df; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double t0 = 0.0, t1 = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { t0 += sh[0][w]; t1 += sh[1][w]; }
    if (seq_logp) seq_logp[s] = (float)t0;
    if (seq_D) seq_D[s] = (float)t1;
  }
}

// ---- Eq. 2: one warp per group ---------------------------------------------------------
__global__ void value_estimate_kernel(const float* __restrict__ reward, const int* __restrict__ group_id,
                                      int S, int P, float beta_v, float* __restrict__ vhat,
                                      int* status) {
  const int p = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (p >= P) return;
  float rmax = -INFINITY;
  int cnt = 0;
  for (int i = lane; i < S; i += 32) {
    const int g = group_id[i];
    const float r = reward[i];
    if (status && p == 0 && (g < 0 || g >= P || !isfinite(r))) set_error(status, -7);
    if (g == p) { rmax = fmaxf(rmax, r); ++cnt; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, o));
    cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  }
  if (cnt == 0) {
    if (lane == 0) vhat[p] = 0.f;
    return;
  }
  double acc = 0.0;
  for (int i = lane; i < S; i += 32)
    if (group_id[i] == p) acc += exp(((double)reward[i] - (double)rmax) / (double)beta_v);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) vhat[p] = (float)((double)rmax + (double)beta_v * log(acc / (double)cnt));
}

// ---- Eq. 3: advantage, residual, loss, coefficient (one CTA, fixed order) -------------
__global__ void loss_kernel(const float* __restrict__ reward, const int* __restrict__ group_id,
                            const float* __restrict__ vhat, const float* __restrict__ seq_D, int S,
                            int P, float beta_loss, float loss_scale, float* __restrict__ coef,
                            float* __restrict__ delta_out, float* __restrict__ loss, DevState* st) {
  __shared__ double sh[32];
  double acc = 0.0;
  for (int i = threadIdx.x; i < S; i += blockDim.x) {
    const int g = group_id[i];
    const float vh = (g >= 0 && g < P) ? vhat[g] : 0.f;
    const double A = (double)reward[i] - (double)vh;
    const double dl = (double)beta_loss * (double)seq_D[i] - A;
    coef[i] = (float)(2.0 * (double)loss_scale * (double)beta_loss * dl);
    if (delta_out) delta_out[i] = (float)dl;
    acc += dl * dl;
  }
  acc = warp_sum_d(acc);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) sh[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += sh[w];
    *loss = (float)((double)loss_scale * t);
    st->fwd_tag = 0x0A91;  // = kFwdTag of the contraction kernel
  }
}

// =====================================================================================
// Kernels of the single-call forward+backward path, which stages e = exp(z - zref) for a
// range of whole sequences instead of recomputing the logits in the backward.
// =====================================================================================
struct RangeRec {
  int row_begin, row_end;  // compacted rows
  int seq_begin, seq_end;  // sequences whose live rows lie in the range (plus empty ones between)
};

// zref[i] = h_i . w_{y_i} + 40: a per-row reference close enough to the row's largest
// logit that exp(z - zref) neither overflows (needs z_max - z_y < 128) nor loses the
// dominant terms (z_max >= z_y, so they are >= e^-40).  One warp per live row.
constexpr float kRefShift = 40.f;
__global__ void ztgt_kernel(const __nv_bfloat16* __restrict__ Hc, const __nv_bfloat16* __restrict__ W,
                            const int* __restrict__ tgt_c, const DevState* st, int d, int V,
                            float* __restrict__ zref) {
  const int n_live = st->n_live;
  const int warps_per_block = blockDim.x >> 5, lane = threadIdx.x & 31;
  for (int i = blockIdx.x * warps_per_block + (threadIdx.x >> 5); i < n_live;
       i += gridDim.x * warps_per_block) {
    const int t = min(max(tgt_c[i], 0), V - 1);  // a bad target has already raised the error word
    const uint4* h = reinterpret_cast<const uint4*>(Hc + (size_t)i * d);
    const uint4* w = reinterpret_cast<const uint4*>(W + (size_t)t * d);
    float acc = 0.f;
    for (int k = lane; k < (d >> 3); k += 32) {
      const uint4 a = h[k], b = __ldg(w + k);
      const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
      const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 x = __bfloat1622float2(pa[q]), y = __bfloat1622float2(pb[q]);
        acc = fmaf(x.x, y.x, acc);
        acc = fmaf(x.y, y.y, acc);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) zref[i] = acc + kRefShift;
  }
}

// Greedy packing of consecutive sequences into ranges of at most stage_rows live rows.
// One thread; S is small.  The n ranges found occupy the LAST n of the max_ranges records (in
// order), the records before them are left empty: the host enqueues max_ranges range slots
// without knowing n, and the last slot is then always the last range.  A sequence longer
// than stage_rows cannot be staged (-11), and more ranges than records means the caller's
// bounds on the live rows were too small (-13): the error word is raised and no range is
// produced.
__global__ void plan_ranges_kernel(const int* __restrict__ cstart, const int* __restrict__ cend, int S,
                                   int stage_rows, int max_ranges, RangeRec* __restrict__ ranges,
                                   DevState* st) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  for (int pass = 0; pass < 2; ++pass) {
    // pass 0 counts the ranges, pass 1 writes them behind the empty records
    int n = 0, rb = -1, re = 0, sb = 0;
    const int shift = pass == 0 ? 0 : max_ranges - st->n_ranges;
    for (int s = 0; s < S; ++s) {
      const int b = cstart[s], e = cend[s];
      if (e <= b) continue;
      if (e - b > stage_rows) {
        for (int k = 0; k < max_ranges; ++k) ranges[k] = RangeRec{0, 0, 0, 0};
        set_error(&st->status, -11);
        st->n_ranges = 0;
        return;
      }
      if (rb < 0) { rb = b; sb = s; }
      if (e - rb > stage_rows) {  // close the open range before this sequence
        if (pass) ranges[shift + n] = RangeRec{rb, re, sb, s};
        ++n;
        rb = b;
        sb = s;
      }
      re = e;
    }
    if (rb >= 0) {
      if (pass) ranges[shift + n] = RangeRec{rb, re, sb, S};
      ++n;
    }
    if (pass == 0) {
      if (n > max_ranges) {
        for (int k = 0; k < max_ranges; ++k) ranges[k] = RangeRec{0, 0, 0, 0};
        set_error(&st->status, -13);
        st->n_ranges = 0;
        return;
      }
      st->n_ranges = n;
      for (int k = 0; k < max_ranges - n; ++k) ranges[k] = RangeRec{0, 0, 0, 0};
    }
  }
}

// lse = zref + ln(sum_v e), token log-prob, and alpha = exp(zref - lse) = 1 / sum_v e.
__global__ void merge_e_kernel(const float* __restrict__ pl, const float* __restrict__ pz,
                               const float* __restrict__ ps, const float* __restrict__ zref,
                               const RangeRec* __restrict__ range, int R, int C, int vtiles,
                               const int* __restrict__ live_rows, float* __restrict__ lse,
                               float* __restrict__ lp_c, float* __restrict__ ent_c,
                               float* __restrict__ alpha, float* __restrict__ ztc,
                               float* __restrict__ token_logp, DevState* st) {
  const int rb = range->row_begin, re = range->row_end;
  if (blockIdx.x == 0 && threadIdx.x == 0) st->ent_tag = kEntTag;
  const int nrb = (re - rb + kSweepRows - 1) / kSweepRows;
  for (int i = rb + blockIdx.x * blockDim.x + threadIdx.x; i < re; i += gridDim.x * blockDim.x) {
    const int ns = sweep_splits_of_block((i - rb) / kSweepRows, nrb, R, C, vtiles);
    const size_t o = (size_t)i * kMaxSplits;
    float L = 0.f, z = 0.f, sz = 0.f;
    for (int s = 0; s < ns; ++s) {
      L += pl[o + s];
      sz += ps[o + s];
      z += pz[o + s];
    }
    // the per-row reference is the target logit + 40: a sum that is not a positive finite
    // number means some logit was more than ~128 above the target's (or the inputs are not finite)
    if (!(L > 0.f) || !isfinite(L)) set_error(&st->status, -12);
    const float l = zref[i] + logf(L);
    lse[i] = l;
    ent_c[i] = l - sz / L;
    ztc[i] = z;
    alpha[i] = 1.f / L;
    lp_c[i] = z - l;
    if (token_logp) token_logp[live_rows[i]] = z - l;
  }
}

// Coefficients c_i = 2 lambda beta_loss delta_i of the sequences of one range.
__global__ void coef_range_kernel(const float* __restrict__ reward, const int* __restrict__ group_id,
                                  const float* __restrict__ vhat, const float* __restrict__ seq_D,
                                  const RangeRec* __restrict__ range, int P, float beta_loss,
                                  float loss_scale, float* __restrict__ coef) {
  for (int i = range->seq_begin + blockIdx.x * blockDim.x + threadIdx.x; i < range->seq_end;
       i += gridDim.x * blockDim.x) {
    const int g = group_id[i];
    const float vh = (g >= 0 && g < P) ? vhat[g] : 0.f;
    const double A = (double)reward[i] - (double)vh;
    const double dl = (double)beta_loss * (double)seq_D[i] - A;
    coef[i] = (float)(2.0 * (double)loss_scale * (double)beta_loss * dl);
  }
}

// With s_n = -c_n * alpha_n:  g[n,v] = s_n * e'[n,v], where e' is e with the target entry
// replaced by e_y - 1/alpha = (p_y - 1)/alpha.  So dH = rowscale(e'.W) and dW = e'^T.(s o H):
// this kernel writes Hs = bf16(s_n H_n), the row scales, and patches the target entries.
// Rows between the range end and the next multiple of 256 get zero Hs rows (the dW
// contraction reads whole 64-row slabs).  One warp per row.
// The coefficient is the row's own (coef_row, token-level objectives) or its sequence's.
__global__ void scale_patch_kernel(const __nv_bfloat16* __restrict__ Hc, const int* __restrict__ seq_c,
                                   const int* __restrict__ tgt_c, const float* __restrict__ coef,
                                   const float* __restrict__ coef_row,
                                   const float* __restrict__ alpha, const float* __restrict__ lse,
                                   const float* __restrict__ ztc, const RangeRec* __restrict__ range,
                                   int d, int V, int ldg, __nv_bfloat16* __restrict__ Hs,
                                   float* __restrict__ rowscale, __nv_bfloat16* __restrict__ E) {
  const int rb = range->row_begin, re = range->row_end;
  const int pad_end = rb + ((re - rb + 255) & ~255);
  const int warps_per_block = blockDim.x >> 5, lane = threadIdx.x & 31;
  const int vec = d >> 3;
  for (int i = rb + blockIdx.x * warps_per_block + (threadIdx.x >> 5); i < pad_end;
       i += gridDim.x * warps_per_block) {
    uint4* dst = reinterpret_cast<uint4*>(Hs + (size_t)i * d);
    if (i < re) {
      const float a = alpha[i];
      const float s = -(coef_row ? coef_row[i] : coef[seq_c[i]]) * a;
      const uint4* src = reinterpret_cast<const uint4*>(Hc + (size_t)i * d);
      for (int k = lane; k < vec; k += 32) {
        uint4 x = src[k];
        __nv_bfloat162* px = reinterpret_cast<__nv_bfloat162*>(&x);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float2 f = __bfloat1622float2(px[q]);
          px[q] = __floats2bfloat162_rn(s * f.x, s * f.y);
        }
        dst[k] = x;
      }
      if (lane == 0) {
        rowscale[i] = s;
        const int t = tgt_c[i];
        if (t >= 0 && t < V)
          E[(size_t)(i - rb) * ldg + t] = __float2bfloat16_rn(expm1f(ztc[i] - lse[i]) / a);
      }
    } else {
      for (int k = lane; k < vec; k += 32) dst[k] = make_uint4(0, 0, 0, 0);
    }
  }
}

// =====================================================================================
// GRPO with token-level importance weights (the paper's baseline objective, the display
// in its Background section) on the same staged-exponential pipeline.
// =====================================================================================
// Group-normalised advantage: A_i = (r_i - mean_p) / (std_p + eps) over the members of the
// sequence's group p (population standard deviation).  One warp per group, then the members
// are written by the same warp.  A group without members writes nothing.
__global__ void group_advantage_kernel(const float* __restrict__ reward, const int* __restrict__ group_id,
                                       int S, int P, float eps, float* __restrict__ adv) {
  const int p = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (p >= P) return;
  double sum = 0.0;
  int cnt = 0;
  for (int i = lane; i < S; i += 32)
    if (group_id[i] == p) { sum += (double)reward[i]; ++cnt; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    sum += __shfl_xor_sync(0xffffffffu, sum, o);
    cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
  }
  if (cnt == 0) return;
  const double mean = sum / (double)cnt;
  double ss = 0.0;
  for (int i = lane; i < S; i += 32)
    if (group_id[i] == p) { const double dlt = (double)reward[i] - mean; ss += dlt * dlt; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const double sd = sqrt(ss / (double)cnt);
  for (int i = lane; i < S; i += 32)
    if (group_id[i] == p) adv[i] = (float)(((double)reward[i] - mean) / (sd + (double)eps));
}

// Compaction of one more per-row float array (the previous policy's log-probs).
__global__ void gather_f32_kernel(const float* __restrict__ src, const int* __restrict__ live_rows,
                                  const DevState* st, float* __restrict__ dst) {
  const int n_live = st->n_live;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_live; i += gridDim.x * blockDim.x)
    dst[i] = src[live_rows[i]];
}

// One CTA per sequence of the range.  Per response token, with r = exp(lp - lp_old),
// w = exp(lp_old - lp_inf) (data) and the sequence's advantage A:
//     term  = w * min(r A, clip(r, 1-eps, 1+eps) A)
//     coef  = dLoss/dlp = -lambda/|y| * w * A * r   where the unclipped branch is the minimum,
//             0 where the clipped (constant) branch is.
// Writes the per-row coefficients and, per sequence, (1/|y|) sum_t term and the number of
// tokens on the clipped branch; fixed reduction order.
__global__ void grpo_coef_kernel(const float* __restrict__ lp_c, const float* __restrict__ qold_c,
                                 const float* __restrict__ qinf_c, const int* __restrict__ cstart,
                                 const int* __restrict__ cend, const float* __restrict__ adv,
                                 const int* __restrict__ seq_range, float clip_eps, float loss_scale,
                                 float* __restrict__ coef_row, float* __restrict__ seq_obj,
                                 int* __restrict__ seq_clipped) {
  __shared__ double sh[8];
  __shared__ int shc[8];
  const int s = blockIdx.x;
  if (s < seq_range[0] || s >= seq_range[1]) return;  // whole CTA
  const int b = cstart[s], e = cend[s];
  const double A = (double)adv[s];
  const double inv_len = e > b ? 1.0 / (double)(e - b) : 0.0;
  const double lo = 1.0 - (double)clip_eps, hi = 1.0 + (double)clip_eps;
  double acc = 0.0;
  int nclip = 0;
  for (int i = b + threadIdx.x; i < e; i += blockDim.x) {
    const double lp = (double)lp_c[i], lo_ = (double)qold_c[i];
    const double r = exp(lp - lo_);
    const double w = exp(lo_ - (double)qinf_c[i]);
    const double rc = fmin(fmax(r, lo), hi);
    const double t_un = r * A, t_cl = rc * A;
    const bool unclipped = t_un <= t_cl;
    acc += w * (unclipped ? t_un : t_cl);
    nclip += unclipped ? 0 : 1;
    coef_row[i] = unclipped ? (float)(-(double)loss_scale * inv_len * w * A * r) : 0.f;
  }
  acc = warp_sum_d(acc);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) nclip += __shfl_down_sync(0xffffffffu, nclip, o);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { sh[warp] = acc; shc[warp] = nclip; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    int n = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { t += sh[w]; n += shc[w]; }
    seq_obj[s] = (float)(t * inv_len);
    seq_clipped[s] = n;
  }
}

// loss = -lambda * sum_i seq_obj[i];  clip_frac = clipped tokens / response tokens.
__global__ void grpo_loss_kernel(const float* __restrict__ seq_obj, const int* __restrict__ seq_clipped,
                                 int S, float loss_scale, float* __restrict__ loss,
                                 float* __restrict__ clip_frac, DevState* st) {
  __shared__ double sh[8];
  __shared__ long long shc[8];
  double acc = 0.0;
  long long n = 0;
  for (int i = threadIdx.x; i < S; i += blockDim.x) { acc += (double)seq_obj[i]; n += seq_clipped[i]; }
  acc = warp_sum_d(acc);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) n += __shfl_down_sync(0xffffffffu, n, o);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { sh[warp] = acc; shc[warp] = n; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    long long c = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { t += sh[w]; c += shc[w]; }
    *loss = (float)(-(double)loss_scale * t);
    if (clip_frac) *clip_frac = st->n_live > 0 ? (float)((double)c / (double)st->n_live) : 0.f;
  }
}

// =====================================================================================
// Batch diagnostics from what a loss forward left in the workspace (one CTA, fixed order).
// =====================================================================================
// stats[0] live tokens, [1] mean |D_i| and [2] max |D_i| over the sequences with response tokens,
// [3] sum D_i / live tokens, [4] mean advantage r_i - vhat[g_i], [5] fraction of the groups with
// members whose rewards are all equal, [6] mean reward, [7] 0.
constexpr int kStatsCount = 8;
__global__ void batch_stats_kernel(const float* __restrict__ seq_D, const int* __restrict__ cstart,
                                   const int* __restrict__ cend, const float* __restrict__ reward,
                                   const int* __restrict__ group_id, const float* __restrict__ vhat, int S, int P,
                                   DevState* st, float* __restrict__ stats) {
  __shared__ double sh[4][8];
  __shared__ float shmax[8];
  __shared__ int shcnt[3][8];
  if (st->fwd_tag != 0x0A91) {
    if (threadIdx.x == 0) set_error(&st->status, -10);
    return;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  double sum_abs = 0.0, sum_d = 0.0, sum_adv = 0.0, sum_r = 0.0;
  float max_abs = 0.f;
  int n_seq_live = 0;
  for (int i = threadIdx.x; i < S; i += blockDim.x) {
    const float r = reward[i];
    const int g = group_id[i];
    sum_r += (double)r;
    sum_adv += (double)r - (double)((g >= 0 && g < P) ? vhat[g] : 0.f);
    if (cend[i] > cstart[i]) {
      const float dd = seq_D[i];
      sum_abs += fabs((double)dd);
      sum_d += (double)dd;
      max_abs = fmaxf(max_abs, fabsf(dd));
      ++n_seq_live;
    }
  }
  // groups: one warp per group in turn; all-equal when the members' minimum equals their maximum
  int n_groups = 0, n_equal = 0;
  for (int p = warp; p < P; p += nwarps) {
    float lo = INFINITY, hi = -INFINITY;
    for (int i = lane; i < S; i += 32)
      if (group_id[i] == p) { lo = fminf(lo, reward[i]); hi = fmaxf(hi, reward[i]); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (hi >= lo) { ++n_groups; n_equal += (hi == lo) ? 1 : 0; }   // same value in every lane
  }
  sum_abs = warp_sum_d(sum_abs);
  sum_d = warp_sum_d(sum_d);
  sum_adv = warp_sum_d(sum_adv);
  sum_r = warp_sum_d(sum_r);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    max_abs = fmaxf(max_abs, __shfl_down_sync(0xffffffffu, max_abs, o));
    n_seq_live += __shfl_down_sync(0xffffffffu, n_seq_live, o);
  }
  if (lane == 0) {
    sh[0][warp] = sum_abs; sh[1][warp] = sum_d; sh[2][warp] = sum_adv; sh[3][warp] = sum_r;
    shmax[warp] = max_abs;
    shcnt[0][warp] = n_seq_live; shcnt[1][warp] = n_groups; shcnt[2][warp] = n_equal;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double t[4] = {0.0, 0.0, 0.0, 0.0};
    float mx = 0.f;
    int c[3] = {0, 0, 0};
    for (int w = 0; w < nwarps; ++w) {
      for (int k = 0; k < 4; ++k) t[k] += sh[k][w];
      mx = fmaxf(mx, shmax[w]);
      for (int k = 0; k < 3; ++k) c[k] += shcnt[k][w];
    }
    const int n_live = st->n_live;
    stats[0] = (float)n_live;
    stats[1] = c[0] > 0 ? (float)(t[0] / (double)c[0]) : 0.f;
    stats[2] = mx;
    stats[3] = n_live > 0 ? (float)(t[1] / (double)n_live) : 0.f;
    stats[4] = S > 0 ? (float)(t[2] / (double)S) : 0.f;
    stats[5] = c[1] > 0 ? (float)((double)c[2] / (double)c[1]) : 0.f;
    stats[6] = S > 0 ? (float)(t[3] / (double)S) : 0.f;
    stats[7] = 0.f;
  }
}

// =====================================================================================
// Policy-entropy statistic read back from what a forward left in the workspace.
// =====================================================================================
// One CTA per sequence: mean of the per-row entropies over the sequence's response tokens
// (0 for a sequence without any), and the scatter of the per-row values to their rows.
__global__ void entropy_seq_kernel(const float* __restrict__ ent_c, const int* __restrict__ cstart,
                                   const int* __restrict__ cend, const int* __restrict__ live_rows,
                                   float* __restrict__ token_entropy, float* __restrict__ seq_entropy,
                                   DevState* st) {
  __shared__ double sh[8];
  if (st->ent_tag != kEntTag) {
    if (blockIdx.x == 0 && threadIdx.x == 0) set_error(&st->status, -10);
    return;
  }
  const int s = blockIdx.x;
  const int b = cstart[s], e = cend[s];
  double acc = 0.0;
  for (int i = b + threadIdx.x; i < e; i += blockDim.x) {
    const float h = ent_c[i];
    acc += h;
    if (token_entropy) token_entropy[live_rows[i]] = h;
  }
  acc = warp_sum_d(acc);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) sh[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0 && seq_entropy) {
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += sh[w];
    seq_entropy[s] = e > b ? (float)(t / (double)(e - b)) : 0.f;
  }
}

// Mean over all response tokens of the batch (one CTA, fixed order; 0 when none is live).
__global__ void entropy_mean_kernel(const float* __restrict__ ent_c, const DevState* st,
                                    float* __restrict__ mean_entropy) {
  __shared__ double sh[32];
  if (st->ent_tag != kEntTag) return;
  const int n_live = st->n_live;
  double acc = 0.0;
  for (int i = threadIdx.x; i < n_live; i += blockDim.x) acc += ent_c[i];
  acc = warp_sum_d(acc);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) sh[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += sh[w];
    *mean_entropy = n_live > 0 ? (float)(t / (double)n_live) : 0.f;
  }
}

}  // namespace oapl
