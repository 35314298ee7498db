// The O(N) and O(S) kernels around the contractions: live-row compaction, merge of
// the per-split log-sum-exp partials, segmented per-sequence sums, Eq. 2 and Eq. 3.
// All reductions run in a fixed order (no floating-point atomics), so results are
// bitwise reproducible from run to run.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace oapl {

constexpr int kScanBlock = 1024;

struct DevState {
  int n_live;    // live rows counted by the last forward
  int status;    // first device-detected error (0 = none)
  int fwd_tag;   // set by the forward, checked by the backward
  int reserved;
};

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

// ---- gather live rows of H into a dense [round_up(n_live,128), d] matrix ----------
__global__ void gather_rows_kernel(const __nv_bfloat16* __restrict__ H, const int* __restrict__ live_rows,
                                   const DevState* st, int d, __nv_bfloat16* __restrict__ Hc) {
  const int n_live = st->n_live;
  const int n_pad = (n_live + 127) & ~127;
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
  if (blockIdx.x == 0 && threadIdx.x == 0 && st->fwd_tag != 0x0A91) set_error(&st->status, -10);
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
__global__ void merge_lse_kernel(const float* __restrict__ pm, const float* __restrict__ pl,
                                 const float* __restrict__ pz, int C, const DevState* st,
                                 const int* __restrict__ live_rows, float* __restrict__ lse,
                                 float* __restrict__ lp_c, float* __restrict__ token_logp) {
  const int n_live = st->n_live;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_live; i += gridDim.x * blockDim.x) {
    float M = -INFINITY;
    for (int s = 0; s < C; ++s) M = fmaxf(M, pm[(size_t)i * C + s]);
    float L = 0.f, z = 0.f;
    for (int s = 0; s < C; ++s) {
      L += pl[(size_t)i * C + s] * expf(pm[(size_t)i * C + s] - M);
      z += pz[(size_t)i * C + s];
    }
    const float l = M + logf(L);
    lse[i] = l;
    lp_c[i] = z - l;
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
                                int use_q) {
  __shared__ double sh[2][8];
  const int s = blockIdx.x;
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

}  // namespace oapl
