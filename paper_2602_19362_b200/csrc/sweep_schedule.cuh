// Schedule of the vocabulary-sweep kernels, shared by the contraction kernel (which
// walks it) and the merge kernels (which need to know how many partial results a row has).
//
// The rows of a range are cut into 256-row blocks (one per CTA pair).  A wave is R row
// blocks x C vocabulary splits = R*C CTA pairs, each sweeping its split's vocabulary tiles
// for one row block.  The last, incomplete wave (rem < R row blocks) is re-split into Ct >= C
// vocabulary splits so that it still occupies (almost) every CTA for a proportionally
// shorter time instead of leaving most of them idle.
#pragma once

namespace oapl {

constexpr int kMaxSplits = 16;
constexpr int kSweepRows = 256;  // rows per row block of the sweep

struct SweepShape {
  int nfull;  // complete waves
  int rem;    // row blocks in the tail wave (0 = none)
  int Ct;     // vocabulary splits of the tail wave
};

__host__ __device__ inline SweepShape sweep_shape(int n_row_blocks, int R, int C, int vtiles) {
  SweepShape s;
  s.nfull = n_row_blocks / R;
  s.rem = n_row_blocks - s.nfull * R;
  s.Ct = 0;
  if (s.rem) {
    int ct = (R * C) / s.rem;
    if (ct > kMaxSplits) ct = kMaxSplits;
    if (ct > vtiles) ct = vtiles;
    if (ct < 1) ct = 1;
    s.Ct = ct;
  }
  return s;
}

// Number of vocabulary splits (= partial results per row) of row block `rbk` of the range.
__host__ __device__ inline int sweep_splits_of_block(int rbk, int n_row_blocks, int R, int C, int vtiles) {
  const SweepShape s = sweep_shape(n_row_blocks, R, C, vtiles);
  return rbk < s.nfull * R ? C : s.Ct;
}

}  // namespace oapl
