// Carrying the state across time segments (Appendix D: a sequence too long for on-chip memory is scanned chunk by
// chunk, each chunk continuing from the scan state the previous one ended in).
//
// A segment g that starts from a zero state ends in a local state e_g, and multiplies whatever state it was given by
// P_g = prod_t a_t = exp(A_n * sum_{t in g} delta_t).  The true state before segment g+1 is therefore
//     H_{g+1} = P_g * H_g + e_g,   H_0 = the caller's initial state (zero if none),
// i.e. an exclusive scan over segments of the pairs (P_g, e_g) under the operator
// (a, b) o (a', b') = (a a', a' b + b').  The adjoint that flows backwards through the segments obeys the same law
// in reversed order, with the same P_g.
//
// One block owns 32 adjacent (channel, state) columns of one batch entry.  threadIdx.x is the column (coalesced
// access), threadIdx.y is a contiguous range of segments: each thread folds its range with the operator, the range
// aggregates are scanned across the block through shared memory, and a second sweep writes the carried values.
#include "ssm_common.cuh"

namespace ssm {

constexpr int kCarryCols = 32;
constexpr int kCarryRanges = 8;

__global__ void __launch_bounds__(kCarryCols* kCarryRanges) ssm_carry_kernel(const CarryParams p) {
  __shared__ AffinePair s_agg[kCarryRanges][kCarryCols];
  const int col = blockIdx.x * kCarryCols + threadIdx.x;  // index into D*N
  const int b = blockIdx.y;
  const int r = threadIdx.y;
  const int DN = p.D * p.N;
  const bool valid = col < DN;
  const int d = valid ? col / p.N : 0;
  const float A2 = valid ? p.A[col] * kLog2e : 0.f;

  const int per = (p.nseg + kCarryRanges - 1) / kCarryRanges;
  const int i0 = min(p.nseg, r * per), i1 = min(p.nseg, i0 + per);  // positions in scan order
  auto seg_of = [&](int i) { return p.reverse ? p.nseg - 1 - i : i; };

  AffinePair agg{1.f, 0.f};
  if (valid) {
    for (int i = i0; i < i1; ++i) {
      const size_t sg = (size_t)b * p.nseg + seg_of(i);
      const AffinePair e{ex2_approx(A2 * p.dsum[sg * p.D + d]), p.local[sg * DN + col]};
      agg = combine(agg, e);
    }
  }
  s_agg[r][threadIdx.x] = agg;
  __syncthreads();
  // everything before this thread's range, starting from what flows into the first segment
  AffinePair pre{1.f, (valid && p.init != nullptr) ? p.init[(size_t)b * DN + col] : 0.f};
  for (int rr = 0; rr < r; ++rr) pre = combine(pre, s_agg[rr][threadIdx.x]);
  if (valid) {
    float carry = pre.b;  // exclusive scan
    for (int i = i0; i < i1; ++i) {
      const size_t sg = (size_t)b * p.nseg + seg_of(i);
      p.carried[sg * DN + col] = carry;
      carry = fmaf(ex2_approx(A2 * p.dsum[sg * p.D + d]), carry, p.local[sg * DN + col]);
    }
  }
}

cudaError_t launch_carry(const CarryParams& p, cudaStream_t s) {
  dim3 grid((p.D * p.N + kCarryCols - 1) / kCarryCols, p.batch);
  dim3 block(kCarryCols, kCarryRanges);
  ssm_carry_kernel<<<grid, block, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace ssm
