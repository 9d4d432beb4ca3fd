// C ABI of the selective-scan library: argument validation, the time-split plan, the workspace layout and the
// launch sequences.  See include/ssm_scan.h for the contract of every entry point.
#include <algorithm>

#include "ssm_common.cuh"

namespace ssm {

int fwd_channels_per_block(int N);
int bwd_channels_per_block(int N);
bool complex_supported(const ssm_problem_t& p);
size_t complex_bwd_workspace_bytes(const ssm_problem_t& p);
size_t complex_saved_state_bytes(const ssm_problem_t& p);
cudaError_t complex_fwd(const ssm_problem_t& prob, const void* x, const void* delta, const float* A, const void* B,
                        const void* C, const float* D_skip, const void* z, const float* h0, void* out, float* h_last,
                        void* saved_states, cudaStream_t s);
cudaError_t complex_bwd(const ssm_problem_t& prob, const void* x, const void* delta, const float* A, const void* B,
                        const void* C, const float* D_skip, const void* z, const void* dout, const float* h0,
                        const float* dh_last, const void* saved_states, void* dx, void* ddelta, float* dA, void* dB,
                        void* dC, float* dD, void* dz, float* dh0, void* workspace, cudaStream_t s);
cudaError_t complex_step(const ssm_problem_t& prob, const void* x, const void* delta, const float* A, const void* B,
                         const void* C, const float* D_skip, const void* z, float* h, void* out, cudaStream_t s);
bool bwd_local_fast_applicable(const ssm_problem_t& prob, const BwdParams& p);
int fwd_states_per_thread();
int fwd_fast_channels_per_warp();
int bwd_fast_channels_per_warp();
bool bwd_fast_applicable(const ssm_problem_t& prob, const BwdParams& p);
// ssm_repack.cu
enum { kRepackBf16 = 0, kRepackF32 = 1, kRepackA = 2 };
constexpr int kRepackMax = 6;
struct RepackJob {
  const void* src;
  void* dst;
  int rows, n_src, n_dst, kind;
};
struct RepackJobs {
  RepackJob job[kRepackMax];
  int count;
};
void repack_add(RepackJobs& jobs, const void* src, void* dst, long long rows, int n_src, int n_dst, int kind);
cudaError_t repack_run(const RepackJobs& jobs, cudaStream_t s);
size_t fwd_handoff_bytes_per_worker();
size_t bwd_handoff_bytes_per_worker(bool static_B, bool static_C);

// Shapes the tuned warp-per-worker kernels take (they also want 16-byte aligned pointers, checked per call).
static bool tuned_shape(const ssm_problem_t& p) {
  const bool static_bc = p.flags & (SSM_FLAG_STATIC_B | SSM_FLAG_STATIC_C);
  return p.io_dtype == SSM_BF16 && p.N == 16 && p.D % 8 == 0 && !(p.flags & SSM_FLAG_COMPLEX) &&
         !(static_bc && (p.flags & SSM_FLAG_ZOH_BBAR));   // non-selective B / C: tuned with the default B-bar rule only
}
// Workers the hand-off slots of a workspace allow for `chains` chains: none while every chain can have a warp of its
// own in the first round (one warp per SM sub-partition); else at least two rounds (a kernel may share chains between
// more warps than there are chains) and at most 12 resident warps per SM.
constexpr int kMaxWarpsPerSM = 12;
static int shared_workers(long long chains) {
  if (chains <= 4LL * kNumSMs) return 0;
  return (int)std::min<long long>(std::max<long long>(chains, 8LL * kNumSMs), (long long)kMaxWarpsPerSM * kNumSMs);
}

constexpr size_t kStatusBytes = 256;   // head of every workspace: the status word
static inline size_t align_up(size_t v) { return (v + 255) & ~(size_t)255; }

// bf16 problems with fewer than 16 states run as 16-state problems on the tuned kernels, with A, B, C (and the state
// arrays) widened by columns that stay zero (ssm_repack.cu); `wide` is that problem.
constexpr int kWideN = 16;
static bool widen_route(const ssm_problem_t& p, ssm_problem_t* wide) {
  if (p.io_dtype != SSM_BF16 || p.N >= kWideN || p.D % 8 != 0 || (p.flags & SSM_FLAG_COMPLEX)) return false;
  if ((long long)p.batch * p.L > 0x7fffffffLL || (long long)p.batch * p.D > 0x7fffffffLL) return false;
  if (wide) {
    *wide = p;
    wide->N = kWideN;
  }
  return true;
}
// Buffers of the widened arrays, placed behind the wide problem's own workspace (whose head holds the status word).
struct WidenLayout {
  size_t A, B, C, h0, h_last, dh_last, dA, dB, dC, dh0, total;
};
static WidenLayout widen_layout(const ssm_problem_t& p, size_t inner_bytes, bool bwd) {
  WidenLayout w{};
  size_t off = align_up(inner_bytes > (size_t)kStatusBytes ? inner_bytes : (size_t)kStatusBytes);
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off += align_up(bytes);
    return at;
  };
  const size_t rows_t = (size_t)p.batch * p.L, rows_s = (size_t)p.batch * p.D;
  const size_t bsz = (p.flags & SSM_FLAG_STATIC_B) ? (size_t)p.D * kWideN * sizeof(float) : rows_t * kWideN * 2;
  const size_t csz = (p.flags & SSM_FLAG_STATIC_C) ? (size_t)p.D * kWideN * sizeof(float) : rows_t * kWideN * 2;
  w.A = take((size_t)p.D * kWideN * sizeof(float));
  w.B = take(bsz);
  w.C = take(csz);
  w.h0 = take(rows_s * kWideN * sizeof(float));
  if (!bwd) {
    w.h_last = take(rows_s * kWideN * sizeof(float));
  } else {
    w.dh_last = take(rows_s * kWideN * sizeof(float));
    w.dA = take((size_t)p.D * kWideN * sizeof(float));
    w.dB = take(bsz);
    w.dC = take(csz);
    w.dh0 = take(rows_s * kWideN * sizeof(float));
  }
  w.total = off;
  return w;
}

static ssm_status_t validate_problem(const ssm_problem_t* p) {
  if (p == nullptr) return SSM_ERR_INVALID_ARG;
  if (p->batch < 1 || p->L < 1 || p->D < 1 || p->N < 1) return SSM_ERR_INVALID_ARG;
  if (p->flags & ~(uint32_t)(SSM_FLAG_HAS_Z | SSM_FLAG_HAS_DSKIP | SSM_FLAG_SAVE_STATES | SSM_FLAG_GENERAL_A | SSM_FLAG_TEST_WITHHOLD |
                             SSM_FLAG_DELTA_SOFTPLUS | SSM_FLAG_ZOH_BBAR | SSM_FLAG_STATIC_B | SSM_FLAG_STATIC_C | SSM_FLAG_COMPLEX))
    return SSM_ERR_INVALID_ARG;
  if (p->io_dtype != SSM_F32 && p->io_dtype != SSM_BF16) return SSM_ERR_UNSUPPORTED;
  if (p->N != 1 && p->N != 2 && p->N != 4 && p->N != 8 && p->N != 16 && p->N != 32 && p->N != 64) return SSM_ERR_UNSUPPORTED;
  if (p->batch > 65535) return SSM_ERR_UNSUPPORTED;  // batch is a grid z dimension
  if ((p->flags & SSM_FLAG_COMPLEX) && !complex_supported(*p)) return SSM_ERR_UNSUPPORTED;
  return SSM_OK;
}

// The sequence is split in time only when (batch, channel, state) parallelism alone would leave most of the GPU
// idle: every time segment but the first costs one extra sweep of the recurrence.
Plan make_plan(const ssm_problem_t& p) {
  Plan pl{};
  pl.nck = (p.L + kCkptSteps - 1) / kCkptSteps;
  pl.fwd_cpt = 2;
  pl.fwd_ch = fwd_channels_per_block(p.N);
  pl.bwd_ch = bwd_channels_per_block(p.N);
  pl.bwd_groups = (p.D + pl.bwd_ch - 1) / pl.bwd_ch;
  const int S = p.N < 4 ? p.N : 4;
  const long long groups = (long long)p.batch * ((p.D + pl.fwd_cpt - 1) / pl.fwd_cpt);  // thread groups
  const long long warps = std::max<long long>(1, groups * (p.N / S) / 32);
  const long long sub_partitions = 4LL * kNumSMs;
  int nseg = 1;
  if (p.flags & SSM_FLAG_COMPLEX) {
    // the complex path does not split time
  } else if (tuned_shape(p)) {
    // one warp per chain of fwd_fast_channels_per_warp() channels; a split costs half a forward sweep more, so only
    // when fewer than half of the sub-partitions would have a warp, and then into two rounds of chains
    const int cw = fwd_fast_channels_per_warp();
    const long long chains = (long long)p.batch * ((p.D + cw - 1) / cw);
    if (2 * chains < sub_partitions) {
      const long long want = (2 * sub_partitions + chains - 1) / chains;
      const long long max_by_len = std::max(1, p.L / 256);
      nseg = (int)std::min<long long>(std::min(want, max_by_len), 65535);
    }
  } else if (warps < sub_partitions * 3) {
    // generic kernels: a warp is latency-bound, so aim for 6 warps per sub-partition although a split costs half a
    // sweep more (measured 2 to 2.5 times faster than one or two warps per sub-partition)
    const long long want = (6 * sub_partitions + warps - 1) / warps;
    const long long max_by_len = std::max(1, p.L / 256);
    nseg = (int)std::min<long long>(std::min(want, max_by_len), 65535);
  }
  int seg_steps = (p.L + nseg - 1) / nseg;
  seg_steps = (seg_steps + kSegAlign - 1) / kSegAlign * kSegAlign;
  pl.seg_steps = seg_steps;
  pl.nseg = (p.L + seg_steps - 1) / seg_steps;
  return pl;
}

static long long generic_bwd_warps(int N) {   // warps of a block of the generic backward kernel
  const int lpc = N / (N < 4 ? N : 4);
  return std::max(1, bwd_channels_per_block(N) * lpc / 32);
}

// The backward pass splits time on its own terms (the checkpoint states do not depend on the split, so forward and
// backward may disagree about it).  A split costs an adjoint pre-pass over all segments but the first and a carry scan;
// it pays when the chains alone leave the SM sub-partitions with too few warps.  Segments are at least 256 steps.
Plan make_bwd_plan(const ssm_problem_t& p) {
  Plan pl = make_plan(p);
  if (tuned_shape(p)) {
    // the tuned kernel's chains (and the channel groups of its dB / dC partial sums) are narrower than the generic ones
    pl.bwd_ch = bwd_fast_channels_per_warp();
    pl.bwd_groups = (p.D + pl.bwd_ch - 1) / pl.bwd_ch;
  }
  const long long chains = (long long)p.batch * pl.bwd_groups;
  const long long resident = 4LL * kNumSMs;
  int nseg = 1;
  if (p.flags & SSM_FLAG_COMPLEX) {
    // the complex path does not split time
  } else if (tuned_shape(p)) {
    // the tuned kernel wants two warps per SM sub-partition (a lone warp cannot cover its own latencies), i.e. two
    // rounds of chains; the adjoint pre-pass that a split costs is about a tenth of the backward work
    if (chains < 2 * resident) {
      const long long want = (2 * resident + chains - 1) / chains;
      const long long max_by_len = std::max(1, p.L / 256);
      nseg = (int)std::min<long long>(std::min(want, max_by_len), 65535);
    }
  } else if (chains * generic_bwd_warps(p.N) < 4 * resident) {
    // generic kernel: latency-bound warps, so aim for 8 per sub-partition (measured against 2: 1.1 to 1.5 times faster)
    const long long want = (8 * resident + chains * generic_bwd_warps(p.N) - 1) / (chains * generic_bwd_warps(p.N));
    const long long max_by_len = std::max(1, p.L / 256);
    nseg = (int)std::min<long long>(std::min(want, max_by_len), 65535);
  }
  int seg_steps = (p.L + nseg - 1) / nseg;
  seg_steps = (seg_steps + kSegAlign - 1) / kSegAlign * kSegAlign;
  pl.seg_steps = seg_steps;
  pl.nseg = (p.L + seg_steps - 1) / seg_steps;
  return pl;
}

// Every non-empty workspace starts with a status block whose first word is the one ssm_scan_check_status reads.

struct FwdWorkspace {
  size_t seg_end, seg_dsum, h_start, flags, handoff, total;
  int max_workers;
};
static FwdWorkspace fwd_layout(const ssm_problem_t& p, const Plan& pl) {
  FwdWorkspace w{};
  const int cw = fwd_fast_channels_per_warp();
  w.max_workers = tuned_shape(p) ? shared_workers((long long)p.batch * pl.nseg * ((p.D + cw - 1) / cw)) : 0;
  if (pl.nseg == 1 && w.max_workers == 0) return w;
  size_t off = kStatusBytes;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off += align_up(bytes);
    return at;
  };
  if (pl.nseg > 1) {
    const size_t st = (size_t)p.batch * pl.nseg * p.D * p.N * sizeof(float);
    w.seg_end = take(st);
    w.h_start = take(st);
    w.seg_dsum = take((size_t)p.batch * pl.nseg * p.D * sizeof(float));
  }
  if (w.max_workers > 0) {
    w.flags = take((size_t)(w.max_workers + 1) * sizeof(int));
    w.handoff = take((size_t)(w.max_workers + 1) * fwd_handoff_bytes_per_worker());
  }
  w.total = off;
  return w;
}
// Points the forward parameters at the scheduling words of a forward workspace and clears them.
static cudaError_t attach_fwd_sched(const ssm_problem_t& p, const Plan& pl, char* ws, int* abort_word, FwdParams& fp,
                                    cudaStream_t s) {
  const FwdWorkspace w = fwd_layout(p, pl);
  fp.abort = abort_word;
  fp.max_workers = w.max_workers;
  if (w.max_workers == 0) return cudaSuccess;
  fp.flags = reinterpret_cast<int*>(ws + w.flags);
  fp.handoff = reinterpret_cast<float4*>(ws + w.handoff);
  return cudaMemsetAsync(ws + w.flags, 0, (size_t)(w.max_workers + 1) * sizeof(int), s);
}

struct BwdWorkspace {
  size_t dBC_part, dA_part, dD_part, dbias_part, ckpt, seg_local, seg_dsum, mu_in, fwd, flags, handoff, total;
  size_t dBs_part, dCs_part;   // static B / C
  int max_workers;
};
static BwdWorkspace bwd_layout(const ssm_problem_t& p, const Plan& pl, const Plan& pl_fwd) {
  BwdWorkspace w{};
  size_t off = kStatusBytes;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off += align_up(bytes);
    return at;
  };
  const size_t bln = (size_t)p.batch * p.L * p.N;
  const size_t parts = (size_t)p.batch * pl.nseg;
  w.dBC_part = take((size_t)pl.bwd_groups * 2 * bln * sizeof(float));
  w.dA_part = take(parts * p.D * p.N * sizeof(float));
  w.dD_part = take(parts * p.D * sizeof(float));
  w.dbias_part = take(parts * p.D * sizeof(float));
  w.ckpt = take((size_t)p.batch * pl.nck * ckpt_floats_per_step(tuned_shape(p), p.D, p.N) * sizeof(float));
  if (pl.nseg > 1) {
    const size_t st = parts * p.D * p.N * sizeof(float);
    w.seg_local = take(st);
    w.mu_in = take(st);
    w.seg_dsum = take(parts * p.D * sizeof(float));
  }
  w.fwd = take(fwd_layout(p, pl_fwd).total);   // the forward sweep that rebuilds checkpoints uses the forward split
  // (batch, segment, channel group) chains of the tuned kernel; SSM_FLAG_TEST_WITHHOLD forces chains to be shared
  const long long chains = (long long)parts * pl.bwd_groups;
  w.max_workers = !tuned_shape(p) ? 0 : (p.flags & SSM_FLAG_TEST_WITHHOLD) ? (int)std::max<long long>(1, (2 * chains + 2) / 3)
                                                                            : shared_workers(chains);
  w.flags = take((size_t)2 * (w.max_workers + 1) * sizeof(int));   // backward kernel | adjoint pre-pass
  w.handoff = take((size_t)(w.max_workers + 1) *
                   bwd_handoff_bytes_per_worker(p.flags & SSM_FLAG_STATIC_B, p.flags & SSM_FLAG_STATIC_C));
  if (p.flags & SSM_FLAG_STATIC_B) w.dBs_part = take(parts * p.D * p.N * sizeof(float));
  if (p.flags & SSM_FLAG_STATIC_C) w.dCs_part = take(parts * p.D * p.N * sizeof(float));
  w.total = off;
  return w;
}

static bool aligned_to(const void* ptr, size_t a) { return (reinterpret_cast<uintptr_t>(ptr) % a) == 0; }
// static B / C (and their gradients) are float32 whatever the io dtype
static bool static_bc_aligned(const ssm_problem_t& p, const void* B, const void* C, const void* dB, const void* dC) {
  const bool sb = p.flags & SSM_FLAG_STATIC_B, sc = p.flags & SSM_FLAG_STATIC_C;
  return (!sb || (aligned_to(B, 4) && (dB == nullptr || aligned_to(dB, 4)))) &&
         (!sc || (aligned_to(C, 4) && (dC == nullptr || aligned_to(dC, 4))));
}

static ssm_status_t check_ws(const void* ws, size_t have, size_t need) {
  if (need == 0) return SSM_OK;
  if (ws == nullptr || !aligned_to(ws, 256) || have < need) return SSM_ERR_WORKSPACE;
  return SSM_OK;
}

// Runs the passes that establish the state at the start of every segment (nothing to do without a time split).
static cudaError_t run_segment_starts(const ssm_problem_t& prob, const Plan& pl, FwdParams fp, char* ws,
                                      const float* h0, const float** h_start, cudaStream_t s) {
  *h_start = h0;  // one segment: [batch][1][D][N] is the layout of the caller's initial state
  if (pl.nseg == 1) return cudaSuccess;
  const FwdWorkspace w = fwd_layout(prob, pl);
  fp.seg_end = reinterpret_cast<float*>(ws + w.seg_end);
  fp.seg_dsum = reinterpret_cast<float*>(ws + w.seg_dsum);
  fp.h_start = nullptr;
  fp.ckpt = nullptr;
  fp.h_last = nullptr;
  cudaError_t e = launch_fwd(prob, pl, fp, kFwdSummary, s);
  if (e != cudaSuccess) return e;
  CarryParams cp{};
  cp.local = fp.seg_end;
  cp.dsum = fp.seg_dsum;
  cp.A = fp.A;
  cp.init = h0;
  cp.carried = reinterpret_cast<float*>(ws + w.h_start);
  cp.batch = prob.batch;
  cp.nseg = pl.nseg;
  cp.D = prob.D;
  cp.N = prob.N;
  cp.reverse = 0;
  e = launch_carry(cp, s);
  *h_start = cp.carried;
  return e;
}

}  // namespace ssm

using namespace ssm;

extern "C" {

size_t ssm_scan_fwd_workspace_bytes(const ssm_problem_t* p) {
  if (validate_problem(p) != SSM_OK) return 0;
  ssm_problem_t wide;
  if (widen_route(*p, &wide)) return widen_layout(*p, ssm_scan_fwd_workspace_bytes(&wide), false).total;
  return fwd_layout(*p, make_plan(*p)).total;
}

size_t ssm_scan_bwd_workspace_bytes(const ssm_problem_t* p) {
  if (validate_problem(p) != SSM_OK) return 0;
  if (p->flags & SSM_FLAG_COMPLEX) return complex_bwd_workspace_bytes(*p);
  ssm_problem_t wide;
  if (widen_route(*p, &wide)) return widen_layout(*p, ssm_scan_bwd_workspace_bytes(&wide), true).total;
  return bwd_layout(*p, make_bwd_plan(*p), make_plan(*p)).total;
}

size_t ssm_scan_saved_state_bytes(const ssm_problem_t* p) {
  if (validate_problem(p) != SSM_OK) return 0;
  if (p->flags & SSM_FLAG_COMPLEX) return complex_saved_state_bytes(*p);
  ssm_problem_t wide;
  if (widen_route(*p, &wide)) return ssm_scan_saved_state_bytes(&wide);
  const size_t nck = (size_t)(p->L + kCkptSteps - 1) / kCkptSteps;
  return (size_t)p->batch * nck * ckpt_floats_per_step(tuned_shape(*p), p->D, p->N) * sizeof(float);
}

int32_t ssm_scan_checkpoint_steps(void) { return kCkptSteps; }

const char* ssm_status_string(ssm_status_t s) {
  switch (s) {
    case SSM_OK: return "SSM_OK";
    case SSM_ERR_INVALID_ARG: return "SSM_ERR_INVALID_ARG: null or misaligned pointer, bad dimension or flag";
    case SSM_ERR_UNSUPPORTED: return "SSM_ERR_UNSUPPORTED: N must be a power of two up to 64 and io_dtype f32 or bf16";
    case SSM_ERR_WORKSPACE: return "SSM_ERR_WORKSPACE: workspace missing, misaligned or too small";
    case SSM_ERR_CUDA: return "SSM_ERR_CUDA: a CUDA call or kernel launch failed";
    case SSM_ERR_TIMEOUT: return "SSM_ERR_TIMEOUT: a bounded device-side wait gave up";
    case SSM_ERR_BOUNDS: return "SSM_ERR_BOUNDS: an index left its range (bounds-checking build)";
    default: return "unknown ssm_status_t";
  }
}

ssm_status_t ssm_scan_check_status(const ssm_problem_t* p, const void* workspace, void* stream) {
  const ssm_status_t st = validate_problem(p);
  if (st != SSM_OK) return st;
  if (workspace == nullptr) return SSM_ERR_WORKSPACE;
  int word = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return SSM_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return SSM_ERR_CUDA;
  return word == 0 ? SSM_OK : (word == 2 ? SSM_ERR_BOUNDS : SSM_ERR_TIMEOUT);
}

ssm_status_t ssm_scan_plan(const ssm_problem_t* p, int32_t* n_segments, int32_t* segment_steps,
                           int32_t* channels_per_block, int32_t* states_per_thread) {
  const ssm_status_t st = validate_problem(p);
  if (st != SSM_OK) return st;
  ssm_problem_t wide;
  if (widen_route(*p, &wide)) return ssm_scan_plan(&wide, n_segments, segment_steps, channels_per_block, states_per_thread);
  const Plan pl = make_plan(*p);
  if (n_segments) *n_segments = pl.nseg;
  if (segment_steps) *segment_steps = pl.seg_steps;
  if (channels_per_block) *channels_per_block = pl.fwd_ch;
  if (states_per_thread) *states_per_thread = tuned_shape(*p) ? fwd_states_per_thread() : (p->N < 4 ? p->N : 4);
  return SSM_OK;
}

ssm_status_t ssm_scan_bwd_plan(const ssm_problem_t* p, int32_t* n_segments, int32_t* segment_steps,
                               int32_t* channels_per_group) {
  const ssm_status_t st = validate_problem(p);
  if (st != SSM_OK) return st;
  ssm_problem_t wide;
  if (widen_route(*p, &wide)) return ssm_scan_bwd_plan(&wide, n_segments, segment_steps, channels_per_group);
  const Plan pl = make_bwd_plan(*p);
  if (n_segments) *n_segments = pl.nseg;
  if (segment_steps) *segment_steps = pl.seg_steps;
  if (channels_per_group) *channels_per_group = pl.bwd_ch;
  return SSM_OK;
}

static ssm_status_t fwd_impl(const ssm_problem_t* p, const void* x, const void* delta, const float* delta_bias,
                             const float* A, const void* B, const void* C, const float* D_skip, const void* z,
                             const float* h0, void* out, float* h_last, void* saved_states, void* workspace,
                             size_t workspace_bytes, void* stream) {
  ssm_status_t st = validate_problem(p);
  if (st != SSM_OK) return st;
  const bool has_z = p->flags & SSM_FLAG_HAS_Z, has_d = p->flags & SSM_FLAG_HAS_DSKIP;
  const bool save = p->flags & SSM_FLAG_SAVE_STATES;
  if (!x || !delta || !A || !B || !C || !out) return SSM_ERR_INVALID_ARG;
  if ((has_z && !z) || (has_d && !D_skip) || (save && !saved_states)) return SSM_ERR_INVALID_ARG;
  const size_t esz = p->io_dtype == SSM_BF16 ? 2 : 4;
  for (const void* q : {x, delta, B, C, z, (const void*)out})
    if (q && !aligned_to(q, esz)) return SSM_ERR_INVALID_ARG;
  if (!static_bc_aligned(*p, B, C, nullptr, nullptr)) return SSM_ERR_INVALID_ARG;
  for (const void* q : {(const void*)A, (const void*)D_skip, (const void*)saved_states, (const void*)h0, (const void*)h_last,
                        (const void*)delta_bias})
    if (q && !aligned_to(q, 4)) return SSM_ERR_INVALID_ARG;
  if (p->flags & SSM_FLAG_COMPLEX) {
    if (delta_bias != nullptr) return SSM_ERR_UNSUPPORTED;
    return complex_fwd(*p, x, delta, A, B, C, has_d ? D_skip : nullptr, has_z ? z : nullptr, h0, out, h_last,
                       save ? saved_states : nullptr, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? SSM_OK
               : SSM_ERR_CUDA;
  }
  ssm_problem_t wide;
  if (widen_route(*p, &wide)) {
    const size_t inner = ssm_scan_fwd_workspace_bytes(&wide);
    const WidenLayout wl = widen_layout(*p, inner, false);
    st = check_ws(workspace, workspace_bytes, wl.total);
    if (st != SSM_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    const bool sb = p->flags & SSM_FLAG_STATIC_B, sc = p->flags & SSM_FLAG_STATIC_C;
    const long long rows_t = (long long)p->batch * p->L, rows_s = (long long)p->batch * p->D;
    if (cudaMemsetAsync(ws, 0, kStatusBytes, s) != cudaSuccess) return SSM_ERR_CUDA;
    RepackJobs in{};
    repack_add(in, A, ws + wl.A, p->D, p->N, kWideN, kRepackA);
    repack_add(in, B, ws + wl.B, sb ? p->D : rows_t, p->N, kWideN, sb ? kRepackF32 : kRepackBf16);
    repack_add(in, C, ws + wl.C, sc ? p->D : rows_t, p->N, kWideN, sc ? kRepackF32 : kRepackBf16);
    repack_add(in, h0, ws + wl.h0, rows_s, p->N, kWideN, kRepackF32);
    if (repack_run(in, s) != cudaSuccess) return SSM_ERR_CUDA;
    st = fwd_impl(&wide, x, delta, delta_bias, reinterpret_cast<const float*>(ws + wl.A), ws + wl.B, ws + wl.C, D_skip, z,
                  h0 ? reinterpret_cast<const float*>(ws + wl.h0) : nullptr, out,
                  h_last ? reinterpret_cast<float*>(ws + wl.h_last) : nullptr, saved_states, workspace, inner, stream);
    if (st != SSM_OK) return st;
    RepackJobs outj{};
    repack_add(outj, h_last ? ws + wl.h_last : nullptr, h_last, rows_s, kWideN, p->N, kRepackF32);
    return repack_run(outj, s) == cudaSuccess ? SSM_OK : SSM_ERR_CUDA;
  }
  const Plan pl = make_plan(*p);
  st = check_ws(workspace, workspace_bytes, fwd_layout(*p, pl).total);
  if (st != SSM_OK) return st;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  FwdParams fp{};
  fp.x = x;
  fp.delta = delta;
  fp.z = has_z ? z : nullptr;
  fp.B = B;
  fp.C = C;
  fp.A = A;
  fp.Dskip = has_d ? D_skip : nullptr;
  fp.out = out;
  fp.batch = p->batch;
  fp.L = p->L;
  fp.D = p->D;
  fp.nseg = pl.nseg;
  fp.seg_steps = pl.seg_steps;
  fp.nck = pl.nck;
  fp.general_A = (p->flags & SSM_FLAG_GENERAL_A) ? 1 : 0;
  fp.zoh = (p->flags & SSM_FLAG_ZOH_BBAR) ? 1 : 0;
  fp.static_B = (p->flags & SSM_FLAG_STATIC_B) ? 1 : 0;
  fp.static_C = (p->flags & SSM_FLAG_STATIC_C) ? 1 : 0;
  fp.delta_bias = delta_bias;
  fp.softplus = (p->flags & SSM_FLAG_DELTA_SOFTPLUS) ? 1 : 0;
  if (fwd_layout(*p, pl).total > 0) {
    if (cudaMemsetAsync(workspace, 0, kStatusBytes, s) != cudaSuccess) return SSM_ERR_CUDA;
    if (attach_fwd_sched(*p, pl, static_cast<char*>(workspace), static_cast<int*>(workspace), fp, s) != cudaSuccess)
      return SSM_ERR_CUDA;
  }
  const float* h_start = nullptr;
  if (run_segment_starts(*p, pl, fp, static_cast<char*>(workspace), h0, &h_start, s) != cudaSuccess) return SSM_ERR_CUDA;
  if (fp.max_workers > 0 && pl.nseg > 1) {
    // the summary pass used the hand-off flags: clear them again for the full pass
    if (attach_fwd_sched(*p, pl, static_cast<char*>(workspace), static_cast<int*>(workspace), fp, s) != cudaSuccess)
      return SSM_ERR_CUDA;
  }
  fp.h_start = h_start;
  fp.h_last = h_last;
  fp.ckpt = save ? static_cast<float*>(saved_states) : nullptr;
  fp.ckpt_tiled = tuned_shape(*p) ? 1 : 0;
  if (launch_fwd(*p, pl, fp, kFwdFull, s) != cudaSuccess) return SSM_ERR_CUDA;
  return SSM_OK;
}

ssm_status_t ssm_scan_fwd_state(const ssm_problem_t* p, const void* x, const void* delta, const float* A,
                                const void* B, const void* C, const float* D_skip, const void* z, const float* h0,
                                void* out, float* h_last, void* saved_states, void* workspace, size_t workspace_bytes,
                                void* stream) {
  return fwd_impl(p, x, delta, nullptr, A, B, C, D_skip, z, h0, out, h_last, saved_states, workspace, workspace_bytes,
                  stream);
}

ssm_status_t ssm_scan_fwd(const ssm_problem_t* p, const void* x, const void* delta, const float* A, const void* B,
                          const void* C, const float* D_skip, const void* z, void* out, void* saved_states,
                          void* workspace, size_t workspace_bytes, void* stream) {
  return fwd_impl(p, x, delta, nullptr, A, B, C, D_skip, z, nullptr, out, nullptr, saved_states, workspace,
                  workspace_bytes, stream);
}

ssm_status_t ssm_scan_fwd_fused_dt(const ssm_problem_t* p, const void* x, const void* delta_pre,
                                   const float* delta_bias, const float* A, const void* B, const void* C,
                                   const float* D_skip, const void* z, const float* h0, void* out, float* h_last,
                                   void* saved_states, void* workspace, size_t workspace_bytes, void* stream) {
  return fwd_impl(p, x, delta_pre, delta_bias, A, B, C, D_skip, z, h0, out, h_last, saved_states, workspace,
                  workspace_bytes, stream);
}

ssm_status_t ssm_step(const ssm_problem_t* p, const void* x, const void* delta, const float* A, const void* B,
                      const void* C, const float* D_skip, const void* z, float* h, void* out, void* stream) {
  ssm_status_t st = validate_problem(p);
  if (st != SSM_OK) return st;
  if (p->L != 1) return SSM_ERR_INVALID_ARG;
  const bool has_z = p->flags & SSM_FLAG_HAS_Z, has_d = p->flags & SSM_FLAG_HAS_DSKIP;
  if (!x || !delta || !A || !B || !C || !h || !out) return SSM_ERR_INVALID_ARG;
  if ((has_z && !z) || (has_d && !D_skip)) return SSM_ERR_INVALID_ARG;
  const size_t esz = p->io_dtype == SSM_BF16 ? 2 : 4;
  for (const void* q : {x, delta, B, C, z, (const void*)out})
    if (q && !aligned_to(q, esz)) return SSM_ERR_INVALID_ARG;
  if (!static_bc_aligned(*p, B, C, nullptr, nullptr)) return SSM_ERR_INVALID_ARG;
  for (const void* q : {(const void*)A, (const void*)D_skip, (const void*)h})
    if (q && !aligned_to(q, 4)) return SSM_ERR_INVALID_ARG;
  // the state and A are accessed 16 bytes at a time when a channel has at least 4 states, B and C four values at a time
  if (p->N >= 4 && (!aligned_to(A, 16) || !aligned_to(h, 16))) return SSM_ERR_INVALID_ARG;
  if (p->N >= 4 && !(p->flags & SSM_FLAG_COMPLEX)) {
    const size_t ab = (p->flags & SSM_FLAG_STATIC_B) ? 16 : 4 * esz, ac = (p->flags & SSM_FLAG_STATIC_C) ? 16 : 4 * esz;
    if (!aligned_to(B, ab) || !aligned_to(C, ac)) return SSM_ERR_INVALID_ARG;
  }
  if (p->flags & SSM_FLAG_COMPLEX)
    return complex_step(*p, x, delta, A, B, C, has_d ? D_skip : nullptr, has_z ? z : nullptr, h, out,
                        static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? SSM_OK
               : SSM_ERR_CUDA;
  StepParams sp{};
  sp.x = x;
  sp.delta = delta;
  sp.z = has_z ? z : nullptr;
  sp.B = B;
  sp.C = C;
  sp.A = A;
  sp.Dskip = has_d ? D_skip : nullptr;
  sp.h = h;
  sp.out = out;
  sp.batch = p->batch;
  sp.D = p->D;
  sp.N = p->N;
  sp.zoh = (p->flags & SSM_FLAG_ZOH_BBAR) ? 1 : 0;
  sp.static_B = (p->flags & SSM_FLAG_STATIC_B) ? 1 : 0;
  sp.static_C = (p->flags & SSM_FLAG_STATIC_C) ? 1 : 0;
  if (launch_step(*p, sp, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SSM_ERR_CUDA;
  return SSM_OK;
}

static ssm_status_t bwd_impl(const ssm_problem_t* p, const void* x, const void* delta, const float* delta_bias,
                             const float* A, const void* B, const void* C, const float* D_skip, const void* z,
                             const void* dout, const float* h0, const float* dh_last, const void* saved_states,
                             void* dx, void* ddelta, float* ddelta_bias, float* dA, void* dB, void* dC, float* dD,
                             void* dz, float* dh0, void* workspace, size_t workspace_bytes, void* stream) {
  ssm_status_t st = validate_problem(p);
  if (st != SSM_OK) return st;
  const bool has_z = p->flags & SSM_FLAG_HAS_Z, has_d = p->flags & SSM_FLAG_HAS_DSKIP;
  if (!x || !delta || !A || !B || !C || !dout || !dx || !ddelta || !dA || !dB || !dC) return SSM_ERR_INVALID_ARG;
  if ((has_z && !z) || (has_d && !D_skip)) return SSM_ERR_INVALID_ARG;
  const size_t esz = p->io_dtype == SSM_BF16 ? 2 : 4;
  for (const void* q : {x, delta, B, C, z, dout, (const void*)dx, (const void*)ddelta, (const void*)dB,
                        (const void*)dC, (const void*)dz})
    if (q && !aligned_to(q, esz)) return SSM_ERR_INVALID_ARG;
  if (!static_bc_aligned(*p, B, C, dB, dC)) return SSM_ERR_INVALID_ARG;
  for (const void* q : {(const void*)A, (const void*)D_skip, saved_states, (const void*)dA, (const void*)dD,
                        (const void*)delta_bias, (const void*)ddelta_bias, (const void*)h0, (const void*)dh_last,
                        (const void*)dh0})
    if (q && !aligned_to(q, 4)) return SSM_ERR_INVALID_ARG;
  if (p->flags & SSM_FLAG_COMPLEX) {
    if (delta_bias != nullptr || ddelta_bias != nullptr) return SSM_ERR_UNSUPPORTED;
    st = check_ws(workspace, workspace_bytes, complex_bwd_workspace_bytes(*p));
    if (st != SSM_OK) return st;
    return complex_bwd(*p, x, delta, A, B, C, has_d ? D_skip : nullptr, has_z ? z : nullptr, dout, h0, dh_last,
                       saved_states, dx, ddelta, dA, dB, dC, has_d ? dD : nullptr, has_z ? dz : nullptr, dh0, workspace,
                       static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? SSM_OK
               : SSM_ERR_CUDA;
  }
  ssm_problem_t wide;
  if (widen_route(*p, &wide)) {
    const size_t inner = ssm_scan_bwd_workspace_bytes(&wide);
    const WidenLayout wl = widen_layout(*p, inner, true);
    st = check_ws(workspace, workspace_bytes, wl.total);
    if (st != SSM_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace);
    const bool sb = p->flags & SSM_FLAG_STATIC_B, sc = p->flags & SSM_FLAG_STATIC_C;
    const long long rows_t = (long long)p->batch * p->L, rows_s = (long long)p->batch * p->D;
    RepackJobs in{};
    repack_add(in, A, ws + wl.A, p->D, p->N, kWideN, kRepackA);
    repack_add(in, B, ws + wl.B, sb ? p->D : rows_t, p->N, kWideN, sb ? kRepackF32 : kRepackBf16);
    repack_add(in, C, ws + wl.C, sc ? p->D : rows_t, p->N, kWideN, sc ? kRepackF32 : kRepackBf16);
    repack_add(in, h0, ws + wl.h0, rows_s, p->N, kWideN, kRepackF32);
    repack_add(in, dh_last, ws + wl.dh_last, rows_s, p->N, kWideN, kRepackF32);
    if (repack_run(in, s) != cudaSuccess) return SSM_ERR_CUDA;
    st = bwd_impl(&wide, x, delta, delta_bias, reinterpret_cast<const float*>(ws + wl.A), ws + wl.B, ws + wl.C, D_skip, z,
                  dout, h0 ? reinterpret_cast<const float*>(ws + wl.h0) : nullptr,
                  dh_last ? reinterpret_cast<const float*>(ws + wl.dh_last) : nullptr, saved_states, dx, ddelta,
                  ddelta_bias, reinterpret_cast<float*>(ws + wl.dA), ws + wl.dB, ws + wl.dC, dD, dz,
                  dh0 ? reinterpret_cast<float*>(ws + wl.dh0) : nullptr, workspace, inner, stream);
    if (st != SSM_OK) return st;
    RepackJobs outj{};
    repack_add(outj, ws + wl.dA, dA, p->D, kWideN, p->N, kRepackF32);
    repack_add(outj, ws + wl.dB, dB, sb ? p->D : rows_t, kWideN, p->N, sb ? kRepackF32 : kRepackBf16);
    repack_add(outj, ws + wl.dC, dC, sc ? p->D : rows_t, kWideN, p->N, sc ? kRepackF32 : kRepackBf16);
    repack_add(outj, dh0 ? ws + wl.dh0 : nullptr, dh0, rows_s, kWideN, p->N, kRepackF32);
    return repack_run(outj, s) == cudaSuccess ? SSM_OK : SSM_ERR_CUDA;
  }
  const Plan pl = make_bwd_plan(*p), pl_fwd = make_plan(*p);
  const BwdWorkspace w = bwd_layout(*p, pl, pl_fwd);
  st = check_ws(workspace, workspace_bytes, w.total);
  if (st != SSM_OK) return st;

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);

  if (cudaMemsetAsync(ws, 0, kStatusBytes, s) != cudaSuccess) return SSM_ERR_CUDA;
  // checkpoint states: the caller's, or rebuilt here with one more forward sweep
  const float* ckpt = static_cast<const float*>(saved_states);
  if (ckpt == nullptr) {
    FwdParams fp{};
    fp.x = x;
    fp.delta = delta;
    fp.B = B;
    fp.C = C;
    fp.A = A;
    fp.batch = p->batch;
    fp.L = p->L;
    fp.D = p->D;
    fp.nseg = pl_fwd.nseg;
    fp.seg_steps = pl_fwd.seg_steps;
    fp.nck = pl_fwd.nck;
    fp.general_A = (p->flags & SSM_FLAG_GENERAL_A) ? 1 : 0;
    fp.zoh = (p->flags & SSM_FLAG_ZOH_BBAR) ? 1 : 0;
    fp.static_B = (p->flags & SSM_FLAG_STATIC_B) ? 1 : 0;
    fp.static_C = (p->flags & SSM_FLAG_STATIC_C) ? 1 : 0;
    fp.delta_bias = delta_bias;
    fp.softplus = (p->flags & SSM_FLAG_DELTA_SOFTPLUS) ? 1 : 0;
    if (attach_fwd_sched(*p, pl_fwd, ws + w.fwd, reinterpret_cast<int*>(ws), fp, s) != cudaSuccess) return SSM_ERR_CUDA;
    const float* h_start = nullptr;
    if (run_segment_starts(*p, pl_fwd, fp, ws + w.fwd, h0, &h_start, s) != cudaSuccess) return SSM_ERR_CUDA;
    if (fp.max_workers > 0 && pl_fwd.nseg > 1 &&
        attach_fwd_sched(*p, pl_fwd, ws + w.fwd, reinterpret_cast<int*>(ws), fp, s) != cudaSuccess)
      return SSM_ERR_CUDA;
    fp.h_start = h_start;
    fp.ckpt = reinterpret_cast<float*>(ws + w.ckpt);
    fp.ckpt_tiled = tuned_shape(*p) ? 1 : 0;
    if (launch_fwd(*p, pl_fwd, fp, kFwdCkptOnly, s) != cudaSuccess) return SSM_ERR_CUDA;
    ckpt = fp.ckpt;
  }

  BwdParams bp{};
  bp.x = x;
  bp.delta = delta;
  bp.z = has_z ? z : nullptr;
  bp.B = B;
  bp.C = C;
  bp.A = A;
  bp.Dskip = has_d ? D_skip : nullptr;
  bp.dout = dout;
  bp.ckpt = ckpt;
  bp.ckpt_tiled = tuned_shape(*p) ? 1 : 0;
  bp.dx = dx;
  bp.ddelta = ddelta;
  bp.dz = has_z ? dz : nullptr;
  bp.dBC_part = reinterpret_cast<float*>(ws + w.dBC_part);
  bp.dA_part = reinterpret_cast<float*>(ws + w.dA_part);
  bp.dD_part = reinterpret_cast<float*>(ws + w.dD_part);
  bp.batch = p->batch;
  bp.L = p->L;
  bp.D = p->D;
  bp.nseg = pl.nseg;
  bp.seg_steps = pl.seg_steps;
  bp.nck = pl.nck;
  bp.groups = pl.bwd_groups;
  bp.general_A = (p->flags & SSM_FLAG_GENERAL_A) ? 1 : 0;
  bp.zoh = (p->flags & SSM_FLAG_ZOH_BBAR) ? 1 : 0;
  bp.static_B = (p->flags & SSM_FLAG_STATIC_B) ? 1 : 0;
  bp.static_C = (p->flags & SSM_FLAG_STATIC_C) ? 1 : 0;
  bp.dBs_part = bp.static_B ? reinterpret_cast<float*>(ws + w.dBs_part) : nullptr;
  bp.dCs_part = bp.static_C ? reinterpret_cast<float*>(ws + w.dCs_part) : nullptr;
  bp.test_withhold = (p->flags & SSM_FLAG_TEST_WITHHOLD) ? 1 : 0;
  bp.delta_bias = delta_bias;
  bp.softplus = (p->flags & SSM_FLAG_DELTA_SOFTPLUS) ? 1 : 0;
  bp.dh0 = dh0;
  bp.mu_in = dh_last;  // one segment: [batch][1][D][N] is the layout of the caller's adjoint
  bp.dbias_part = ddelta_bias != nullptr ? reinterpret_cast<float*>(ws + w.dbias_part) : nullptr;
  bp.abort = reinterpret_cast<int*>(ws);
  bp.flags = reinterpret_cast<int*>(ws + w.flags);
  bp.handoff = reinterpret_cast<float4*>(ws + w.handoff);
  bp.max_workers = w.max_workers;
  // the hand-off flags of the tuned kernel start at zero (the status word was cleared above)
  if (cudaMemsetAsync(ws + w.flags, 0, w.handoff - w.flags, s) != cudaSuccess) return SSM_ERR_CUDA;

  if (pl.nseg == 2 && dh_last == nullptr && (bp.seg_local = reinterpret_cast<float*>(ws + w.mu_in),
                                              bp.seg_dsum = reinterpret_cast<float*>(ws + w.seg_dsum),
                                              bwd_local_fast_applicable(*p, bp))) {
    // two segments and nothing flowing in from outside: the adjoint leaving segment 1 IS the inflow of segment 0, so
    // the tuned pre-pass writes it there and the carry scan is skipped
    bp.local_as_inflow = 1;
    if (launch_bwd(*p, pl, bp, kBwdLocal, s) != cudaSuccess) return SSM_ERR_CUDA;
    bp.mu_in = bp.seg_local;
  } else if (pl.nseg > 1) {
    bp.seg_local = reinterpret_cast<float*>(ws + w.seg_local);
    bp.seg_dsum = reinterpret_cast<float*>(ws + w.seg_dsum);
    if (launch_bwd(*p, pl, bp, kBwdLocal, s) != cudaSuccess) return SSM_ERR_CUDA;
    CarryParams cp{};
    cp.local = bp.seg_local;
    cp.dsum = bp.seg_dsum;
    cp.A = A;
    cp.carried = reinterpret_cast<float*>(ws + w.mu_in);
    cp.batch = p->batch;
    cp.nseg = pl.nseg;
    cp.D = p->D;
    cp.N = p->N;
    cp.reverse = 1;
    cp.init = dh_last;
    if (launch_carry(cp, s) != cudaSuccess) return SSM_ERR_CUDA;
    bp.mu_in = cp.carried;
  }
  // the generic kernel (taken when a pointer is not 16-byte aligned) writes one partial sum per 32 channels
  if (!bwd_fast_applicable(*p, bp)) bp.groups = (p->D + bwd_channels_per_block(p->N) - 1) / bwd_channels_per_block(p->N);
  if (launch_bwd(*p, pl, bp, kBwdFull, s) != cudaSuccess) return SSM_ERR_CUDA;

  ReduceParams rp{};
  rp.dBC_part = bp.dBC_part;
  rp.dB = bp.static_B ? nullptr : dB;   // static B / C: float32 [D][N] sums over batch and time instead
  rp.dC = bp.static_C ? nullptr : dC;
  rp.dBs = bp.static_B ? static_cast<float*>(dB) : nullptr;
  rp.dCs = bp.static_C ? static_cast<float*>(dC) : nullptr;
  rp.dBs_part = bp.dBs_part;
  rp.dCs_part = bp.dCs_part;
  rp.dA_part = bp.dA_part;
  rp.dD_part = bp.dD_part;
  rp.dA = dA;
  rp.dD = has_d ? dD : nullptr;
  rp.dbias_part = bp.dbias_part;
  rp.dbias = ddelta_bias;
  rp.bln = (long long)p->batch * p->L * p->N;
  rp.groups = bp.groups;
  rp.parts = p->batch * pl.nseg;
  rp.D = p->D;
  rp.N = p->N;
  if (launch_bwd_reduce(*p, rp, s) != cudaSuccess) return SSM_ERR_CUDA;
  return SSM_OK;
}

ssm_status_t ssm_scan_bwd(const ssm_problem_t* p, const void* x, const void* delta, const float* A, const void* B,
                          const void* C, const float* D_skip, const void* z, const void* dout,
                          const void* saved_states, void* dx, void* ddelta, float* dA, void* dB, void* dC, float* dD,
                          void* dz, void* workspace, size_t workspace_bytes, void* stream) {
  return bwd_impl(p, x, delta, nullptr, A, B, C, D_skip, z, dout, nullptr, nullptr, saved_states, dx, ddelta, nullptr,
                  dA, dB, dC, dD, dz, nullptr, workspace, workspace_bytes, stream);
}

ssm_status_t ssm_scan_bwd_state(const ssm_problem_t* p, const void* x, const void* delta, const float* A, const void* B,
                                const void* C, const float* D_skip, const void* z, const void* dout, const float* h0,
                                const float* dh_last, const void* saved_states, void* dx, void* ddelta, float* dA,
                                void* dB, void* dC, float* dD, void* dz, float* dh0, void* workspace,
                                size_t workspace_bytes, void* stream) {
  return bwd_impl(p, x, delta, nullptr, A, B, C, D_skip, z, dout, h0, dh_last, saved_states, dx, ddelta, nullptr, dA,
                  dB, dC, dD, dz, dh0, workspace, workspace_bytes, stream);
}

ssm_status_t ssm_scan_bwd_fused_dt_state(const ssm_problem_t* p, const void* x, const void* delta_pre,
                                         const float* delta_bias, const float* A, const void* B, const void* C,
                                         const float* D_skip, const void* z, const void* dout, const float* h0,
                                         const float* dh_last, const void* saved_states, void* dx, void* ddelta_pre,
                                         float* ddelta_bias, float* dA, void* dB, void* dC, float* dD, void* dz,
                                         float* dh0, void* workspace, size_t workspace_bytes, void* stream) {
  return bwd_impl(p, x, delta_pre, delta_bias, A, B, C, D_skip, z, dout, h0, dh_last, saved_states, dx, ddelta_pre,
                  ddelta_bias, dA, dB, dC, dD, dz, dh0, workspace, workspace_bytes, stream);
}

ssm_status_t ssm_scan_bwd_fused_dt(const ssm_problem_t* p, const void* x, const void* delta_pre,
                                   const float* delta_bias, const float* A, const void* B, const void* C,
                                   const float* D_skip, const void* z, const void* dout, const void* saved_states,
                                   void* dx, void* ddelta_pre, float* ddelta_bias, float* dA, void* dB, void* dC,
                                   float* dD, void* dz, void* workspace, size_t workspace_bytes, void* stream) {
  return bwd_impl(p, x, delta_pre, delta_bias, A, B, C, D_skip, z, dout, nullptr, nullptr, saved_states, dx, ddelta_pre,
                  ddelta_bias, dA, dB, dC, dD, dz, nullptr, workspace, workspace_bytes, stream);
}

}  // extern "C"
