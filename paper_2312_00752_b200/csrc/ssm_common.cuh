// Shared declarations of the selective-scan kernels (sm_100a).  Internal to the library: nothing here is part of
// the C ABI, and nothing here is used by the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ssm_scan.h"

namespace ssm {

// Time steps between two checkpoint states (the state h at the start of every such block is what backward restarts
// its recomputation from: 8 steps of a thread's 16 recurrences are what its registers can hold, so no second level of
// recomputation is needed; the price is 8 bytes per element of checkpoint traffic in each direction, paid from HBM
// bandwidth the arithmetic-bound kernels leave idle).  Segment lengths of the time split are multiples of this.
constexpr int kCkptSteps = 8;
// Segment lengths of the time split are multiples of this (the tile length of every kernel divides it).
constexpr int kSegAlign = 32;
static_assert(kSegAlign % kCkptSteps == 0, "segments start on a checkpoint");
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kNumSMs = 148;

// ---------------------------------------------------------------------------------------------- plan (host)
struct Plan {
  int nseg;        // time segments per sequence (1: a thread sweeps the whole sequence)
  int seg_steps;   // steps per segment (multiple of kSegAlign; the last segment may be shorter)
  int nck;         // checkpoints per sequence = ceil(L / kCkptSteps)
  int fwd_cpt;     // channels per thread, forward
  int fwd_ch;      // channels per block, forward
  int bwd_ch;      // channels per block, backward (= channel-group size of the dB/dC partial sums)
  int bwd_groups;  // ceil(D / bwd_ch)
};
Plan make_plan(const ssm_problem_t& p);

// ---------------------------------------------------------------------------------------------- kernel params
// Offset (in floats) of state n of channel d in checkpoint kc of batch entry b.
//   plain: [batch][nck][D][N].
//   tiled (N = 16 only): [batch][nck][ceil(D / 32)][4][32][4] -- within a group of 32 channels the four 16-byte quarters
//   of a channel's 16 states are split over four planes, so that the 32 lanes of a warp that own one channel each write
//   (and read) 512 contiguous bytes per instruction instead of 16 bytes every 64.
__host__ __device__ __forceinline__ size_t ckpt_offset(int tiled, int b, int nck, int kc, int D, int N, int d, int n) {
  if (tiled) return ((((size_t)b * nck + kc) * ((D + 31) / 32) + (d >> 5)) * 4 + (n >> 2)) * 128 + (size_t)(d & 31) * 4 + (n & 3);
  return (((size_t)b * nck + kc) * D + d) * N + n;
}
// floats of the checkpoint states of one batch entry and checkpoint
__host__ __device__ __forceinline__ size_t ckpt_floats_per_step(int tiled, int D, int N) {
  return tiled ? (size_t)((D + 31) / 32) * 512 : (size_t)D * N;
}

struct FwdParams {
  const void* x;
  const void* delta;
  const void* z;       // null: no gate
  const void* B;
  const void* C;
  const float* A;
  const float* Dskip;  // null: no skip term
  void* out;           // FULL mode
  const float* h_start;  // [batch][nseg][D][N] start state of each segment; null: zero
  float* ckpt;           // checkpoint states to write (layout: ckpt_offset below); null: none
  int ckpt_tiled;        // 1: the layout of the tuned bf16 / N = 16 kernels
  float* seg_end;        // SUMMARY mode: [batch][nseg][D][N] end state of each segment started from zero
  float* seg_dsum;       // SUMMARY mode: [batch][nseg][D] sum of delta over the segment
  float* h_last;         // FULL mode: [batch][D][N] state after the last step; null: not wanted
  const float* delta_bias;  // [D] added to delta before the softplus; null: none
  int softplus;          // 1: `delta` is the pre-activation, the step size is softplus(delta + delta_bias)
  int batch, L, D, nseg, seg_steps, nck;
  int general_A;       // 1: never take the arithmetic-progression fast path
  int zoh;             // 1: B-bar = (exp(delta A) - 1) / A * B (Eq. 4) instead of delta * B
  int static_B, static_C;  // 1: B / C is a float32 [D][N] parameter (not input-dependent: Algorithm 1) instead of [batch][L][N]
  int* abort;            // tuned kernel: status word (non-zero: a bounded wait gave up); null: no chain may be shared
  int* flags;            // tuned kernel: [max_workers + 1] hand-off flags, zero before the launch
  float4* handoff;       // tuned kernel: carried state of a chain that two workers share
  int max_workers;       // tuned kernel: workers the hand-off slots allow (0: no chain may be shared)
};

// Work distribution of the warp-per-worker kernels.  The work is `chains` independent sequences of `tiles` tiles each
// (a chain is one time segment of 32 adjacent channels of one batch entry; tiles of a chain must run in order).  The
// linear tile space [0, chains * tiles) is cut into `workers` equal ranges, one per resident warp.  A range that starts
// or ends inside a chain shares that chain with the neighbouring worker: the state crosses from one to the other once,
// through `handoff`, guarded by `flags` (indexed by the receiving worker).  Every worker runs the piece that other
// workers wait for first (the leading part of its last chain), then its whole chains, then the piece that waits (the
// trailing part of its first chain); so with all workers resident a wait is satisfied after at most a short time, and
// the bounded poll below is a safety net, not a scheduling device.
struct WarpSched {
  int chains, tiles, workers, quota;   // quota: tiles per worker = ceil(chains * tiles / workers)
  int spin_limit;                      // polls of a flag before the worker gives up and raises *abort
  int withhold;                        // test hook: never publish a flag
  int* flags;                          // [workers + 1], zero before the launch
  int* abort;                          // one word, zero before the launch; non-zero: some wait gave up
  float4* handoff;                     // [workers + 1][32 lanes][vectors per lane]
};

struct CarryParams {
  const float* local;   // [batch][nseg][D][N]: per-segment result computed with zero inflow (end state e, or l)
  const float* dsum;    // [batch][nseg][D]: sum of delta over the segment
  const float* A;       // [D][N]
  const float* init;    // [batch][D][N]: what flows into the first segment in scan order; null: zero
  float* carried;       // [batch][nseg][D][N]: inflow of each segment (forward: state before its first step;
                        //                      reverse: adjoint flowing in from the following segment)
  int batch, nseg, D, N;
  int reverse;
};

struct BwdParams {
  const void* x;
  const void* delta;
  const void* z;
  const void* B;
  const void* C;
  const float* A;
  const float* Dskip;
  const void* dout;
  const float* ckpt;      // checkpoint states (layout: ckpt_offset below)
  int ckpt_tiled;         // 1: the layout of the tuned bf16 / N = 16 kernels
  const float* mu_in;     // [batch][nseg][D][N] adjoint inflow of each segment; null: zero
  float* seg_local;       // LOCAL mode: [batch][nseg][D][N] adjoint leaving each segment with zero inflow
  int local_as_inflow;    // tuned LOCAL kernel, two segments, no outside adjoint: write the result of segment 1 as the
                          // inflow of segment 0 and zero as the inflow of segment 1 (the layout of mu_in), so that the
                          // carry scan over two segments is not needed
  float* seg_dsum;        // LOCAL mode: [batch][nseg][D]
  void* dx;
  void* ddelta;
  void* dz;               // null: not produced
  float* dBC_part;        // [groups][2][batch*L*N] float partial sums over the channels of one block
  float* dA_part;         // [batch*nseg][D][N]
  float* dD_part;         // [batch*nseg][D]
  int batch, L, D, nseg, seg_steps, nck, groups;
  int general_A;          // 1: never take the arithmetic-progression fast path
  const float* delta_bias;  // as in FwdParams
  int softplus;
  float* dbias_part;      // [batch*nseg][D] sums of the pre-activation gradient; null: not wanted
  float* dh0;             // [batch][D][N] gradient of the initial state (the adjoint mu that leaves the first step);
                          // null: not wanted
  int zoh;                // as in FwdParams
  int static_B, static_C;  // as in FwdParams
  float* dBs_part;        // static B: [batch*nseg][D][N] per-thread sums over time of the dB terms
  float* dCs_part;        // static C: same for dC
  int test_withhold;      // test hook: never publish hand-off flags, poll only 1000 times
  int* abort;             // status word of the workspace (non-zero: a bounded wait gave up)
  int* flags;             // tuned kernel: [max_workers + 1] hand-off flags, zero before the launch
  float4* handoff;        // tuned kernel: carried values of a chain that two workers share
  int max_workers;        // tuned kernel: workers the hand-off slots allow (0: no chain may be shared)
};

struct ReduceParams {
  const float* dBC_part;  // [groups][2][rows*N]
  void* dB;
  void* dC;
  const float* dA_part;   // [parts][D*N]
  const float* dD_part;   // [parts][D]
  float* dA;
  float* dD;              // null: skip
  const float* dbias_part;  // [parts][D]
  float* dbias;           // null: skip
  long long bln;          // batch*L*N
  int groups, parts, D, N;
  const float* dBs_part;  // static B / C: [parts][D*N] partial sums; null: B / C are input-dependent
  const float* dCs_part;
  float* dBs;             // static B: float32 [D][N] (then dB above is null)
  float* dCs;
};

cudaError_t launch_fwd(const ssm_problem_t& prob, const Plan& plan, const FwdParams& p, int mode, cudaStream_t s);
cudaError_t launch_carry(const CarryParams& p, cudaStream_t s);
cudaError_t launch_bwd(const ssm_problem_t& prob, const Plan& plan, const BwdParams& p, int mode, cudaStream_t s);
cudaError_t launch_bwd_reduce(const ssm_problem_t& prob, const ReduceParams& p, cudaStream_t s);

struct StepParams {
  const void* x;        // [batch][D]
  const void* delta;    // [batch][D]
  const void* z;        // [batch][D] or null
  const void* B;        // [batch][N]
  const void* C;        // [batch][N]
  const float* A;       // [D][N]
  const float* Dskip;   // [D] or null
  float* h;             // [batch][D][N], updated in place
  void* out;            // [batch][D]
  int batch, D, N;
  int zoh;              // as in FwdParams
  int static_B, static_C;  // as in FwdParams
};
cudaError_t launch_step(const ssm_problem_t& prob, const StepParams& p, cudaStream_t s);

enum FwdMode { kFwdFull = 0, kFwdSummary = 1, kFwdCkptOnly = 2 };
enum BwdMode { kBwdFull = 0, kBwdLocal = 1 };

// ---------------------------------------------------------------------------------------------- device helpers
#ifdef __CUDACC__
// Bounds-checking build (-DSSM_DEBUG_BOUNDS; a memory checker is not available on the GPUs this is developed on): the
// tuned kernels range-check every tile row index (clamped to row 0 on violation) and every global row / channel offset
// they store to (the store is skipped), and record a violation as the value 2 in the status word of the workspace.
// Nothing traps or asserts, so a bad index can be found on a small case without losing the context.
#ifdef SSM_DEBUG_BOUNDS
#define SSM_TILE_ROW(r, limit, status) \
  (((unsigned)(r) < (unsigned)(limit)) ? (r) : (((status) != nullptr ? atomicExch((status), 2) : 0), 0))
#define SSM_IN_RANGE(cond, status) ((cond) ? true : (((status) != nullptr ? atomicExch((status), 2) : 0), false))
#else
#define SSM_TILE_ROW(r, limit, status) (r)
#define SSM_IN_RANGE(cond, status) true
#endif

__device__ __forceinline__ float ex2_approx(float v) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
  return r;
}
__device__ __forceinline__ float rcp_approx(float v) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
  return r;
}

template <typename IO>
__device__ __forceinline__ float io_to_float(IO v);
template <>
__device__ __forceinline__ float io_to_float<float>(float v) { return v; }
template <>
__device__ __forceinline__ float io_to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename IO>
__device__ __forceinline__ IO float_to_io(float v);
template <>
__device__ __forceinline__ float float_to_io<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 float_to_io<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// 16-byte asynchronous global -> shared copy; with valid == false nothing is read and the destination is zero-filled
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src, bool valid) {
  const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
  const int bytes = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(gmem_src), "r"(bytes) : "memory");
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// The pieces of one worker (see WarpSched), in the order in which it runs them.
struct WorkList {
  int c0, o0, c1, o1;     // first chain and first tile in it; last chain and one past the last tile in it
  int head, wf, nwhole;   // 1: the leading part of chain c1 is a piece of its own; first whole chain; whole chains
  int count;              // pieces
};
__device__ __forceinline__ WorkList make_worklist(const WarpSched& sc, int worker) {
  WorkList w{};
  const long long total = (long long)sc.chains * sc.tiles;
  const long long lo = (long long)worker * sc.quota;
  if (worker >= sc.workers || lo >= total) return w;   // count = 0
  long long hi = lo + sc.quota;
  if (hi > total) hi = total;
  w.c0 = (int)(lo / sc.tiles);
  w.o0 = (int)(lo - (long long)w.c0 * sc.tiles);
  w.c1 = (int)((hi - 1) / sc.tiles);
  w.o1 = (int)(hi - (long long)w.c1 * sc.tiles);
  if (w.c0 == w.c1) {
    w.count = 1;
    return w;
  }
  w.head = w.o1 < sc.tiles ? 1 : 0;
  const int tail = w.o0 > 0 ? 1 : 0;
  w.wf = w.c0 + tail;
  w.nwhole = (w.c1 - w.head) - w.wf + 1;
  w.count = w.head + w.nwhole + tail;
  return w;
}
// piece i of the list: tiles [from, to) of `chain`
__device__ __forceinline__ void get_piece(const WorkList& w, int tiles, int i, int& chain, int& from, int& to) {
  if (w.c0 == w.c1) {
    chain = w.c0; from = w.o0; to = w.o1;
  } else if (i < w.head) {
    chain = w.c1; from = 0; to = w.o1;
  } else if (i - w.head < w.nwhole) {
    chain = w.wf + i - w.head; from = 0; to = tiles;
  } else {
    chain = w.c0; from = w.o0; to = tiles;
  }
}
// Waits (lane 0 polls, bounded) until the worker that runs the earlier part of the chain has published it.
// Returns false to the whole warp when the wait gave up or another worker raised the abort word.
__device__ __forceinline__ bool wait_handoff(const WarpSched& sc, int worker, int lane) {
  int ok = 1;
  if (lane == 0) {
    int spins = 0;
    while (ld_acquire(sc.flags + worker) == 0) {
      __nanosleep(64);
      if (++spins > sc.spin_limit || ld_acquire(sc.abort) != 0) {
        atomicExch(sc.abort, 1);
        ok = 0;
        break;
      }
    }
  }
  ok = __shfl_sync(0xffffffffu, ok, 0);
  return ok != 0;
}
// Publishes the hand-off of the chain part this worker just finished (all lanes have written their vectors).
__device__ __forceinline__ void publish_handoff(const WarpSched& sc, int worker, int lane) {
  __threadfence();
  __syncwarp();
  if (lane == 0 && !sc.withhold) st_release(sc.flags + worker + 1, 1);
}

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// halves of a packed bf16 pair, widened to float (bf16 is the upper half of a float)
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
// the same through one byte-permute whose selector (0x1044: low half, 0x3244: high half) may differ per lane
__device__ __forceinline__ float bf16sel(uint32_t w, uint32_t sel) { return __uint_as_float(__byte_perm(w, 0u, sel)); }

__device__ __forceinline__ float2 f2mul(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 f2fma(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 f2dup(float v) { return make_float2(v, v); }

// softplus(v) = max(v, 0) + log1p(e^-|v|) for the tuned path: for small e = e^-|v| a short series (relative error
// below 2e-7), otherwise the hardware logarithm (absolute error ~2e-7 on a value above 0.06)
__device__ __forceinline__ float softplus_fast(float v) {
  const float e = ex2_approx(-fabsf(v) * kLog2e);
  const float series = e * fmaf(e, fmaf(e, fmaf(e, fmaf(e, 0.2f, -0.25f), 0.33333334f), -0.5f), 1.f);
  float lg;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lg) : "f"(1.f + e));
  return fmaxf(v, 0.f) + (e < 0.0625f ? series : lg * 0.6931471805599453f);
}

// sigmoid(v) from dt = softplus(v): sigmoid(v) = 1 - e^-dt (the derivative of the softplus, for the backward of the fused
// step size); a short series below dt = 1/32, where the difference would cancel
__device__ __forceinline__ float sigmoid_from_softplus(float dt) {
  const float closed = 1.f - ex2_approx(-dt * kLog2e);
  const float series = dt * fmaf(dt, fmaf(dt, 0.16666667f, -0.5f), 1.f);
  return dt < 0.03125f ? series : closed;
}

// softplus(v) = log(1 + e^v) = max(v, 0) + log1p(e^-|v|) with the precise library log1p (generic kernels)
__device__ __forceinline__ float softplus_precise(float v) { return fmaxf(v, 0.f) + log1pf(__expf(-fabsf(v))); }

// Zero-order-hold discretization of one (step, state), Eq. 4 for diagonal A: the input gain E with B-bar = E B is
// E = (exp(dt A) - 1) / A (E = dt at A = 0), taken from a precise expm1 so that a small dt A loses nothing; the decay
// is then a = 1 + E A.
__device__ __forceinline__ void zoh_discretize(float dt, float A, float& a, float& E) {
  if (A == 0.f) {
    a = 1.f;
    E = dt;
  } else {
    const float em1 = expm1f(dt * A);
    a = 1.f + em1;
    E = __fdividef(em1, A);
  }
}
// dE/dA = (dt a - E) / A = dt^2 (1/2 + x/3 + x^2/8 + ...), x = dt A: the series where the closed form cancels
__device__ __forceinline__ float zoh_gain_dA(float dt, float A, float a, float E) {
  const float x = dt * A;
  if (fabsf(x) < 0.25f) {
    float g = fmaf(x, 1.f / 45360.f, 1.f / 5760.f);
    g = fmaf(x, g, 1.f / 840.f);
    g = fmaf(x, g, 1.f / 144.f);
    g = fmaf(x, g, 1.f / 30.f);
    g = fmaf(x, g, 0.125f);
    g = fmaf(x, g, 1.f / 3.f);
    g = fmaf(x, g, 0.5f);
    return dt * dt * g;
  }
  return __fdividef(fmaf(dt, a, -E), A);
}

// The tuned kernels (bf16 io) take the closed forms E = (a - 1) / A, dE/dA = (dt a - E) / A from the decays they have
// anyway while every |dt A| of a sub-block of steps is at least kZohSmall: the relative error of E is then that of a
// (about 2.4e-7) divided by |dt A|, at most 5e-4 (a quarter of the bf16 rounding of the results), and the dE/dA term
// carries the same relative error into dA.  A sub-block with a smaller |dt A| anywhere in the warp (A = 0 included)
// runs the variant with the selects below.  The threshold sits below the step sizes of the layer workloads
// (delta >= 1e-3 with |A| >= 1), which therefore take the closed forms.
constexpr float kZohSmall = 0.00048828125f;   // 2^-11
__device__ __forceinline__ float2 zoh_gain_closed(float2 a, float2 invA) {
  return f2mul(f2fma(a, f2dup(1.f), f2dup(-1.f)), invA);
}
__device__ __forceinline__ float2 zoh_gain_dA_closed(float2 a, float2 E, float dt, float2 invA) {
  return f2mul(f2fma(f2dup(dt), a, f2mul(E, f2dup(-1.f))), invA);
}
// The same two quantities for a pair of states, without a branch, accurate for every dt A.  `a` are the decays
// the kernel has anyway, y2 = dt * A * log2(e), invA = 1 / A (0 where A = 0).  The closed forms (a - 1) / A and
// (dt a - E) / A lose all their digits as dt A -> 0 (a is rounded to 2^-24 next to 1), so for |dt A| < 1/4 the series
// in y = dt A take over; they also cover A = 0 (E = dt, dE/dA = dt^2 / 2).
__device__ __forceinline__ float2 zoh_gain_pair(float2 a, float2 y2, float dt, float2 invA) {
  constexpr float kLn2 = 0.6931471805599453f;
  constexpr float c1 = kLn2 / 2.f, c2 = kLn2 * kLn2 / 6.f, c3 = kLn2 * kLn2 * kLn2 / 24.f,
                  c4 = kLn2 * kLn2 * kLn2 * kLn2 / 120.f;
  float2 g = f2fma(y2, f2dup(c4), f2dup(c3));
  g = f2fma(y2, g, f2dup(c2));
  g = f2fma(y2, g, f2dup(c1));
  g = f2fma(y2, g, f2dup(1.f));
  const float2 Es = f2mul(f2dup(dt), g);
  const float2 Ec = f2mul(f2fma(a, f2dup(1.f), f2dup(-1.f)), invA);
  constexpr float kSmall = 0.25f * kLog2e;
  return make_float2(fabsf(y2.x) < kSmall ? Es.x : Ec.x, fabsf(y2.y) < kSmall ? Es.y : Ec.y);
}
__device__ __forceinline__ float2 zoh_gain_dA_pair(float2 a, float2 E, float2 y2, float dt, float2 invA) {
  constexpr float kLn2 = 0.6931471805599453f;
  constexpr float c1 = kLn2 / 3.f, c2 = kLn2 * kLn2 / 8.f, c3 = kLn2 * kLn2 * kLn2 / 30.f,
                  c4 = kLn2 * kLn2 * kLn2 * kLn2 / 144.f;
  float2 g = f2fma(y2, f2dup(c4), f2dup(c3));
  g = f2fma(y2, g, f2dup(c2));
  g = f2fma(y2, g, f2dup(c1));
  g = f2fma(y2, g, f2dup(0.5f));
  const float2 Gs = f2mul(f2dup(dt * dt), g);
  const float2 Gc = f2mul(f2fma(f2dup(dt), a, f2mul(E, f2dup(-1.f))), invA);
  constexpr float kSmall = 0.25f * kLog2e;
  return make_float2(fabsf(y2.x) < kSmall ? Gs.x : Gc.x, fabsf(y2.y) < kSmall ? Gs.y : Gc.y);
}

// tanh through the hardware unit (one special-function operation; relative error about 2^-11: bf16 io only)
__device__ __forceinline__ float tanh_approx(float v) {
  float r;
  asm("tanh.approx.f32 %0, %1;" : "=f"(r) : "f"(v));
  return r;
}
// s * silu(z) for a pair of elements with the hardware tanh: silu(z) = z/2 + z/2 tanh(z/2)
__device__ __forceinline__ float2 gate_pair_tanh(float2 s, float2 z) {
  const float2 hz = f2mul(z, f2dup(0.5f));
  const float2 sl = f2fma(hz, make_float2(tanh_approx(hz.x), tanh_approx(hz.y)), hz);
  return f2mul(s, sl);
}

// sigmoid(z) through one ex2 and one reciprocal
__device__ __forceinline__ float sigmoid_fast(float z) { return rcp_approx(1.0f + ex2_approx(-kLog2e * z)); }

// The associative operator of the recurrence h' = a h + b:  (a, b) o (a2, b2) = (a a2, a2 b + b2), i.e. "apply
// (a, b) first, then (a2, b2)".
struct AffinePair {
  float a, b;
};
__device__ __forceinline__ AffinePair combine(AffinePair first, AffinePair second) {
  return {first.a * second.a, fmaf(second.a, first.b, second.b)};
}
#endif

}  // namespace ssm
