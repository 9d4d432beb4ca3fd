// Forward selective scan: discretization, recurrence, readout, skip term and gate in one kernel
// (Algorithm 2 steps 5-6; Eq. 2a/2b; Eq. 4's A-bar; Section 3.3 "kernel fusion").
//
// Work decomposition.  The recurrence is sequential in time and independent across (batch, channel, state), and on
// this GPU the path is bound by FP32 issue rate rather than by memory, so a thread sweeps time sequentially and
// the parallelism comes from (batch, channel, state): a thread owns S = min(4, N) states of CPT adjacent
// channels, N / S adjacent lanes share a channel, and the sum over n of the readout is finished with xor
// shuffles.  Only when the channels alone cannot fill the GPU is the sequence also split into time segments
// (see ssm_carry.cu for how the state crosses segment boundaries).
//
// Modes: FULL writes `out` (and, if asked, the checkpoint states); SUMMARY runs a segment from a zero state and
// emits only its end state and the sum of delta (first pass of the time split); CKPT_ONLY rebuilds the checkpoint
// states for a backward call that was not given saved states.
#include "ssm_common.cuh"

namespace ssm {

// threads per block: 16 thread groups (of N / 4 lanes each) for N >= 16, 32 groups otherwise (keeps the staged tiles
// below 48 KB)
__host__ __device__ constexpr int fwd_threads(int N) { return N >= 16 ? 4 * N : (N == 8 ? 64 : 32); }
constexpr int kFwdTile = 32;  // time steps staged in shared memory at a time

template <typename IO, int N, int CPT, int MODE>
__global__ void __launch_bounds__(fwd_threads(N)) ssm_fwd_kernel(const FwdParams p) {
  constexpr int kFwdThreads = fwd_threads(N);
  constexpr int S = N < 4 ? N : 4;
  constexpr int LPC = N / S;                  // lanes per channel
  constexpr int SLOTS = kFwdThreads / LPC;    // thread groups (one per CPT channels) in the block
  constexpr int CH = SLOTS * CPT;             // channels per block
  constexpr int TT = kFwdTile;
  constexpr bool kReadout = (MODE == kFwdFull);
  constexpr int TZ = kReadout ? TT : 1;
  constexpr int FIN = (CPT + LPC - 1) / LPC;  // channels a lane finalises per step

  __shared__ __align__(16) IO s_x[TT][CH];
  __shared__ __align__(16) IO s_d[TT][CH];
  __shared__ __align__(16) IO s_z[TZ][CH];
  __shared__ __align__(16) IO s_o[TZ][CH];
  __shared__ __align__(16) float s_B[TT][N];
  __shared__ __align__(16) float s_C[TZ][N];

  const IO* __restrict__ gx = static_cast<const IO*>(p.x);
  const IO* __restrict__ gd = static_cast<const IO*>(p.delta);
  const IO* __restrict__ gz = static_cast<const IO*>(p.z);
  const IO* __restrict__ gB = static_cast<const IO*>(p.B);
  const IO* __restrict__ gC = static_cast<const IO*>(p.C);
  IO* __restrict__ gout = static_cast<IO*>(p.out);

  const int tid = threadIdx.x;
  const int j = tid % LPC;
  const int slot = tid / LPC;
  const int d_cta = blockIdx.x * CH;
  const int seg = blockIdx.y;
  const int b = blockIdx.z;
  const int t_begin = seg * p.seg_steps;
  const int t_end = min(p.L, t_begin + p.seg_steps);
  const int d_thr = d_cta + slot * CPT;
  const int D = p.D;

  float A2[CPT][S], Ar[CPT][S], h[CPT][S], dsum[CPT], dbias[CPT];
  float Bst[CPT][S], Cst[CPT][S];   // static B / C (parameters [D][N]): this thread's entries
#pragma unroll
  for (int q = 0; q < CPT; ++q) {
    const int d = d_thr + q;
    const bool valid = d < D;
    dsum[q] = 0.f;
    dbias[q] = (valid && p.delta_bias != nullptr) ? p.delta_bias[d] : 0.f;
#pragma unroll
    for (int k = 0; k < S; ++k) {
      Ar[q][k] = valid ? p.A[(size_t)d * N + j * S + k] : 0.f;
      Bst[q][k] = (valid && p.static_B) ? static_cast<const float*>(p.B)[(size_t)d * N + j * S + k] : 0.f;
      Cst[q][k] = (valid && p.static_C) ? static_cast<const float*>(p.C)[(size_t)d * N + j * S + k] : 0.f;
      A2[q][k] = Ar[q][k] * kLog2e;
      h[q][k] = (valid && p.h_start != nullptr)
                    ? p.h_start[(((size_t)b * p.nseg + seg) * D + d) * N + j * S + k]
                    : 0.f;
    }
  }
  // the channels this lane finalises (skip term, gate, store)
  float Dk_fin[FIN];
  int c_fin[FIN];
#pragma unroll
  for (int r = 0; r < FIN; ++r) {
    const int q = r * LPC + j;
    c_fin[r] = slot * CPT + q;
    const int d = d_cta + c_fin[r];
    Dk_fin[r] = (q < CPT && d < D && p.Dskip != nullptr) ? p.Dskip[d] : 0.f;
  }

  for (int t0 = t_begin; t0 < t_end; t0 += TT) {
    const int nt = min(TT, t_end - t0);
    const size_t row0 = (size_t)b * p.L + t0;
    __syncthreads();  // the previous tile's shared memory is no longer read
    for (int i = tid; i < TT * CH; i += kFwdThreads) {
      const int tt = i / CH, c = i % CH;
      const int d = d_cta + c;
      const bool ok = tt < nt && d < D;
      const size_t g = (row0 + tt) * D + d;
      s_x[tt][c] = ok ? gx[g] : float_to_io<IO>(0.f);
      s_d[tt][c] = ok ? gd[g] : float_to_io<IO>(0.f);
      if constexpr (kReadout) s_z[tt][c] = (ok && gz != nullptr) ? gz[g] : float_to_io<IO>(0.f);
    }
    for (int i = tid; i < TT * N; i += kFwdThreads) {
      const int tt = i / N, n = i % N;
      const bool ok = tt < nt;
      const size_t g = (row0 + tt) * N + n;
      s_B[tt][n] = (ok && !p.static_B) ? io_to_float<IO>(gB[g]) : 0.f;
      if constexpr (kReadout) s_C[tt][n] = (ok && !p.static_C) ? io_to_float<IO>(gC[g]) : 0.f;
    }
    __syncthreads();

#pragma unroll 2
    for (int tt = 0; tt < nt; ++tt) {
      if (MODE != kFwdSummary && p.ckpt != nullptr && ((t0 + tt) % kCkptSteps) == 0) {
        // the state before this step starts a checkpoint block
        const int kc = (t0 + tt) / kCkptSteps;
#pragma unroll
        for (int q = 0; q < CPT; ++q) {
          const int d = d_thr + q;
          if (d < D) {
            float* dst = p.ckpt + ckpt_offset(p.ckpt_tiled, b, p.nck, kc, D, N, d, j * S);
#pragma unroll
            for (int k = 0; k < S; ++k) dst[k] = h[q][k];
          }
        }
      }
      float Bv[S], Cv[S];
#pragma unroll
      for (int k = 0; k < S; ++k) {
        Bv[k] = s_B[tt][j * S + k];
        if constexpr (kReadout) Cv[k] = s_C[tt][j * S + k];
      }
      float y[CPT], u[CPT];
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        float dt = io_to_float<IO>(s_d[tt][slot * CPT + q]) + dbias[q];
        if (p.softplus) dt = softplus_precise(dt);
        u[q] = io_to_float<IO>(s_x[tt][slot * CPT + q]);
        const float du = dt * u[q];
        if (MODE == kFwdSummary) dsum[q] += dt;
        y[q] = 0.f;
#pragma unroll
        for (int k = 0; k < S; ++k) {
          const float Bk = p.static_B ? Bst[q][k] : Bv[k];
          float a, bx = du * Bk;
          if (p.zoh) {
            float E;
            zoh_discretize(dt, Ar[q][k], a, E);
            bx = E * u[q] * Bk;
          } else {
            a = ex2_approx(dt * A2[q][k]);
          }
          h[q][k] = fmaf(a, h[q][k], bx);
          if constexpr (kReadout) y[q] = fmaf(p.static_C ? Cst[q][k] : Cv[k], h[q][k], y[q]);
        }
      }
      if constexpr (kReadout) {
#pragma unroll
        for (int q = 0; q < CPT; ++q) {
#pragma unroll
          for (int m = LPC / 2; m >= 1; m >>= 1) y[q] += __shfl_xor_sync(0xffffffffu, y[q], m);
        }
#pragma unroll
        for (int r = 0; r < FIN; ++r) {
          float ym = y[0], um = u[0];
#pragma unroll
          for (int q = 1; q < CPT; ++q) {
            if (r * LPC + j == q) {
              ym = y[q];
              um = u[q];
            }
          }
          float s = fmaf(Dk_fin[r], um, ym);
          if (gz != nullptr) {
            const float zz = io_to_float<IO>(s_z[tt][c_fin[r] < CH ? c_fin[r] : 0]);
            s = s * zz * sigmoid_fast(zz);
          }
          if (r * LPC + j < CPT) s_o[tt][c_fin[r]] = float_to_io<IO>(s);
        }
      }
    }

    if constexpr (kReadout) {
      __syncthreads();
      for (int i = tid; i < nt * CH; i += kFwdThreads) {
        const int tt = i / CH, c = i % CH;
        const int d = d_cta + c;
        if (d < D) gout[(row0 + tt) * D + d] = s_o[tt][c];
      }
    }
  }

  if (MODE == kFwdFull && p.h_last != nullptr && seg == p.nseg - 1) {
#pragma unroll
    for (int q = 0; q < CPT; ++q) {
      const int d = d_thr + q;
      if (d < D) {
#pragma unroll
        for (int k = 0; k < S; ++k) p.h_last[((size_t)b * D + d) * N + j * S + k] = h[q][k];
      }
    }
  }
  if (MODE == kFwdSummary) {
#pragma unroll
    for (int q = 0; q < CPT; ++q) {
      const int d = d_thr + q;
      if (d < D) {
        float* dst = p.seg_end + (((size_t)b * p.nseg + seg) * D + d) * N + j * S;
#pragma unroll
        for (int k = 0; k < S; ++k) dst[k] = h[q][k];
        if (j == 0) p.seg_dsum[((size_t)b * p.nseg + seg) * D + d] = dsum[q];
      }
    }
  }
}

template <typename IO, int N, int CPT>
static cudaError_t launch_fwd_mode(const Plan& plan, const FwdParams& p, int mode, cudaStream_t s) {
  constexpr int S = N < 4 ? N : 4;
  constexpr int kFwdThreads = fwd_threads(N);
  constexpr int CH = (kFwdThreads / (N / S)) * CPT;
  dim3 grid((p.D + CH - 1) / CH, plan.nseg, p.batch);
  switch (mode) {
    case kFwdFull: ssm_fwd_kernel<IO, N, CPT, kFwdFull><<<grid, kFwdThreads, 0, s>>>(p); break;
    case kFwdSummary: ssm_fwd_kernel<IO, N, CPT, kFwdSummary><<<grid, kFwdThreads, 0, s>>>(p); break;
    default: ssm_fwd_kernel<IO, N, CPT, kFwdCkptOnly><<<grid, kFwdThreads, 0, s>>>(p); break;
  }
  return cudaGetLastError();
}

template <typename IO>
static cudaError_t launch_fwd_io(const ssm_problem_t& prob, const Plan& plan, const FwdParams& p, int mode,
                                 cudaStream_t s) {
  switch (prob.N) {
    case 64: return launch_fwd_mode<IO, 64, 2>(plan, p, mode, s);
    case 32: return launch_fwd_mode<IO, 32, 2>(plan, p, mode, s);
    case 16: return launch_fwd_mode<IO, 16, 2>(plan, p, mode, s);
    case 8: return launch_fwd_mode<IO, 8, 2>(plan, p, mode, s);
    case 4: return launch_fwd_mode<IO, 4, 2>(plan, p, mode, s);
    case 2: return launch_fwd_mode<IO, 2, 2>(plan, p, mode, s);
    case 1: return launch_fwd_mode<IO, 1, 2>(plan, p, mode, s);
    default: return cudaErrorInvalidValue;
  }
}

int fwd_channels_per_block(int N) {
  const int S = N < 4 ? N : 4;
  return (fwd_threads(N) / (N / S)) * 2;
}

bool fwd_fast_applicable(const ssm_problem_t& prob, const FwdParams& p);
cudaError_t launch_fwd_fast(const Plan& plan, const FwdParams& p, int mode, cudaStream_t s);

cudaError_t launch_fwd(const ssm_problem_t& prob, const Plan& plan, const FwdParams& p, int mode, cudaStream_t s) {
  if (fwd_fast_applicable(prob, p)) return launch_fwd_fast(plan, p, mode, s);
  if (prob.io_dtype == SSM_BF16) return launch_fwd_io<__nv_bfloat16>(prob, plan, p, mode, s);
  return launch_fwd_io<float>(prob, plan, p, mode, s);
}

}  // namespace ssm
