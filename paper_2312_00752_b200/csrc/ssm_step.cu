// One recurrent step of the selective SSM (the recurrent mode of Eq. 2 used for autoregressive inference, Section 2
// "Computation"): for every (batch, channel)
//     h[n] <- exp(delta * A[n]) * h[n] + delta * x * B[n];   out = (sum_n C[n] h[n] + D_skip * x) * silu(z)
// (or with the zero-order-hold B-bar of Eq. 4 in place of delta * B),
// with the state h [batch][D][N] updated in place.  Constant time per token, no history.
//
// The work is a single pass over the state (2 * 4 N bytes per channel against a few bytes of inputs), so the kernel is
// a plain streaming kernel.  A thread owns 4 states of one channel (all N of them for N < 4): the N / 4 lanes of a
// channel are adjacent, so every 16-byte access of a warp to the state covers 512 contiguous bytes, and the readout sum
// is finished with xor-shuffles.  B and C of the batch entry are read through the read-only cache.
#include "ssm_common.cuh"

namespace ssm {

template <int N>
struct StepGeom {
  static constexpr int S = N < 4 ? N : 4;    // states per thread
  static constexpr int LPC = N / S;          // lanes per channel
  static constexpr int CH = 128 / LPC;       // channels per block of 128 threads
};

// this thread's S values of a row of N: io dtype (B, C of the batch entry; one 8-byte load for four bf16 values) or float
template <typename IO, int S>
__device__ __forceinline__ void load_io_row(const IO* __restrict__ src, float (&v)[S]) {
  if constexpr (S == 4 && sizeof(IO) == 2) {
    const uint2 w = __ldg(reinterpret_cast<const uint2*>(src));
    v[0] = __uint_as_float(w.x << 16);
    v[1] = __uint_as_float(w.x & 0xffff0000u);
    v[2] = __uint_as_float(w.y << 16);
    v[3] = __uint_as_float(w.y & 0xffff0000u);
  } else if constexpr (S == 4) {
    const float4 w = __ldg(reinterpret_cast<const float4*>(src));
    v[0] = w.x; v[1] = w.y; v[2] = w.z; v[3] = w.w;
  } else {
#pragma unroll
    for (int k = 0; k < S; ++k) v[k] = io_to_float<IO>(__ldg(src + k));
  }
}

// ZOH: the B-bar rule of Eq. 4; SB / SC: B / C are float32 parameters [D][N] instead of inputs [batch][N]
template <typename IO, int N, bool ZOH, bool SB, bool SC>
__global__ void __launch_bounds__(128) ssm_step_kernel(const StepParams p) {
  constexpr int S = StepGeom<N>::S, LPC = StepGeom<N>::LPC, CH = StepGeom<N>::CH;
  const int j = threadIdx.x % LPC;
  const int d = blockIdx.x * CH + threadIdx.x / LPC;
  const int b = blockIdx.y;
  const bool valid = d < p.D;          // (whole lane groups are valid or not: the shuffles below stay inside a group)
  const int dc = valid ? d : 0;
  const size_t e = (size_t)b * p.D + dc;
  const float dt = io_to_float<IO>(static_cast<const IO*>(p.delta)[e]);
  const float u = io_to_float<IO>(static_cast<const IO*>(p.x)[e]);
  const float du = dt * u;
  float* hrow = p.h + e * N + j * S;
  float hv[S], av[S], Bv[S], Cv[S];
  load_io_row<float, S>(p.A + (size_t)dc * N + j * S, av);
  if constexpr (SB) load_io_row<float, S>(static_cast<const float*>(p.B) + (size_t)dc * N + j * S, Bv);
  else load_io_row<IO, S>(static_cast<const IO*>(p.B) + (size_t)b * N + j * S, Bv);
  if constexpr (SC) load_io_row<float, S>(static_cast<const float*>(p.C) + (size_t)dc * N + j * S, Cv);
  else load_io_row<IO, S>(static_cast<const IO*>(p.C) + (size_t)b * N + j * S, Cv);
  if constexpr (S == 4) {
    const float4 h4 = *reinterpret_cast<const float4*>(hrow);
    hv[0] = h4.x; hv[1] = h4.y; hv[2] = h4.z; hv[3] = h4.w;
  } else {
#pragma unroll
    for (int k = 0; k < S; ++k) hv[k] = hrow[k];
  }
  float y = 0.f;
#pragma unroll
  for (int k = 0; k < S; ++k) {
    float a, bx = du * Bv[k];
    if constexpr (ZOH) {
      float E;
      zoh_discretize(dt, av[k], a, E);
      bx = E * u * Bv[k];
    } else {
      a = ex2_approx(dt * (av[k] * kLog2e));
    }
    hv[k] = fmaf(a, hv[k], bx);
    y = fmaf(Cv[k], hv[k], y);
  }
  if (valid) {
    if constexpr (S == 4) {
      *reinterpret_cast<float4*>(hrow) = make_float4(hv[0], hv[1], hv[2], hv[3]);
    } else {
#pragma unroll
      for (int k = 0; k < S; ++k) hrow[k] = hv[k];
    }
  }
#pragma unroll
  for (int m = LPC / 2; m >= 1; m >>= 1) y += __shfl_xor_sync(0xffffffffu, y, m);
  if (valid && j == 0) {
    float s = y;
    if (p.Dskip != nullptr) s = fmaf(p.Dskip[d], u, s);
    if (p.z != nullptr) {
      const float zz = io_to_float<IO>(static_cast<const IO*>(p.z)[e]);
      s = s * zz * sigmoid_fast(zz);
    }
    static_cast<IO*>(p.out)[e] = float_to_io<IO>(s);
  }
}

template <typename IO, int N>
static void launch_step_n(const StepParams& p, cudaStream_t s) {
  const dim3 grid((unsigned)((p.D + StepGeom<N>::CH - 1) / StepGeom<N>::CH), (unsigned)p.batch);
  const int v = (p.zoh ? 1 : 0) | (p.static_B ? 2 : 0) | (p.static_C ? 4 : 0);
  switch (v) {
    case 0: ssm_step_kernel<IO, N, false, false, false><<<grid, 128, 0, s>>>(p); break;
    case 1: ssm_step_kernel<IO, N, true, false, false><<<grid, 128, 0, s>>>(p); break;
    case 2: ssm_step_kernel<IO, N, false, true, false><<<grid, 128, 0, s>>>(p); break;
    case 3: ssm_step_kernel<IO, N, true, true, false><<<grid, 128, 0, s>>>(p); break;
    case 4: ssm_step_kernel<IO, N, false, false, true><<<grid, 128, 0, s>>>(p); break;
    case 5: ssm_step_kernel<IO, N, true, false, true><<<grid, 128, 0, s>>>(p); break;
    case 6: ssm_step_kernel<IO, N, false, true, true><<<grid, 128, 0, s>>>(p); break;
    default: ssm_step_kernel<IO, N, true, true, true><<<grid, 128, 0, s>>>(p); break;
  }
}

template <typename IO>
static cudaError_t launch_step_io(const StepParams& p, cudaStream_t s) {
  switch (p.N) {
    case 64: launch_step_n<IO, 64>(p, s); break;
    case 32: launch_step_n<IO, 32>(p, s); break;
    case 16: launch_step_n<IO, 16>(p, s); break;
    case 8: launch_step_n<IO, 8>(p, s); break;
    case 4: launch_step_n<IO, 4>(p, s); break;
    case 2: launch_step_n<IO, 2>(p, s); break;
    case 1: launch_step_n<IO, 1>(p, s); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_step(const ssm_problem_t& prob, const StepParams& p, cudaStream_t s) {
  if (prob.io_dtype == SSM_BF16) return launch_step_io<__nv_bfloat16>(p, s);
  return launch_step_io<float>(p, s);
}

}  // namespace ssm
