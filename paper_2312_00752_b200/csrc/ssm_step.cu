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

template <typename IO, int N>
__global__ void __launch_bounds__(128) ssm_step_kernel(const StepParams p) {
  constexpr int S = StepGeom<N>::S, LPC = StepGeom<N>::LPC, CH = StepGeom<N>::CH;
  const int j = threadIdx.x % LPC;
  const int d = blockIdx.x * CH + threadIdx.x / LPC;
  const int b = blockIdx.y;
  const bool valid = d < p.D;          // (whole lane groups are valid or not: the shuffles below stay inside a group)
  const int dc = valid ? d : 0;
  const size_t e = (size_t)b * p.D + dc;
  const IO* __restrict__ gB = static_cast<const IO*>(p.B) + (size_t)b * N + j * S;
  const IO* __restrict__ gC = static_cast<const IO*>(p.C) + (size_t)b * N + j * S;
  const float* __restrict__ sB = static_cast<const float*>(p.B) + (size_t)dc * N + j * S;   // static B / C: float32 [D][N]
  const float* __restrict__ sC = static_cast<const float*>(p.C) + (size_t)dc * N + j * S;
  const float dt = io_to_float<IO>(static_cast<const IO*>(p.delta)[e]);
  const float u = io_to_float<IO>(static_cast<const IO*>(p.x)[e]);
  const float du = dt * u;
  float* hrow = p.h + e * N + j * S;
  const float* arow = p.A + (size_t)dc * N + j * S;
  float hv[S], av[S];
  if constexpr (S == 4) {
    const float4 h4 = *reinterpret_cast<const float4*>(hrow);
    const float4 a4 = __ldg(reinterpret_cast<const float4*>(arow));
    hv[0] = h4.x; hv[1] = h4.y; hv[2] = h4.z; hv[3] = h4.w;
    av[0] = a4.x; av[1] = a4.y; av[2] = a4.z; av[3] = a4.w;
  } else {
#pragma unroll
    for (int k = 0; k < S; ++k) {
      hv[k] = hrow[k];
      av[k] = __ldg(arow + k);
    }
  }
  float y = 0.f;
#pragma unroll
  for (int k = 0; k < S; ++k) {
    const float Bk = p.static_B ? __ldg(sB + k) : io_to_float<IO>(__ldg(gB + k));
    float a, bx = du * Bk;
    if (p.zoh) {
      float E;
      zoh_discretize(dt, av[k], a, E);
      bx = E * u * Bk;
    } else {
      a = ex2_approx(dt * (av[k] * kLog2e));
    }
    hv[k] = fmaf(a, hv[k], bx);
    y = fmaf(p.static_C ? __ldg(sC + k) : io_to_float<IO>(__ldg(gC + k)), hv[k], y);
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

template <typename IO>
static cudaError_t launch_step_io(const StepParams& p, cudaStream_t s) {
  auto grid = [&](int ch) { return dim3((unsigned)((p.D + ch - 1) / ch), (unsigned)p.batch); };
  switch (p.N) {
    case 64: ssm_step_kernel<IO, 64><<<grid(StepGeom<64>::CH), 128, 0, s>>>(p); break;
    case 32: ssm_step_kernel<IO, 32><<<grid(StepGeom<32>::CH), 128, 0, s>>>(p); break;
    case 16: ssm_step_kernel<IO, 16><<<grid(StepGeom<16>::CH), 128, 0, s>>>(p); break;
    case 8: ssm_step_kernel<IO, 8><<<grid(StepGeom<8>::CH), 128, 0, s>>>(p); break;
    case 4: ssm_step_kernel<IO, 4><<<grid(StepGeom<4>::CH), 128, 0, s>>>(p); break;
    case 2: ssm_step_kernel<IO, 2><<<grid(StepGeom<2>::CH), 128, 0, s>>>(p); break;
    case 1: ssm_step_kernel<IO, 1><<<grid(StepGeom<1>::CH), 128, 0, s>>>(p); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_step(const ssm_problem_t& prob, const StepParams& p, cudaStream_t s) {
  if (prob.io_dtype == SSM_BF16) return launch_step_io<__nv_bfloat16>(p, s);
  return launch_step_io<float>(p, s);
}

}  // namespace ssm
