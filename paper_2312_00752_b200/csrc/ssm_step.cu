// One recurrent step of the selective SSM (the recurrent mode of Eq. 2 used for autoregressive inference, Section 2
// "Computation"): for every (batch, channel)
//     h[n] <- exp(delta * A[n]) * h[n] + delta * x * B[n];   out = (sum_n C[n] h[n] + D_skip * x) * silu(z)
// (or with the zero-order-hold B-bar of Eq. 4 in place of delta * B),
// with the state h [batch][D][N] updated in place.  Constant time per token, no history.
//
// The work is a single pass over the state (2 * 4 N bytes per channel against a few bytes of inputs), so the kernel is
// a plain streaming kernel: one thread per (batch, channel), the N states of a channel read and written with 16-byte
// accesses, B and C of the batch entry read through the read-only cache.
#include "ssm_common.cuh"

namespace ssm {

template <typename IO, int N>
__global__ void __launch_bounds__(128) ssm_step_kernel(const StepParams p) {
  const int d = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = blockIdx.y;
  if (d >= p.D) return;
  const size_t e = (size_t)b * p.D + d;
  const IO* __restrict__ gB = static_cast<const IO*>(p.B) + (size_t)b * N;
  const IO* __restrict__ gC = static_cast<const IO*>(p.C) + (size_t)b * N;
  const float* __restrict__ sB = static_cast<const float*>(p.B) + (size_t)d * N;   // static B / C: float32 [D][N]
  const float* __restrict__ sC = static_cast<const float*>(p.C) + (size_t)d * N;
  const float dt = io_to_float<IO>(static_cast<const IO*>(p.delta)[e]);
  const float u = io_to_float<IO>(static_cast<const IO*>(p.x)[e]);
  const float du = dt * u;
  float* hrow = p.h + e * N;
  const float* arow = p.A + (size_t)d * N;
  float hv[N], av[N];
  if (N % 4 == 0) {
#pragma unroll
    for (int k = 0; k < N; k += 4) {
      const float4 h4 = *reinterpret_cast<const float4*>(hrow + k);
      const float4 a4 = __ldg(reinterpret_cast<const float4*>(arow + k));
      hv[k] = h4.x; hv[k + 1] = h4.y; hv[k + 2] = h4.z; hv[k + 3] = h4.w;
      av[k] = a4.x; av[k + 1] = a4.y; av[k + 2] = a4.z; av[k + 3] = a4.w;
    }
  } else {
#pragma unroll
    for (int k = 0; k < N; ++k) {
      hv[k] = hrow[k];
      av[k] = __ldg(arow + k);
    }
  }
  float y = 0.f;
#pragma unroll
  for (int k = 0; k < N; ++k) {
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
  if (N % 4 == 0) {
#pragma unroll
    for (int k = 0; k < N; k += 4) *reinterpret_cast<float4*>(hrow + k) = make_float4(hv[k], hv[k + 1], hv[k + 2], hv[k + 3]);
  } else {
#pragma unroll
    for (int k = 0; k < N; ++k) hrow[k] = hv[k];
  }
  float s = y;
  if (p.Dskip != nullptr) s = fmaf(p.Dskip[d], u, s);
  if (p.z != nullptr) {
    const float zz = io_to_float<IO>(static_cast<const IO*>(p.z)[e]);
    s = s * zz * sigmoid_fast(zz);
  }
  static_cast<IO*>(p.out)[e] = float_to_io<IO>(s);
}

template <typename IO>
static cudaError_t launch_step_io(const StepParams& p, cudaStream_t s) {
  dim3 grid((p.D + 127) / 128, p.batch);
  switch (p.N) {
    case 64: ssm_step_kernel<IO, 64><<<grid, 128, 0, s>>>(p); break;
    case 32: ssm_step_kernel<IO, 32><<<grid, 128, 0, s>>>(p); break;
    case 16: ssm_step_kernel<IO, 16><<<grid, 128, 0, s>>>(p); break;
    case 8: ssm_step_kernel<IO, 8><<<grid, 128, 0, s>>>(p); break;
    case 4: ssm_step_kernel<IO, 4><<<grid, 128, 0, s>>>(p); break;
    case 2: ssm_step_kernel<IO, 2><<<grid, 128, 0, s>>>(p); break;
    case 1: ssm_step_kernel<IO, 1><<<grid, 128, 0, s>>>(p); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_step(const ssm_problem_t& prob, const StepParams& p, cudaStream_t s) {
  if (prob.io_dtype == SSM_BF16) return launch_step_io<__nv_bfloat16>(p, s);
  return launch_step_io<float>(p, s);
}

}  // namespace ssm
