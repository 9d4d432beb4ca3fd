// Short causal depthwise convolution (+ SiLU) in front of the selective scan (Section 3.4, Figure 3), forward and
// backward.  See include/ssm_conv1d.h for the definition and the contract.
//
// The operation moves 2 (forward) or 3 (backward) tensors of (batch, L, D) elements and does a handful of
// multiply-adds per element, so unlike the scan it is bound by HBM bandwidth, and the kernels are plain streaming
// kernels: a thread owns VEC adjacent channels (one 16- or 8-byte access per row, consecutive threads on consecutive
// addresses), walks a chunk of time steps with the W-1 previous inputs in a register window, and keeps several row
// loads in flight before it touches them.  Every element of x is read once per chunk (plus W-1 halo rows per chunk).
//
// Backward recomputes the pre-activation from x, forms dpre = dy * silu'(pre), and emits dx[s] once the W values
// dpre[s .. s+W-1] it depends on have passed through a second register window; dw and dbias are accumulated per thread
// over its chunk, written as partial sums per (batch, chunk) and added in ascending order by a second kernel (fixed
// order, no atomics).
#include <type_traits>

#include "ssm_common.cuh"
#include "ssm_conv1d.h"

namespace ssm {

namespace {

constexpr int kConvThreads = 64;
constexpr int kConvMinSteps = 32;   // time steps per thread and chunk: chosen per launch between these two so that the
constexpr int kConvMaxSteps = 128;  // grid fills the GPU a whole number of times (see choose_steps)
constexpr int kConvAheadFwd = 8;    // rows loaded before the first of them is used
constexpr int kConvAheadBwd = 8;    // (two tensors per row in the backward kernel; 2, 4, 8, 16 measured: 78, 64, 60, 83 us)

struct ConvParams {
  const void* x;
  const float* w;
  const float* bias;     // null: none
  const void* x_prev;    // null: zeros
  void* y;               // forward
  const void* dy;        // backward
  void* dx;
  void* dx_prev;         // null: not wanted
  float* part;           // backward: [batch * chunks][D][W + 1] partial sums of dw (W) and dbias (1)
  int batch, L, D, silu;
  int steps;             // time steps per chunk
};

template <typename IO, int VEC>
__device__ __forceinline__ void load_vec(const IO* __restrict__ p, float (&v)[VEC]) {
  if constexpr (VEC == 1) {
    v[0] = io_to_float<IO>(p[0]);
  } else if constexpr (sizeof(IO) == 4) {
    static_assert(VEC == 4, "float rows move as float4");
    const float4 u = *reinterpret_cast<const float4*>(p);
    v[0] = u.x; v[1] = u.y; v[2] = u.z; v[3] = u.w;
  } else if constexpr (VEC == 8) {
    const uint4 u = *reinterpret_cast<const uint4*>(p);
    v[0] = bf16lo(u.x); v[1] = bf16hi(u.x); v[2] = bf16lo(u.y); v[3] = bf16hi(u.y);
    v[4] = bf16lo(u.z); v[5] = bf16hi(u.z); v[6] = bf16lo(u.w); v[7] = bf16hi(u.w);
  } else {
    static_assert(VEC == 4, "bf16 rows move as 8 or 4 elements");
    const uint2 u = *reinterpret_cast<const uint2*>(p);
    v[0] = bf16lo(u.x); v[1] = bf16hi(u.x); v[2] = bf16lo(u.y); v[3] = bf16hi(u.y);
  }
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 r = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&r);
}

template <typename IO, int VEC>
__device__ __forceinline__ void store_vec(IO* __restrict__ p, const float (&v)[VEC]) {
  if constexpr (VEC == 1) {
    p[0] = float_to_io<IO>(v[0]);
  } else if constexpr (sizeof(IO) == 4) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  } else if constexpr (VEC == 8) {
    *reinterpret_cast<uint4*>(p) =
        make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
  } else {
    *reinterpret_cast<uint2*>(p) = make_uint2(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]));
  }
}

// ------------------------------------------------------------------------------------------------ scalar path
// (any D, any alignment; also the plain statement of the sliding windows that the vector path packs)
// x[b, s, c0 .. c0+VEC) for s in [-(W-1), L): negative s reads the carried context (or zero)
template <typename IO, int W, int VEC>
__device__ __forceinline__ void load_input_row(const ConvParams& p, int b, int s, int c0, float (&v)[VEC]) {
  if (s >= 0) {
    load_vec<IO, VEC>(static_cast<const IO*>(p.x) + ((size_t)b * p.L + s) * p.D + c0, v);
  } else if (p.x_prev != nullptr) {
    load_vec<IO, VEC>(static_cast<const IO*>(p.x_prev) + ((size_t)b * (W - 1) + (s + W - 1)) * p.D + c0, v);
  } else {
#pragma unroll
    for (int q = 0; q < VEC; ++q) v[q] = 0.f;
  }
}

template <typename IO, int W, int VEC>
__global__ void __launch_bounds__(kConvThreads) ssm_conv1d_fwd_kernel(const ConvParams p) {
  const int c0 = (blockIdx.x * kConvThreads + threadIdx.x) * VEC;
  if (c0 >= p.D) return;
  const int b = blockIdx.z;
  const int t0 = blockIdx.y * p.steps;
  const int t1 = min(p.L, t0 + p.steps);
  constexpr int H = W > 1 ? W - 1 : 1;
  constexpr int kConvAhead = kConvAheadFwd;

  float wv[W][VEC], bv[VEC], win[H][VEC];
#pragma unroll
  for (int q = 0; q < VEC; ++q) {
    bv[q] = p.bias != nullptr ? p.bias[c0 + q] : 0.f;
#pragma unroll
    for (int k = 0; k < W; ++k) wv[k][q] = p.w[(size_t)(c0 + q) * W + k];
  }
  // win[i] = x[t - (W-1) + i] at the start of step t
#pragma unroll
  for (int i = 0; i < W - 1; ++i) load_input_row<IO, W, VEC>(p, b, t0 - (W - 1) + i, c0, win[i]);

  const IO* __restrict__ xrow = static_cast<const IO*>(p.x) + ((size_t)b * p.L + t0) * p.D + c0;
  IO* __restrict__ yrow = static_cast<IO*>(p.y) + ((size_t)b * p.L + t0) * p.D + c0;
  for (int t = t0; t < t1; t += kConvAhead) {
    float cur[kConvAhead][VEC];
#pragma unroll
    for (int u = 0; u < kConvAhead; ++u)
      if (t + u < t1) load_vec<IO, VEC>(xrow + (size_t)(t + u - t0) * p.D, cur[u]);
#pragma unroll
    for (int u = 0; u < kConvAhead; ++u) {
      if (t + u < t1) {
        float o[VEC];
#pragma unroll
        for (int q = 0; q < VEC; ++q) {
          float pre = fmaf(wv[W - 1][q], cur[u][q], bv[q]);
#pragma unroll
          for (int k = 0; k < W - 1; ++k) pre = fmaf(wv[k][q], win[k][q], pre);
          o[q] = p.silu ? pre * sigmoid_fast(pre) : pre;
#pragma unroll
          for (int k = 0; k + 1 < W - 1; ++k) win[k][q] = win[k + 1][q];
          if (W > 1) win[H - 1][q] = cur[u][q];
        }
        store_vec<IO, VEC>(yrow + (size_t)(t + u - t0) * p.D, o);
      }
    }
  }
}

template <typename IO, int W, int VEC>
__global__ void __launch_bounds__(kConvThreads) ssm_conv1d_bwd_kernel(const ConvParams p) {
  const int c0 = (blockIdx.x * kConvThreads + threadIdx.x) * VEC;
  if (c0 >= p.D) return;
  const int b = blockIdx.z;
  const int t0 = blockIdx.y * p.steps;
  const int t1 = min(p.L, t0 + p.steps);
  constexpr int kConvAhead = kConvAheadBwd;

  float wv[W][VEC], bv[VEC];
  float xw[W][VEC];   // xw[i] = x[t - (W-1) + i]
  float dp[W][VEC];   // dp[i] = dpre[t - (W-1) + i]; values before this chunk are never used and start as zero
  float dwa[W][VEC], dba[VEC];
#pragma unroll
  for (int q = 0; q < VEC; ++q) {
    bv[q] = p.bias != nullptr ? p.bias[c0 + q] : 0.f;
    dba[q] = 0.f;
#pragma unroll
    for (int k = 0; k < W; ++k) {
      wv[k][q] = p.w[(size_t)(c0 + q) * W + k];
      dwa[k][q] = 0.f;
      dp[k][q] = 0.f;
    }
  }
#pragma unroll
  for (int i = 0; i < W - 1; ++i) load_input_row<IO, W, VEC>(p, b, t0 - (W - 1) + i, c0, xw[i]);

  const IO* __restrict__ gx = static_cast<const IO*>(p.x) + (size_t)b * p.L * p.D + c0;
  const IO* __restrict__ gy = static_cast<const IO*>(p.dy) + (size_t)b * p.L * p.D + c0;
  IO* __restrict__ gdx = static_cast<IO*>(p.dx) + (size_t)b * p.L * p.D + c0;
  // dx[s] needs dpre[s .. s+W-1]: the walk runs W-1 steps past the chunk (dpre is zero past the end of the sequence)
  const int t_stop = t1 + (W - 1);
  for (int t = t0; t < t_stop; t += kConvAhead) {
    float xin[kConvAhead][VEC], gin[kConvAhead][VEC];
#pragma unroll
    for (int u = 0; u < kConvAhead; ++u) {
      if (t + u < t_stop && t + u < p.L) {
        load_vec<IO, VEC>(gx + (size_t)(t + u) * p.D, xin[u]);
        load_vec<IO, VEC>(gy + (size_t)(t + u) * p.D, gin[u]);
      } else {
#pragma unroll
        for (int q = 0; q < VEC; ++q) xin[u][q] = gin[u][q] = 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < kConvAhead; ++u) {
      const int tt = t + u;
      if (tt < t_stop) {
        const bool own = tt < t1;          // this chunk owns the dw / dbias terms of step tt
        const int s = tt - (W - 1);        // the step whose dx is complete now
        float o[VEC];
#pragma unroll
        for (int q = 0; q < VEC; ++q) {
          xw[W - 1][q] = xin[u][q];
          float pre = bv[q];
#pragma unroll
          for (int k = 0; k < W; ++k) pre = fmaf(wv[k][q], xw[k][q], pre);
          float dpre = gin[u][q];
          if (p.silu) {
            const float sg = sigmoid_fast(pre);
            dpre *= sg * fmaf(pre, 1.f - sg, 1.f);
          }
          dp[W - 1][q] = dpre;
          if (own) {
            dba[q] += dpre;
#pragma unroll
            for (int k = 0; k < W; ++k) dwa[k][q] = fmaf(dpre, xw[k][q], dwa[k][q]);
          }
          float acc = 0.f;
#pragma unroll
          for (int k = 0; k < W; ++k) acc = fmaf(wv[k][q], dp[W - 1 - k][q], acc);   // dpre[s + (W-1) - k] = dpre[tt - k]
          o[q] = acc;
#pragma unroll
          for (int k = 0; k + 1 < W; ++k) {
            xw[k][q] = xw[k + 1][q];
            dp[k][q] = dp[k + 1][q];
          }
        }
        if (s >= t0) {
          store_vec<IO, VEC>(gdx + (size_t)s * p.D, o);
        } else if (t0 == 0 && s < 0 && p.dx_prev != nullptr) {
          store_vec<IO, VEC>(static_cast<IO*>(p.dx_prev) + ((size_t)b * (W - 1) + (s + W - 1)) * p.D + c0, o);
        }
      }
    }
  }
  float* part = p.part + ((size_t)(b * gridDim.y + blockIdx.y) * p.D + c0) * (W + 1);
#pragma unroll
  for (int q = 0; q < VEC; ++q) {
#pragma unroll
    for (int k = 0; k < W; ++k) part[q * (W + 1) + k] = dwa[k][q];
    part[q * (W + 1) + W] = dba[q];
  }
}

// ------------------------------------------------------------------------------------------------ vector path
// Four channels per thread, held as two packed float2 pairs so that the multiply-adds issue two-wide; rows stay in
// their loaded form (8 bytes of bf16 or 16 bytes of float) until they are used, which keeps kConvAhead* of them in
// flight per thread at little register cost; row pointers advance by one stride per step.
template <typename IO>
struct Raw4;
template <>
struct Raw4<__nv_bfloat16> {
  uint2 r;
};
template <>
struct Raw4<float> {
  float4 r;
};
__device__ __forceinline__ Raw4<__nv_bfloat16> load_raw4(const __nv_bfloat16* __restrict__ p) {
  return {*reinterpret_cast<const uint2*>(p)};
}
__device__ __forceinline__ Raw4<float> load_raw4(const float* __restrict__ p) {
  return {*reinterpret_cast<const float4*>(p)};
}
__device__ __forceinline__ void unpack4(const Raw4<__nv_bfloat16>& v, float2 (&o)[2]) {
  o[0] = make_float2(bf16lo(v.r.x), bf16hi(v.r.x));
  o[1] = make_float2(bf16lo(v.r.y), bf16hi(v.r.y));
}
__device__ __forceinline__ void unpack4(const Raw4<float>& v, float2 (&o)[2]) {
  o[0] = make_float2(v.r.x, v.r.y);
  o[1] = make_float2(v.r.z, v.r.w);
}
__device__ __forceinline__ void zero4(Raw4<__nv_bfloat16>& v) { v.r = make_uint2(0u, 0u); }
__device__ __forceinline__ void zero4(Raw4<float>& v) { v.r = make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ void store4(__nv_bfloat16* __restrict__ p, const float2 (&v)[2]) {
  *reinterpret_cast<uint2*>(p) = make_uint2(pack_bf16(v[0].x, v[0].y), pack_bf16(v[1].x, v[1].y));
}
__device__ __forceinline__ void store4(float* __restrict__ p, const float2 (&v)[2]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0].x, v[0].y, v[1].x, v[1].y);
}

// sigmoid of a pair.  FAST: 1/2 + 1/2 tanh(v/2) with the hardware tanh (one special-function operation instead of two;
// relative error about 2^-11, used for bf16 io only, whose own rounding is 2^-9); otherwise ex2 + reciprocal.
template <bool FAST>
__device__ __forceinline__ float2 sigmoid2(float2 v) {
  if (FAST) {
    const float2 h = f2mul(v, f2dup(0.5f));
    return f2fma(make_float2(tanh_approx(h.x), tanh_approx(h.y)), f2dup(0.5f), f2dup(0.5f));
  }
  return make_float2(sigmoid_fast(v.x), sigmoid_fast(v.y));
}

template <typename IO, int W>
__device__ __forceinline__ void load_taps4(const ConvParams& p, int c0, float2 (&wv)[W][2], float2 (&bv)[2]) {
  float wq[4][W], bq[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    bq[q] = p.bias != nullptr ? p.bias[c0 + q] : 0.f;
#pragma unroll
    for (int k = 0; k < W; ++k) wq[q][k] = p.w[(size_t)(c0 + q) * W + k];
  }
  bv[0] = make_float2(bq[0], bq[1]);
  bv[1] = make_float2(bq[2], bq[3]);
#pragma unroll
  for (int k = 0; k < W; ++k) {
    wv[k][0] = make_float2(wq[0][k], wq[1][k]);
    wv[k][1] = make_float2(wq[2][k], wq[3][k]);
  }
}

// x[b, s, c0 .. c0+4) for s in [-(W-1), L) as packed pairs
template <typename IO, int W>
__device__ __forceinline__ void load_input_row4(const ConvParams& p, int b, int s, int c0, float2 (&v)[2]) {
  Raw4<IO> r;
  if (s >= 0) r = load_raw4(static_cast<const IO*>(p.x) + ((size_t)b * p.L + s) * p.D + c0);
  else if (p.x_prev != nullptr) r = load_raw4(static_cast<const IO*>(p.x_prev) + ((size_t)b * (W - 1) + (s + W - 1)) * p.D + c0);
  else zero4(r);
  unpack4(r, v);
}

template <typename IO, int W, bool SILU, bool FAST>
__global__ void __launch_bounds__(kConvThreads) ssm_conv1d_fwd_vec4_kernel(const ConvParams p) {
  const int c0 = (blockIdx.x * kConvThreads + threadIdx.x) * 4;
  if (c0 >= p.D) return;
  const int b = blockIdx.z;
  const int t0 = blockIdx.y * p.steps;
  const int t1 = min(p.L, t0 + p.steps);
  constexpr int H = W > 1 ? W - 1 : 1;
  constexpr int A = kConvAheadFwd;

  float2 wv[W][2], bv[2], win[H][2];
  load_taps4<IO, W>(p, c0, wv, bv);
#pragma unroll
  for (int i = 0; i < W - 1; ++i) load_input_row4<IO, W>(p, b, t0 - (W - 1) + i, c0, win[i]);

  const IO* __restrict__ xp = static_cast<const IO*>(p.x) + ((size_t)b * p.L + t0) * p.D + c0;
  IO* __restrict__ yp = static_cast<IO*>(p.y) + ((size_t)b * p.L + t0) * p.D + c0;
  const size_t stride = (size_t)p.D;
  // Rows are fetched one batch ahead: while a batch is computed the loads of the next one are in flight.
  Raw4<IO> nxt[A];
  auto fetch = [&](int t) {   // rows t .. t+A-1 of the chunk
#pragma unroll
    for (int u = 0; u < A; ++u)
      if (t + u < t1) nxt[u] = load_raw4(xp + u * stride);
    xp += A * stride;
  };
  auto batch = [&](int t, int n, auto full_tag) {   // n rows from t (n == A when full_tag is true)
    constexpr bool FULL = decltype(full_tag)::value;
    Raw4<IO> raw[A];
#pragma unroll
    for (int u = 0; u < A; ++u) raw[u] = nxt[u];
    fetch(t + A);
#pragma unroll
    for (int u = 0; u < A; ++u) {
      if (FULL || u < n) {
        float2 cur[2], o[2];
        unpack4(raw[u], cur);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float2 pre = f2fma(wv[W - 1][h], cur[h], bv[h]);
#pragma unroll
          for (int k = 0; k < W - 1; ++k) pre = f2fma(wv[k][h], win[k][h], pre);
          o[h] = SILU ? f2mul(pre, sigmoid2<FAST>(pre)) : pre;
#pragma unroll
          for (int k = 0; k + 1 < W - 1; ++k) win[k][h] = win[k + 1][h];
          if (W > 1) win[H - 1][h] = cur[h];
        }
        store4(yp + u * stride, o);
      }
    }
    yp += A * stride;
  };
  fetch(t0);
  int t = t0;
  for (; t + A <= t1; t += A) batch(t, A, std::true_type{});
  if (t < t1) batch(t, t1 - t, std::false_type{});
}

template <typename IO, int W, bool SILU, bool FAST>
__global__ void __launch_bounds__(kConvThreads) ssm_conv1d_bwd_vec4_kernel(const ConvParams p) {
  const int c0 = (blockIdx.x * kConvThreads + threadIdx.x) * 4;
  if (c0 >= p.D) return;
  const int b = blockIdx.z;
  const int t0 = blockIdx.y * p.steps;
  const int t1 = min(p.L, t0 + p.steps);
  constexpr int A = kConvAheadBwd;

  float2 wv[W][2], bv[2];
  float2 xw[W][2];    // xw[i] = x[t - (W-1) + i]
  float2 dp[W][2];    // dp[i] = dpre[t - (W-1) + i]; values before this chunk are never used and start as zero
  float2 dwa[W][2], dba[2];
  load_taps4<IO, W>(p, c0, wv, bv);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    dba[h] = make_float2(0.f, 0.f);
#pragma unroll
    for (int k = 0; k < W; ++k) dwa[k][h] = dp[k][h] = make_float2(0.f, 0.f);
  }
#pragma unroll
  for (int i = 0; i < W - 1; ++i) load_input_row4<IO, W>(p, b, t0 - (W - 1) + i, c0, xw[i]);

  const size_t stride = (size_t)p.D;
  const IO* __restrict__ xp = static_cast<const IO*>(p.x) + ((size_t)b * p.L + t0) * p.D + c0;
  const IO* __restrict__ gp = static_cast<const IO*>(p.dy) + ((size_t)b * p.L + t0) * p.D + c0;
  IO* __restrict__ dxp = static_cast<IO*>(p.dx) + ((size_t)b * p.L + t0 - (W - 1)) * p.D + c0;   // row of s = t - (W-1)
  // dx[s] needs dpre[s .. s+W-1]: the walk runs W-1 steps past the chunk (dpre is zero past the end of the sequence)
  const int t_stop = t1 + (W - 1);
  // Rows are fetched one batch ahead: while batch t is computed the loads of batch t + A are in flight.
  Raw4<IO> nx[A], ng[A];   // the next batch, still in its loaded form
  auto fetch = [&](int t) {   // rows t .. t+A-1 (zeros outside the walk or past the end of the sequence)
#pragma unroll
    for (int u = 0; u < A; ++u) {
      if (t + u < t_stop && t + u < p.L) {
        nx[u] = load_raw4(xp + u * stride);
        ng[u] = load_raw4(gp + u * stride);
      } else {
        zero4(nx[u]);
        zero4(ng[u]);
      }
    }
    xp += A * stride;
    gp += A * stride;
  };
  auto batch = [&](int t, auto full_tag) {   // rows t .. t+A-1; FULL: all of them inside the chunk and the sequence
    constexpr bool FULL = decltype(full_tag)::value;
    Raw4<IO> rx[A], rg[A];
#pragma unroll
    for (int u = 0; u < A; ++u) {
      rx[u] = nx[u];
      rg[u] = ng[u];
    }
    fetch(t + A);
#pragma unroll
    for (int u = 0; u < A; ++u) {
      const int tt = t + u;
      if (FULL || tt < t_stop) {
        const bool own = FULL || tt < t1;  // this chunk owns the dw / dbias terms of step tt
        const int s = tt - (W - 1);        // the step whose dx is complete now
        float2 g2[2], o[2];
        unpack4(rx[u], xw[W - 1]);
        unpack4(rg[u], g2);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float2 pre = bv[h];
#pragma unroll
          for (int k = 0; k < W; ++k) pre = f2fma(wv[k][h], xw[k][h], pre);
          float2 dpre = g2[h];
          if (SILU) {
            const float2 sg = sigmoid2<FAST>(pre);
            const float2 om = f2fma(sg, f2dup(-1.f), f2dup(1.f));
            dpre = f2mul(dpre, f2mul(sg, f2fma(pre, om, f2dup(1.f))));
          }
          dp[W - 1][h] = dpre;
          if (own) {
            dba[h].x += dpre.x;
            dba[h].y += dpre.y;
#pragma unroll
            for (int k = 0; k < W; ++k) dwa[k][h] = f2fma(dpre, xw[k][h], dwa[k][h]);
          }
          float2 acc = f2mul(wv[0][h], dp[W - 1][h]);
#pragma unroll
          for (int k = 1; k < W; ++k) acc = f2fma(wv[k][h], dp[W - 1 - k][h], acc);   // dpre[s + (W-1) - k] = dpre[tt - k]
          o[h] = acc;
#pragma unroll
          for (int k = 0; k + 1 < W; ++k) {
            xw[k][h] = xw[k + 1][h];
            dp[k][h] = dp[k + 1][h];
          }
        }
        if (s >= t0) {
          store4(dxp + u * stride, o);
        } else if (t0 == 0 && s < 0 && p.dx_prev != nullptr) {
          store4(static_cast<IO*>(p.dx_prev) + ((size_t)b * (W - 1) + (s + W - 1)) * p.D + c0, o);
        }
      }
    }
    dxp += A * stride;
  };
  fetch(t0);
  int t = t0;
  for (; t + A <= t1; t += A) batch(t, std::true_type{});
  for (; t < t_stop; t += A) batch(t, std::false_type{});

  float* part = p.part + ((size_t)(b * gridDim.y + blockIdx.y) * p.D + c0) * (W + 1);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
#pragma unroll
    for (int k = 0; k < W; ++k) {
      part[(2 * h) * (W + 1) + k] = dwa[k][h].x;
      part[(2 * h + 1) * (W + 1) + k] = dwa[k][h].y;
    }
    part[(2 * h) * (W + 1) + W] = dba[h].x;
    part[(2 * h + 1) * (W + 1) + W] = dba[h].y;
  }
}

// dw[d][k] and dbias[d] from the partial sums of all (batch, chunk) blocks, in a fixed order: a block owns 32
// adjacent outputs; its 8 slices of threads each add a contiguous range of the parts in ascending order (coalesced
// 128-byte reads, independent loads in flight), and the 8 range sums are added in ascending order through shared memory.
constexpr int kRedOutputs = 32, kRedSlices = 8;
__global__ void __launch_bounds__(kRedOutputs* kRedSlices) ssm_conv1d_reduce_kernel(const float* __restrict__ part, int parts,
                                                                                   int D, int W, float* __restrict__ dw,
                                                                                   float* __restrict__ dbias) {
  __shared__ float s_sum[kRedSlices][kRedOutputs];
  const int lane = threadIdx.x % kRedOutputs, slice = threadIdx.x / kRedOutputs;
  const int n = D * (W + 1);
  const int i = blockIdx.x * kRedOutputs + lane;   // index into [D][W + 1]
  const int per = (parts + kRedSlices - 1) / kRedSlices;
  const int q0 = min(parts, slice * per), q1 = min(parts, q0 + per);
  float s = 0.f;
  if (i < n) {
#pragma unroll 4
    for (int q = q0; q < q1; ++q) s += part[(size_t)q * n + i];
  }
  s_sum[slice][lane] = s;
  __syncthreads();
  if (slice == 0 && i < n) {
    float tot = s_sum[0][lane];
#pragma unroll
    for (int r = 1; r < kRedSlices; ++r) tot += s_sum[r][lane];
    const int d = i / (W + 1), k = i % (W + 1);
    if (k < W) dw[(size_t)d * W + k] = tot;
    else if (dbias != nullptr) dbias[d] = tot;
  }
}

// Steps per chunk.  Every block costs about (steps + W - 1) row visits and the blocks run in
// ceil(blocks / resident blocks) rounds, so the run time goes like rounds * (steps + W - 1): pick the chunk length in
// [kConvMinSteps, kConvMaxSteps] that minimises it (a grid that fills the GPU a whole number of times; for small
// problems the shortest chunk, i.e. the most parallelism), longer chunks winning ties (fewer halo rows).
int choose_steps(long long blocks_per_chunk, int L, int W, long long resident) {
  int best = kConvMinSteps;
  long long best_cost = -1;
  for (int steps = kConvMinSteps; steps <= kConvMaxSteps; ++steps) {
    const long long chunks = (L + steps - 1) / steps;
    const long long rounds = (blocks_per_chunk * chunks + resident - 1) / resident;
    const long long cost = rounds * (steps + W - 1);
    if (best_cost < 0 || cost <= best_cost) {
      best_cost = cost;
      best = steps;
    }
  }
  return best;
}

template <typename Kernel>
cudaError_t launch_conv_kernel(Kernel kernel, ConvParams p, int W, int channels_per_thread, int* chunks_out, cudaStream_t s) {
  const int vecs = (p.D + channels_per_thread - 1) / channels_per_thread;
  const int gx = (vecs + kConvThreads - 1) / kConvThreads;
  int dev = 0, sms = 0, per_sm = 0;
  cudaError_t e;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kConvThreads, 0)) != cudaSuccess) return e;
  p.steps = choose_steps((long long)gx * p.batch, p.L, W, (long long)sms * (per_sm > 0 ? per_sm : 1));
  const int chunks = (p.L + p.steps - 1) / p.steps;
  if (chunks_out != nullptr) *chunks_out = chunks;
  dim3 grid(gx, chunks, p.batch);
  kernel<<<grid, kConvThreads, 0, s>>>(p);
  return cudaGetLastError();
}

// vector_ok: four channels per thread with packed arithmetic; otherwise the scalar kernels.  The tanh-based sigmoid is
// used for bf16 io only.
template <typename IO, int W>
cudaError_t launch_conv_w(const ConvParams& p, bool backward, bool vector_ok, int* chunks, cudaStream_t s) {
  constexpr bool FAST = sizeof(IO) == 2;
  if (!vector_ok)
    return backward ? launch_conv_kernel(ssm_conv1d_bwd_kernel<IO, W, 1>, p, W, 1, chunks, s)
                    : launch_conv_kernel(ssm_conv1d_fwd_kernel<IO, W, 1>, p, W, 1, chunks, s);
  if (p.silu)
    return backward ? launch_conv_kernel(ssm_conv1d_bwd_vec4_kernel<IO, W, true, FAST>, p, W, 4, chunks, s)
                    : launch_conv_kernel(ssm_conv1d_fwd_vec4_kernel<IO, W, true, FAST>, p, W, 4, chunks, s);
  return backward ? launch_conv_kernel(ssm_conv1d_bwd_vec4_kernel<IO, W, false, FAST>, p, W, 4, chunks, s)
                  : launch_conv_kernel(ssm_conv1d_fwd_vec4_kernel<IO, W, false, FAST>, p, W, 4, chunks, s);
}

template <typename IO>
cudaError_t launch_conv_io(const ConvParams& p, int W, bool backward, bool vector_ok, int* chunks, cudaStream_t s) {
  switch (W) {
    case 1: return launch_conv_w<IO, 1>(p, backward, vector_ok, chunks, s);
    case 2: return launch_conv_w<IO, 2>(p, backward, vector_ok, chunks, s);
    case 3: return launch_conv_w<IO, 3>(p, backward, vector_ok, chunks, s);
    case 4: return launch_conv_w<IO, 4>(p, backward, vector_ok, chunks, s);
    default: return cudaErrorInvalidValue;
  }
}

ssm_status_t validate_conv(const ssm_conv_problem_t* p) {
  if (p == nullptr || p->batch < 1 || p->L < 1 || p->D < 1) return SSM_ERR_INVALID_ARG;
  if (p->flags & ~(uint32_t)(SSM_CONV_FLAG_SILU | SSM_CONV_FLAG_HAS_BIAS)) return SSM_ERR_INVALID_ARG;
  if (p->io_dtype != SSM_F32 && p->io_dtype != SSM_BF16) return SSM_ERR_UNSUPPORTED;
  if (p->width < 1 || p->width > 4) return SSM_ERR_UNSUPPORTED;
  if (p->batch > 65535 || (p->L + kConvMinSteps - 1) / kConvMinSteps > 65535) return SSM_ERR_UNSUPPORTED;  // grid y / z
  return SSM_OK;
}

inline bool aligned(const void* q, size_t a) { return q == nullptr || (reinterpret_cast<uintptr_t>(q) % a) == 0; }

}  // namespace

}  // namespace ssm

using namespace ssm;

extern "C" {

ssm_status_t ssm_conv1d_fwd(const ssm_conv_problem_t* p, const void* x, const float* w, const float* bias,
                            const void* x_prev, void* y, void* stream) {
  ssm_status_t st = validate_conv(p);
  if (st != SSM_OK) return st;
  const bool has_bias = p->flags & SSM_CONV_FLAG_HAS_BIAS;
  if (!x || !w || !y || (has_bias && !bias)) return SSM_ERR_INVALID_ARG;
  const size_t esz = p->io_dtype == SSM_BF16 ? 2 : 4;
  if (!aligned(x, esz) || !aligned(y, esz) || !aligned(x_prev, esz) || !aligned(w, 4) || !aligned(bias, 4))
    return SSM_ERR_INVALID_ARG;
  ConvParams cp{};
  cp.x = x;
  cp.w = w;
  cp.bias = has_bias ? bias : nullptr;
  cp.x_prev = p->width > 1 ? x_prev : nullptr;
  cp.y = y;
  cp.batch = p->batch;
  cp.L = p->L;
  cp.D = p->D;
  cp.silu = (p->flags & SSM_CONV_FLAG_SILU) ? 1 : 0;
  // 4 elements per access (8 bytes for bf16): a warp still covers whole 128-byte lines of a row, and the smaller
  // register footprint keeps more rows in flight per SM than 16-byte accesses did
  const size_t va = 4 * esz;
  const bool vec_ok = p->D % 4 == 0 && aligned(x, va) && aligned(y, va) && aligned(x_prev, va);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const cudaError_t e = p->io_dtype == SSM_BF16 ? launch_conv_io<__nv_bfloat16>(cp, p->width, false, vec_ok, nullptr, s)
                                                : launch_conv_io<float>(cp, p->width, false, vec_ok, nullptr, s);
  return e == cudaSuccess ? SSM_OK : SSM_ERR_CUDA;
}

size_t ssm_conv1d_bwd_workspace_bytes(const ssm_conv_problem_t* p) {
  if (validate_conv(p) != SSM_OK) return 0;
  // room for the shortest chunk the launch may choose
  const size_t parts = (size_t)p->batch * ((p->L + kConvMinSteps - 1) / kConvMinSteps);
  return parts * p->D * (p->width + 1) * sizeof(float);
}

ssm_status_t ssm_conv1d_bwd(const ssm_conv_problem_t* p, const void* x, const float* w, const float* bias,
                            const void* x_prev, const void* dy, void* dx, float* dw, float* dbias, void* dx_prev,
                            void* workspace, size_t workspace_bytes, void* stream) {
  ssm_status_t st = validate_conv(p);
  if (st != SSM_OK) return st;
  const bool has_bias = p->flags & SSM_CONV_FLAG_HAS_BIAS;
  if (!x || !w || !dy || !dx || !dw || (has_bias && !bias)) return SSM_ERR_INVALID_ARG;
  const size_t esz = p->io_dtype == SSM_BF16 ? 2 : 4;
  for (const void* q : {x, dy, (const void*)dx, x_prev, (const void*)dx_prev})
    if (!aligned(q, esz)) return SSM_ERR_INVALID_ARG;
  for (const void* q : {(const void*)w, (const void*)bias, (const void*)dw, (const void*)dbias})
    if (!aligned(q, 4)) return SSM_ERR_INVALID_ARG;
  const size_t need = ssm_conv1d_bwd_workspace_bytes(p);
  if (workspace == nullptr || !aligned(workspace, 16) || workspace_bytes < need) return SSM_ERR_WORKSPACE;
  ConvParams cp{};
  cp.x = x;
  cp.w = w;
  cp.bias = has_bias ? bias : nullptr;
  cp.x_prev = p->width > 1 ? x_prev : nullptr;
  cp.dy = dy;
  cp.dx = dx;
  cp.dx_prev = p->width > 1 ? dx_prev : nullptr;
  cp.part = static_cast<float*>(workspace);
  cp.batch = p->batch;
  cp.L = p->L;
  cp.D = p->D;
  cp.silu = (p->flags & SSM_CONV_FLAG_SILU) ? 1 : 0;
  const size_t va = 4 * esz;
  const bool vec_ok = p->D % 4 == 0 && aligned(x, va) && aligned(dy, va) && aligned(dx, va) && aligned(x_prev, va) &&
                      aligned(dx_prev, va);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int chunks = 0;
  cudaError_t e = p->io_dtype == SSM_BF16 ? launch_conv_io<__nv_bfloat16>(cp, p->width, true, vec_ok, &chunks, s)
                                          : launch_conv_io<float>(cp, p->width, true, vec_ok, &chunks, s);
  if (e != cudaSuccess) return SSM_ERR_CUDA;
  const int parts = p->batch * chunks;
  const int n = p->D * (p->width + 1);
  ssm_conv1d_reduce_kernel<<<(n + kRedOutputs - 1) / kRedOutputs, kRedOutputs * kRedSlices, 0, s>>>(
      cp.part, parts, p->D, p->width, dw, has_bias ? dbias : nullptr);
  return cudaGetLastError() == cudaSuccess ? SSM_OK : SSM_ERR_CUDA;
}

}  // extern "C"
