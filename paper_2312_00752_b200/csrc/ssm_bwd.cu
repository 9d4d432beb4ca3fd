// Backward selective scan with recomputation (Section 3.3: "the intermediate states are not stored but recomputed
// in the backward pass"; Appendix D, "Memory").
//
// For loss = sum(dout * out) the adjoint of Eq. 2a/2b with the skip term and the gate is, per (batch, channel):
//     ds_t   = dout_t * silu(z_t),      dz_t = dout_t * s_t * sig(z_t) (1 + z_t (1 - sig(z_t)))
//     lam_t  = C_t ds_t + mu_{t+1},     mu_t = a_t lam_t                  (reverse-time recurrence, mu_{L+1} = 0)
//     dC_t  += ds_t h_t,  dB_t += lam_t delta_t x_t                        (summed over channels)
//     dx_t   = ds_t D_skip + delta_t sum_n lam_t B_t
//     w_t    = mu_t h_{t-1};  ddelta_t = sum_n w_t A + x_t sum_n lam_t B_t;  dA += w_t delta_t;  dD += ds_t x_t
// A block walks its time segment backwards one tile (kBwdTile steps, a whole number of checkpoint blocks) at a time: it
// reloads the inputs of the tile, recomputes h_t forward from the tile's first checkpoint state into shared memory,
// then runs the reverse recurrence over the tile.  Thread layout as in the forward kernel with one channel per thread group.
//
// Reductions are deterministic: dB/dC are summed over the channels of a warp with a fixed xor-shuffle tree, over the
// warps of the block in ascending order, written as per-block partial sums and finally summed over blocks in
// ascending order by ssm_bwd_reduce_kernel; dA/dD are accumulated per thread over time, written per
// (batch, segment) and summed in ascending order by the same kernel.  No floating-point atomics.
#include "ssm_common.cuh"

namespace ssm {

// one checkpoint block per tile: the recomputed states of a tile then take little shared memory and several blocks fit
// an SM (tiles of 32 steps were measured 1.5 to 3 times slower)
constexpr int kBwdTile = 8;
static_assert(kBwdTile % kCkptSteps == 0, "a tile starts on a checkpoint");

template <int N>
struct BwdGeom {
  static constexpr int S = N < 4 ? N : 4;
  static constexpr int LPC = N / S;             // lanes per channel
  // channels per block (one per thread group); fewer for N > 16 so that the recomputed states of a tile fit
  static constexpr int CH = N <= 16 ? 32 : (N == 32 ? 16 : 8);
  static constexpr int THREADS = CH * LPC;
  static constexpr int WARPS = THREADS / 32;
};

template <typename IO, int N>
constexpr size_t bwd_smem_bytes() {
  using G = BwdGeom<N>;
  return sizeof(float) * ((size_t)(kBwdTile + 1) * G::CH * N   // h_0 .. h_T
                          + 2 * (size_t)kBwdTile * N           // B, C
                          + (size_t)kBwdTile * G::CH           // s (pre-gate readout)
                          + (size_t)G::WARPS * kBwdTile * 2 * N)  // per-warp dB/dC sums
         + sizeof(IO) * 4 * (size_t)kBwdTile * G::CH;          // x, delta, z, dout (reused for dx, ddelta, dz)
}

template <typename IO, int N>
__global__ void __launch_bounds__(BwdGeom<N>::THREADS) ssm_bwd_kernel(const BwdParams p) {
  using G = BwdGeom<N>;
  constexpr int S = G::S, LPC = G::LPC, CH = G::CH, WARPS = G::WARPS, T = kBwdTile;
  constexpr int kBwdThreads = G::THREADS;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* s_h = reinterpret_cast<float*>(smem_raw);            // [T+1][CH][N]
  float* s_B = s_h + (size_t)(T + 1) * CH * N;                // [T][N]
  float* s_C = s_B + T * N;                                   // [T][N]
  float* s_s = s_C + T * N;                                   // [T][CH]
  float* s_part = s_s + T * CH;                               // [WARPS][T][2][N]
  IO* s_x = reinterpret_cast<IO*>(s_part + (size_t)WARPS * T * 2 * N);  // [T][CH]  (becomes dx)
  IO* s_d = s_x + T * CH;                                     // [T][CH]  (becomes ddelta)
  IO* s_z = s_d + T * CH;                                     // [T][CH]  (becomes dz)
  IO* s_g = s_z + T * CH;                                     // [T][CH]

  const IO* __restrict__ gx = static_cast<const IO*>(p.x);
  const IO* __restrict__ gd = static_cast<const IO*>(p.delta);
  const IO* __restrict__ gz = static_cast<const IO*>(p.z);
  const IO* __restrict__ gg = static_cast<const IO*>(p.dout);
  const IO* __restrict__ gB = static_cast<const IO*>(p.B);
  const IO* __restrict__ gC = static_cast<const IO*>(p.C);
  IO* __restrict__ gdx = static_cast<IO*>(p.dx);
  IO* __restrict__ gdd = static_cast<IO*>(p.ddelta);
  IO* __restrict__ gdz = static_cast<IO*>(p.dz);

  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int j = tid % LPC;
  const int slot = tid / LPC;
  const int d_cta = blockIdx.x * CH;
  const int seg = blockIdx.y;
  const int b = blockIdx.z;
  const int D = p.D;
  const int d = d_cta + slot;
  const bool valid = d < D;
  const int t_begin = seg * p.seg_steps;
  const int t_end = min(p.L, t_begin + p.seg_steps);
  const bool has_z = gz != nullptr;

  float Ar[S], A2[S], mu[S], dA[S];
  float Bst[S], Cst[S], dBs[S], dCs[S];   // static B / C (parameters [D][N]) and their gradient sums over time
  float dD_acc = 0.f, dbias_acc = 0.f;
  const float Dk = (valid && p.Dskip != nullptr) ? p.Dskip[d] : 0.f;
  const float dbias = (valid && p.delta_bias != nullptr) ? p.delta_bias[d] : 0.f;
#pragma unroll
  for (int k = 0; k < S; ++k) {
    Ar[k] = valid ? p.A[(size_t)d * N + j * S + k] : 0.f;
    Bst[k] = (valid && p.static_B) ? static_cast<const float*>(p.B)[(size_t)d * N + j * S + k] : 0.f;
    Cst[k] = (valid && p.static_C) ? static_cast<const float*>(p.C)[(size_t)d * N + j * S + k] : 0.f;
    dBs[k] = dCs[k] = 0.f;
    A2[k] = Ar[k] * kLog2e;
    mu[k] = (valid && p.mu_in != nullptr) ? p.mu_in[(((size_t)b * p.nseg + seg) * D + d) * N + j * S + k] : 0.f;
    dA[k] = 0.f;
  }

  const int kb_first = t_begin / T;
  const int kb_last = (t_end - 1) / T;
  for (int kb = kb_last; kb >= kb_first; --kb) {
    const int t0 = kb * T;
    const int nt = min(T, t_end - t0);
    const size_t row0 = (size_t)b * p.L + t0;
    __syncthreads();
    for (int i = tid; i < T * CH; i += kBwdThreads) {
      const int tt = i / CH, c = i % CH;
      const bool ok = tt < nt && d_cta + c < D;
      const size_t g = (row0 + tt) * D + d_cta + c;
      const IO zero = float_to_io<IO>(0.f);
      s_x[i] = ok ? gx[g] : zero;
      s_d[i] = ok ? gd[g] : zero;
      s_z[i] = (ok && has_z) ? gz[g] : zero;
      s_g[i] = ok ? gg[g] : zero;
    }
    for (int i = tid; i < T * N; i += kBwdThreads) {
      const bool ok = i / N < nt;
      s_B[i] = (ok && !p.static_B) ? io_to_float<IO>(gB[row0 * N + i]) : 0.f;
      s_C[i] = (ok && !p.static_C) ? io_to_float<IO>(gC[row0 * N + i]) : 0.f;
    }
    float h[S];
#pragma unroll
    for (int k = 0; k < S; ++k) {
      h[k] = valid ? p.ckpt[ckpt_offset(p.ckpt_tiled, b, p.nck, kb * (T / kCkptSteps), D, N, d, j * S + k)] : 0.f;
      s_h[(size_t)slot * N + j * S + k] = h[k];
    }
    __syncthreads();

    // ---- recompute h_1 .. h_nt of this block and the pre-gate readout s_t
    for (int tt = 0; tt < nt; ++tt) {
      float dt = io_to_float<IO>(s_d[tt * CH + slot]) + dbias;
      if (p.softplus) dt = softplus_precise(dt);
      const float u = io_to_float<IO>(s_x[tt * CH + slot]);
      const float du = dt * u;
      float y = 0.f;
#pragma unroll
      for (int k = 0; k < S; ++k) {
        const float Bk = p.static_B ? Bst[k] : s_B[tt * N + j * S + k];
        float a, bx = du * Bk;
        if (p.zoh) {
          float E;
          zoh_discretize(dt, Ar[k], a, E);
          bx = E * u * Bk;
        } else {
          a = ex2_approx(dt * A2[k]);
        }
        h[k] = fmaf(a, h[k], bx);
        y = fmaf(p.static_C ? Cst[k] : s_C[tt * N + j * S + k], h[k], y);
        s_h[((size_t)(tt + 1) * CH + slot) * N + j * S + k] = h[k];
      }
#pragma unroll
      for (int m = LPC / 2; m >= 1; m >>= 1) y += __shfl_xor_sync(0xffffffffu, y, m);
      if (j == 0) s_s[tt * CH + slot] = fmaf(Dk, u, y);
    }
    __syncwarp();

    // ---- reverse recurrence over the block
    for (int tt = nt - 1; tt >= 0; --tt) {
      const float dv = io_to_float<IO>(s_d[tt * CH + slot]) + dbias;
      const float dt = p.softplus ? softplus_precise(dv) : dv;
      const float u = io_to_float<IO>(s_x[tt * CH + slot]);
      const float g = io_to_float<IO>(s_g[tt * CH + slot]);
      const float du = dt * u;
      float ds = g, dzv = 0.f;
      if (has_z) {
        const float zz = io_to_float<IO>(s_z[tt * CH + slot]);
        const float sg = sigmoid_fast(zz);
        ds = g * zz * sg;
        dzv = g * s_s[tt * CH + slot] * sg * fmaf(zz, 1.f - sg, 1.f);
      }
      // lamB = sum_n lam B (default rule; with ZOH sum_n lam E B, the input gradient), lamGB = sum_n lam a B (ZOH
      // only: the step-size gradient through E, dE/ddelta = a)
      float lamB = 0.f, lamGB = 0.f, wA = 0.f;
      float dBp[S], dCp[S];
#pragma unroll
      for (int k = 0; k < S; ++k) {
        const float ht = s_h[((size_t)(tt + 1) * CH + slot) * N + j * S + k];
        const float hp = s_h[((size_t)tt * CH + slot) * N + j * S + k];
        const float Bn = p.static_B ? Bst[k] : s_B[tt * N + j * S + k];
        const float lam = fmaf(p.static_C ? Cst[k] : s_C[tt * N + j * S + k], ds, mu[k]);
        dCp[k] = ds * ht;
        float a;
        if (p.zoh) {
          // B-bar = E B with E = (a - 1) / A: dE/ddelta = a, dE/dA = (dt a - E) / A
          float E;
          zoh_discretize(dt, Ar[k], a, E);
          dBp[k] = lam * E * u;
          lamB = fmaf(lam * E, Bn, lamB);
          lamGB = fmaf(lam * a, Bn, lamGB);
          dA[k] = fmaf(lam * zoh_gain_dA(dt, Ar[k], a, E), Bn * u, dA[k]);
        } else {
          a = ex2_approx(dt * A2[k]);
          dBp[k] = lam * du;
          lamB = fmaf(lam, Bn, lamB);
        }
        dBs[k] += dBp[k];   // static B / C: the same terms summed over time instead of over channels
        dCs[k] += dCp[k];
        mu[k] = a * lam;
        const float w = mu[k] * hp;
        wA = fmaf(w, Ar[k], wA);
        dA[k] = fmaf(w, dt, dA[k]);
      }
#pragma unroll
      for (int m = LPC / 2; m >= 1; m >>= 1) {
        lamB += __shfl_xor_sync(0xffffffffu, lamB, m);
        lamGB += __shfl_xor_sync(0xffffffffu, lamGB, m);
        wA += __shfl_xor_sync(0xffffffffu, wA, m);
      }
      // sum dB/dC over the channels held by this warp (lanes that share j)
#pragma unroll
      for (int k = 0; k < S; ++k) {
#pragma unroll
        for (int m = 16; m >= LPC; m >>= 1) {
          dBp[k] += __shfl_xor_sync(0xffffffffu, dBp[k], m);
          dCp[k] += __shfl_xor_sync(0xffffffffu, dCp[k], m);
        }
      }
      if (lane < LPC) {
#pragma unroll
        for (int k = 0; k < S; ++k) {
          s_part[(((size_t)warp * T + tt) * 2 + 0) * N + j * S + k] = dBp[k];
          s_part[(((size_t)warp * T + tt) * 2 + 1) * N + j * S + k] = dCp[k];
        }
      }
      if (j == 0) {
        dD_acc = fmaf(ds, u, dD_acc);
        // with the softplus the gradient goes to the pre-activation: d softplus(v)/dv = sigmoid(v)
        const float ddv = fmaf(u, p.zoh ? lamGB : lamB, wA) * (p.softplus ? 1.f / (1.f + __expf(-dv)) : 1.f);
        dbias_acc += ddv;
        s_x[tt * CH + slot] = float_to_io<IO>(fmaf(ds, Dk, p.zoh ? lamB : dt * lamB));
        s_d[tt * CH + slot] = float_to_io<IO>(ddv);
        s_z[tt * CH + slot] = float_to_io<IO>(dzv);
      }
    }
    __syncthreads();

    for (int i = tid; i < nt * CH; i += kBwdThreads) {
      const int tt = i / CH, c = i % CH;
      if (d_cta + c < D) {
        const size_t g = (row0 + tt) * D + d_cta + c;
        gdx[g] = s_x[i];
        gdd[g] = s_d[i];
        if (gdz != nullptr) gdz[g] = s_z[i];
      }
    }
    const size_t bln = (size_t)p.batch * p.L * N;
    for (int i = tid; i < nt * 2 * N; i += kBwdThreads) {
      const int tt = i / (2 * N), which = (i / N) & 1, n = i % N;
      float acc = 0.f;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) acc += s_part[(((size_t)w * T + tt) * 2 + which) * N + n];
      p.dBC_part[((size_t)blockIdx.x * 2 + which) * bln + (row0 + tt) * N + n] = acc;
    }
  }

  if (valid) {
    const size_t part = (size_t)b * p.nseg + seg;
#pragma unroll
    for (int k = 0; k < S; ++k) p.dA_part[(part * D + d) * N + j * S + k] = dA[k];
    if (j == 0) p.dD_part[part * D + d] = dD_acc;
    if (j == 0 && p.dbias_part != nullptr) p.dbias_part[part * D + d] = dbias_acc;
#pragma unroll
    for (int k = 0; k < S; ++k) {
      if (p.static_B) p.dBs_part[(part * D + d) * N + j * S + k] = dBs[k];
      if (p.static_C) p.dCs_part[(part * D + d) * N + j * S + k] = dCs[k];
    }
    if (seg == 0 && p.dh0 != nullptr) {
#pragma unroll
      for (int k = 0; k < S; ++k) p.dh0[((size_t)b * D + d) * N + j * S + k] = mu[k];
    }
  }
}

// First pass of the reverse time split: the adjoint mu that leaves each segment when nothing flows into it, and the
// segment's sum of delta.  Only the lam/mu recurrence is needed (no states).
template <typename IO, int N>
__global__ void __launch_bounds__(BwdGeom<N>::THREADS) ssm_bwd_local_kernel(const BwdParams p) {
  using G = BwdGeom<N>;
  constexpr int S = G::S, LPC = G::LPC, CH = G::CH, T = kBwdTile;
  constexpr int kBwdThreads = G::THREADS;
  __shared__ __align__(16) IO s_d[T * CH];
  __shared__ __align__(16) IO s_z[T * CH];
  __shared__ __align__(16) IO s_g[T * CH];
  __shared__ __align__(16) float s_C[T * N];

  const IO* __restrict__ gd = static_cast<const IO*>(p.delta);
  const IO* __restrict__ gz = static_cast<const IO*>(p.z);
  const IO* __restrict__ gg = static_cast<const IO*>(p.dout);
  const IO* __restrict__ gC = static_cast<const IO*>(p.C);
  const int tid = threadIdx.x;
  const int j = tid % LPC, slot = tid / LPC;
  // (segment 0 has no earlier segment to hand its adjoint to: it is not computed)
  const int d_cta = blockIdx.x * CH, seg = blockIdx.y + 1, b = blockIdx.z;
  const int D = p.D, d = d_cta + slot;
  const bool valid = d < D;
  const int t_begin = seg * p.seg_steps;
  const int t_end = min(p.L, t_begin + p.seg_steps);
  const bool has_z = gz != nullptr;

  float A2[S], mu[S], Cst[S], dsum = 0.f;
  const float dbias = (valid && p.delta_bias != nullptr) ? p.delta_bias[d] : 0.f;
#pragma unroll
  for (int k = 0; k < S; ++k) {
    A2[k] = valid ? p.A[(size_t)d * N + j * S + k] * kLog2e : 0.f;
    Cst[k] = (valid && p.static_C) ? static_cast<const float*>(p.C)[(size_t)d * N + j * S + k] : 0.f;
    mu[k] = 0.f;
  }
  for (int kb = (t_end - 1) / T; kb >= t_begin / T; --kb) {
    const int t0 = kb * T;
    const int nt = min(T, t_end - t0);
    const size_t row0 = (size_t)b * p.L + t0;
    __syncthreads();
    for (int i = tid; i < T * CH; i += kBwdThreads) {
      const int tt = i / CH, c = i % CH;
      const bool ok = tt < nt && d_cta + c < D;
      const size_t g = (row0 + tt) * D + d_cta + c;
      const IO zero = float_to_io<IO>(0.f);
      s_d[i] = ok ? gd[g] : zero;
      s_z[i] = (ok && has_z) ? gz[g] : zero;
      s_g[i] = ok ? gg[g] : zero;
    }
    for (int i = tid; i < T * N; i += kBwdThreads)
      s_C[i] = (i / N < nt && !p.static_C) ? io_to_float<IO>(gC[row0 * N + i]) : 0.f;
    __syncthreads();
    for (int tt = nt - 1; tt >= 0; --tt) {
      float dt = io_to_float<IO>(s_d[tt * CH + slot]) + dbias;
      if (p.softplus) dt = softplus_precise(dt);
      float ds = io_to_float<IO>(s_g[tt * CH + slot]);
      if (has_z) {
        const float zz = io_to_float<IO>(s_z[tt * CH + slot]);
        ds = ds * zz * sigmoid_fast(zz);
      }
      dsum += dt;
#pragma unroll
      for (int k = 0; k < S; ++k)
        mu[k] = ex2_approx(dt * A2[k]) * fmaf(p.static_C ? Cst[k] : s_C[tt * N + j * S + k], ds, mu[k]);
    }
  }
  if (valid) {
    const size_t sg = (size_t)b * p.nseg + seg;
#pragma unroll
    for (int k = 0; k < S; ++k) p.seg_local[(sg * D + d) * N + j * S + k] = mu[k];
    if (j == 0) p.seg_dsum[sg * D + d] = dsum;
  }
}

// Second stage of the deterministic reductions: sums the per-block dB/dC partials over channel groups and the
// per-(batch, segment) dA/dD partials, in ascending order, and rounds dB/dC to the io dtype.
template <typename IO>
__global__ void __launch_bounds__(256) ssm_bwd_reduce_kernel(const ReduceParams p) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < p.bln) {
    float sb = 0.f, sc = 0.f;
    for (int g = 0; g < p.groups; ++g) {
      sb += p.dBC_part[((size_t)g * 2 + 0) * p.bln + i];
      sc += p.dBC_part[((size_t)g * 2 + 1) * p.bln + i];
    }
    if (p.dB != nullptr) static_cast<IO*>(p.dB)[i] = float_to_io<IO>(sb);
    if (p.dC != nullptr) static_cast<IO*>(p.dC)[i] = float_to_io<IO>(sc);
  }
  const long long dn = (long long)p.D * p.N;
  if (i < dn) {
    float sa = 0.f;
    for (int q = 0; q < p.parts; ++q) sa += p.dA_part[(size_t)q * dn + i];
    p.dA[i] = sa;
    if (p.dBs != nullptr) {
      float v = 0.f;
      for (int q = 0; q < p.parts; ++q) v += p.dBs_part[(size_t)q * dn + i];
      p.dBs[i] = v;
    }
    if (p.dCs != nullptr) {
      float v = 0.f;
      for (int q = 0; q < p.parts; ++q) v += p.dCs_part[(size_t)q * dn + i];
      p.dCs[i] = v;
    }
  }
  if (p.dD != nullptr && i < p.D) {
    float sd = 0.f;
    for (int q = 0; q < p.parts; ++q) sd += p.dD_part[(size_t)q * p.D + i];
    p.dD[i] = sd;
  }
  if (p.dbias != nullptr && i < p.D) {
    float sb = 0.f;
    for (int q = 0; q < p.parts; ++q) sb += p.dbias_part[(size_t)q * p.D + i];
    p.dbias[i] = sb;
  }
}

template <typename IO, int N>
static cudaError_t launch_bwd_n(const Plan& plan, const BwdParams& p, int mode, cudaStream_t s) {
  using G = BwdGeom<N>;
  dim3 grid((p.D + G::CH - 1) / G::CH, plan.nseg, p.batch);
  constexpr int kBwdThreads = G::THREADS;
  if (mode == kBwdLocal) {
    if (plan.nseg < 2) return cudaSuccess;
    grid.y = plan.nseg - 1;
    ssm_bwd_local_kernel<IO, N><<<grid, kBwdThreads, 0, s>>>(p);
    return cudaGetLastError();
  }
  constexpr size_t smem = bwd_smem_bytes<IO, N>();
  cudaError_t e = cudaFuncSetAttribute(ssm_bwd_kernel<IO, N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  ssm_bwd_kernel<IO, N><<<grid, kBwdThreads, smem, s>>>(p);
  return cudaGetLastError();
}

template <typename IO>
static cudaError_t launch_bwd_io(const ssm_problem_t& prob, const Plan& plan, const BwdParams& p, int mode,
                                 cudaStream_t s) {
  switch (prob.N) {
    case 64: return launch_bwd_n<IO, 64>(plan, p, mode, s);
    case 32: return launch_bwd_n<IO, 32>(plan, p, mode, s);
    case 16: return launch_bwd_n<IO, 16>(plan, p, mode, s);
    case 8: return launch_bwd_n<IO, 8>(plan, p, mode, s);
    case 4: return launch_bwd_n<IO, 4>(plan, p, mode, s);
    case 2: return launch_bwd_n<IO, 2>(plan, p, mode, s);
    case 1: return launch_bwd_n<IO, 1>(plan, p, mode, s);
    default: return cudaErrorInvalidValue;
  }
}

int bwd_channels_per_block(int N) { return N <= 16 ? 32 : (N == 32 ? 16 : 8); }

bool bwd_fast_applicable(const ssm_problem_t& prob, const BwdParams& p);
cudaError_t launch_bwd_fast(const Plan& plan, const BwdParams& p, cudaStream_t s);

bool bwd_local_fast_applicable(const ssm_problem_t& prob, const BwdParams& p);
cudaError_t launch_bwd_local_fast(const Plan& plan, const BwdParams& p, cudaStream_t s);

cudaError_t launch_bwd(const ssm_problem_t& prob, const Plan& plan, const BwdParams& p, int mode, cudaStream_t s) {
  if (mode == kBwdFull && bwd_fast_applicable(prob, p)) return launch_bwd_fast(plan, p, s);
  if (mode == kBwdLocal && bwd_local_fast_applicable(prob, p)) return launch_bwd_local_fast(plan, p, s);
  if (prob.io_dtype == SSM_BF16) return launch_bwd_io<__nv_bfloat16>(prob, plan, p, mode, s);
  return launch_bwd_io<float>(prob, plan, p, mode, s);
}

cudaError_t launch_bwd_reduce(const ssm_problem_t& prob, const ReduceParams& p, cudaStream_t s) {
  const long long work = p.bln > (long long)p.D * p.N ? p.bln : (long long)p.D * p.N;
  const unsigned blocks = (unsigned)((work + 255) / 256);
  if (prob.io_dtype == SSM_BF16) ssm_bwd_reduce_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>(p);
  else ssm_bwd_reduce_kernel<float><<<blocks, 256, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace ssm
