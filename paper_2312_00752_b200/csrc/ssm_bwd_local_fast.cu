// First pass of the reverse time split, tuned path (bf16 io, N = 16, D % 8 == 0, 16-byte aligned pointers): for every
// time segment the adjoint that leaves the segment when nothing flows into it,
//     mu_t = a_t (C_t ds_t + mu_{t+1}),   mu_{end+1} = 0,   ds_t = dout_t * silu(z_t),   a_t = exp(delta_t A),
// evaluated from the last step of the segment to the first, and the segment's sum of delta (the adjoint of Eq. 2a and
// of the gate; the segment results are then combined by the reversed carry scan of ssm_carry.cu, Appendix D).
// Only this lambda / mu recurrence is needed here: no states, no x, no B.
//
// Same construction as the tuned forward kernel run backwards in time: a thread owns 4 states of 2 adjacent channels as
// packed float2 pairs, 4 lanes cover the 16 states of the pair, a warp 16 channels; a block has 2 compute warps and a
// service warp that stages delta, z, dout and C with 16-byte cp.async copies into a three-stage ring of 32-step tiles
// (walked from the last tile of the segment to the first) and widens C to float; each compute warp turns dout and z of
// its own channels into ds once per element, half a tile at a time, in a strip of shared memory of its own.
#include <type_traits>

#include "ssm_common.cuh"

namespace ssm {

namespace {

constexpr int kTT = 32;     // steps per tile
constexpr int kNST = 3;     // ring stages
constexpr int kHalf = 16;   // steps whose ds a compute warp prepares at a time
constexpr int kWarps = 2;   // compute warps per block
constexpr int kCH = 16 * kWarps;
constexpr int kThreads = (kWarps + 1) * 32;

struct LocalSmem {
  uint32_t d[kNST][kTT][kCH / 2];
  uint32_t z[kNST][kTT][kCH / 2];
  uint32_t g[kNST][kTT][kCH / 2];
  uint32_t rawC[2][kTT][8];
  float4 fC[2][kTT][4];
  float ds[kWarps][kHalf][16];
  float dt[kWarps][kHalf][16];   // fused step size only: softplus(delta_pre + bias) of half a tile, per warp
};

__device__ __forceinline__ void block_barrier() { asm volatile("bar.sync 1, %0;" ::"r"(kThreads) : "memory"); }
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

}  // namespace

// SP: `delta` holds the pre-activation and the step size is delta + bias, through the softplus if asked (Algorithm 2 step 4)
template <bool SP>
__global__ void __launch_bounds__(kThreads) ssm_bwd_local_fast_kernel(const BwdParams p) {
  __shared__ __align__(16) LocalSmem sm;
  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int d_cta = blockIdx.x * kCH;
  const int seg = blockIdx.y + 1;   // segment 0 has no earlier segment to hand its adjoint to: it is not computed
  const int b = blockIdx.z;
  const int D = p.D;
  const int t_begin = seg * p.seg_steps;
  const int t_end = min(p.L, t_begin + p.seg_steps);
  const int ntiles = (t_end - t_begin + kTT - 1) / kTT;
  const bool has_z = p.z != nullptr;
  constexpr int CHUNKS = kCH / 8;

  if (warp == kWarps) {
    // ================================================================== service warp
    const __nv_bfloat16* __restrict__ gd = static_cast<const __nv_bfloat16*>(p.delta);
    const __nv_bfloat16* __restrict__ gz = static_cast<const __nv_bfloat16*>(p.z);
    const __nv_bfloat16* __restrict__ gg = static_cast<const __nv_bfloat16*>(p.dout);
    const __nv_bfloat16* __restrict__ gC = static_cast<const __nv_bfloat16*>(p.C);
    auto issue_tile = [&](int i) {   // i counts tiles from the END of the segment
      if (i < ntiles) {
        const int st = i % kNST;
        const int t0 = t_begin + (ntiles - 1 - i) * kTT;
        const size_t row0 = (size_t)b * p.L + t0;
#pragma unroll
        for (int c = lane; c < kTT * CHUNKS; c += 32) {
          const int tt = c / CHUNKS, cc = c % CHUNKS;
          const bool ok = (d_cta + cc * 8 < D) && (t0 + tt < t_end);
          const size_t g = ok ? (row0 + tt) * D + d_cta + cc * 8 : 0;
          cp_async16(&sm.d[st][tt][cc * 4], gd + g, ok);
          cp_async16(&sm.z[st][tt][cc * 4], (has_z ? gz : gd) + g, ok && has_z);
          cp_async16(&sm.g[st][tt][cc * 4], gg + g, ok);
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int c = lane + 32 * k;
          const int tt = c >> 1, hc = c & 1;
          const bool ok = t0 + tt < t_end;
          const size_t g = ok ? (row0 + tt) * 16 + hc * 8 : 0;
          cp_async16(&sm.rawC[i & 1][tt][hc * 4], gC + g, ok);
        }
      }
      cp_async_commit();
    };
    auto widen_C = [&](int i) {
      if (i >= ntiles) return;
      const int fb = i & 1;
#pragma unroll
      for (int k = 0; k < kTT * 8 / 32; ++k) {
        const int c = lane + 32 * k;
        const int tt = c >> 3, w = c & 7;
        const uint32_t vc = sm.rawC[fb][tt][w];
        reinterpret_cast<float2*>(&sm.fC[fb][tt][0])[w] = make_float2(bf16lo(vc), bf16hi(vc));
      }
    };
    issue_tile(0);
    issue_tile(1);
    cp_async_wait_but_one();
    __syncwarp();
    widen_C(0);
    for (int i = 0; i < ntiles; ++i) {
      block_barrier();        // tile i is staged; the compute warps are done with tile i-1
      issue_tile(i + 2);      // overwrites the ring stage of tile i-1
      cp_async_wait_but_one();
      __syncwarp();
      widen_C(i + 1);
    }
    cp_async_wait_all();
    block_barrier();
    return;
  }

  // ==================================================================== compute warps
  const int j = lane & 3;
  const int slot = warp * 8 + (lane >> 2);
  const int d0 = d_cta + 2 * slot;
  const bool valid = d0 < D;
  const int pq = j & 1;
  const uint32_t selA = pq ? 0x3244u : 0x1044u, selB = pq ? 0x1044u : 0x3244u;
  auto chan = [&](int q) { return d0 + (q ^ pq); };

  float2 A2[2][2], mu[2][2];
  float dsum[2] = {0.f, 0.f};
  bool ap = !p.general_A;
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid) a = *reinterpret_cast<const float4*>(p.A + (size_t)chan(q) * 16 + 4 * j);
    const float step = a.y - a.x, tol = 1e-6f * fabsf(a.w);
    ap = ap && fabsf(a.z - (a.x + 2.f * step)) <= tol && fabsf(a.w - (a.x + 3.f * step)) <= tol;
    A2[q][0] = make_float2(a.x * kLog2e, a.y * kLog2e);
    A2[q][1] = make_float2(a.z * kLog2e, a.w * kLog2e);
    mu[q][0] = mu[q][1] = make_float2(0.f, 0.f);
  }
  ap = __all_sync(0xffffffffu, ap);
  // SP: in the preparation stage below a lane always handles channel pair (lane % 8) of its warp
  float bias0 = 0.f, bias1 = 0.f;
  if (SP && p.delta_bias != nullptr) {
    const int c = d_cta + warp * 16 + 2 * (lane & 7);
    if (c < D) {
      bias0 = p.delta_bias[c];
      bias1 = p.delta_bias[c + 1];
    }
  }

  auto compute_tile = [&](int i, auto ap_tag) {
    constexpr bool AP = decltype(ap_tag)::value;
    const int st = i % kNST, fb = i & 1;
#pragma unroll 1
    for (int half = kTT / kHalf - 1; half >= 0; --half) {
      // ds = dout * silu(z) of this warp's 16 channels for 16 steps: 4 pairs per lane
      __syncwarp();
#pragma unroll
      for (int k = 0; k < kHalf / 4; ++k) {
        const int tt = (lane >> 3) + 4 * k, sl = lane & 7;
        const uint32_t gw = sm.g[st][half * kHalf + tt][warp * 8 + sl];
        float v0 = bf16lo(gw), v1 = bf16hi(gw);
        if (has_z) {
          const uint32_t zw = sm.z[st][half * kHalf + tt][warp * 8 + sl];
          const float z0 = bf16lo(zw), z1 = bf16hi(zw);
          v0 *= z0 * sigmoid_fast(z0);
          v1 *= z1 * sigmoid_fast(z1);
        }
        *reinterpret_cast<float2*>(&sm.ds[warp][tt][2 * sl]) = make_float2(v0, v1);
        if (SP) {
          const uint32_t dw = sm.d[st][half * kHalf + tt][warp * 8 + sl];
          float s0 = bf16lo(dw) + bias0, s1 = bf16hi(dw) + bias1;
          if (p.softplus) {
            s0 = softplus_fast(s0);
            s1 = softplus_fast(s1);
          }
          // rows past the end of the segment must stay identity steps
          const bool live = t_begin + (ntiles - 1 - i) * kTT + half * kHalf + tt < t_end;
          *reinterpret_cast<float2*>(&sm.dt[warp][tt][2 * sl]) = live ? make_float2(s0, s1) : make_float2(0.f, 0.f);
        }
      }
      __syncwarp();
#pragma unroll
      for (int t = kHalf - 1; t >= 0; --t) {
        const int row = half * kHalf + t;
        const float2 dsv = *reinterpret_cast<const float2*>(&sm.ds[warp][t][2 * (lane >> 2)]);
        const float4 Cq = sm.fC[fb][row][j];
        float dt[2];
        if (SP) {
          const float2 f = *reinterpret_cast<const float2*>(&sm.dt[warp][t][2 * (lane >> 2)]);
          dt[0] = pq ? f.y : f.x;
          dt[1] = pq ? f.x : f.y;
        } else {
          const uint32_t dw = sm.d[st][row][slot];
          dt[0] = bf16sel(dw, selA);
          dt[1] = bf16sel(dw, selB);
        }
        const float dsq[2] = {pq ? dsv.y : dsv.x, pq ? dsv.x : dsv.y};
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float2 a01, a23;
          if (AP) {
            const float a0 = ex2_approx(dt[q] * A2[q][0].x);
            const float r = ex2_approx(dt[q] * (A2[q][0].y - A2[q][0].x));
            const float r2 = r * r;
            a01 = make_float2(a0, a0 * r);
            a23 = f2mul(a01, f2dup(r2));
          } else {
            const float2 e01 = f2mul(f2dup(dt[q]), A2[q][0]), e23 = f2mul(f2dup(dt[q]), A2[q][1]);
            a01 = make_float2(ex2_approx(e01.x), ex2_approx(e01.y));
            a23 = make_float2(ex2_approx(e23.x), ex2_approx(e23.y));
          }
          const float2 ds2 = f2dup(dsq[q]);
          mu[q][0] = f2mul(a01, f2fma(make_float2(Cq.x, Cq.y), ds2, mu[q][0]));
          mu[q][1] = f2mul(a23, f2fma(make_float2(Cq.z, Cq.w), ds2, mu[q][1]));
          dsum[q] += dt[q];
        }
      }
    }
  };

  for (int i = 0; i < ntiles; ++i) {
    block_barrier();
    if (ap) compute_tile(i, std::true_type{});
    else compute_tile(i, std::false_type{});
  }
  block_barrier();
  if (valid) {
    const size_t sg = (size_t)b * p.nseg + seg;
#pragma unroll
    for (int q = 0; q < 2; ++q)
      *reinterpret_cast<float4*>(p.seg_local + (sg * D + chan(q)) * 16 + 4 * j) =
          make_float4(mu[q][0].x, mu[q][0].y, mu[q][1].x, mu[q][1].y);
    if (j < 2) p.seg_dsum[sg * D + chan(0)] = dsum[0];
  }
}

bool bwd_local_fast_applicable(const ssm_problem_t& prob, const BwdParams& p) {
  auto al16 = [](const void* q) { return q == nullptr || (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
  if (p.static_C) return false;
  return prob.io_dtype == SSM_BF16 && prob.N == 16 && prob.D % 8 == 0 && al16(p.delta) && al16(p.z) && al16(p.dout) &&
         al16(p.C) && al16(p.A) && al16(p.seg_local);
}

cudaError_t launch_bwd_local_fast(const Plan& plan, const BwdParams& p, cudaStream_t s) {
  if (plan.nseg < 2) return cudaSuccess;
  dim3 grid((p.D + kCH - 1) / kCH, plan.nseg - 1, p.batch);
  if (p.softplus || p.delta_bias != nullptr) ssm_bwd_local_fast_kernel<true><<<grid, kThreads, 0, s>>>(p);
  else ssm_bwd_local_fast_kernel<false><<<grid, kThreads, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace ssm
