// First pass of the reverse time split, tuned path (bf16 io, N = 16, D % 8 == 0, 16-byte aligned pointers): for every
// time segment but the first, the adjoint that leaves the segment when nothing flows into it,
//     mu_t = a_t (C_t ds_t + mu_{t+1}),   mu_{end+1} = 0,   ds_t = dout_t * silu(z_t),   a_t = exp(delta_t A),
// evaluated from the last step of the segment to the first, and the segment's sum of delta (the adjoint of Eq. 2a and
// of the gate; the segment results are then combined by the reversed carry scan of ssm_carry.cu, Appendix D).
// Only this lambda / mu recurrence is needed here: no states, no x, no B.  Segment 0 has no earlier segment to hand its
// adjoint to and is not computed.
//
// Same construction as the tuned forward kernel (ssm_fwd_warp.cu) run backwards in time: one warp owns 32 adjacent
// channels of one segment, lane l holds all 16 states of channel l as packed float2 pairs (no exchanges between lanes),
// stages delta, z, dout and C with 16-byte cp.async copies into a three-stage ring of 32-step tiles private to the warp
// (walked from the last tile of the segment to the first), widens C to float once per tile and turns dout and z into ds
// once per element.  The (chain, tile) space is cut into equal ranges, one per resident warp (WarpSched in
// ssm_common.cuh); a chain that two warps share hands mu and the partial sum of delta over once, through L2, behind a
// bounded wait.
#include <type_traits>

#include "ssm_common.cuh"

namespace ssm {

int warp_workers(int chains, int sms, int per_sm, int max_workers);

namespace {

constexpr int kLT = 32;          // steps per tile
constexpr int kLStages = 3;      // ring stages
constexpr int kLWarps = 4;       // warps per block
constexpr int kLocalHandoffVec = 5;   // float4 per lane: 16 adjoint values, sum of delta

// SC: C is a per-channel parameter [D][16] (no C tile)
template <bool SP, bool SC>
struct LocalWarpSmem {
  uint32_t d[kLStages][kLT][16];   // bf16 pairs, 32 channels
  uint32_t z[kLStages][kLT][16];
  uint32_t g[kLStages][kLT][16];
  uint32_t rC[SC ? 1 : kLStages][SC ? 1 : kLT][12];  // bf16 pairs, 16 states; rows padded against bank conflicts of the widening pass
  float fC[SC ? 1 : kLT][20];               // C of the current tile widened to float (padded likewise)
  float dF[SP ? kLT : 1][32];      // SP: step sizes after bias and softplus
};

__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

}  // namespace

// SP: `delta` holds the pre-activation and the step size is delta + bias, through the softplus if asked (Algorithm 2 step 4)
// WHOLE: every tile and every channel group of the problem is whole, so the staging and the tile loop carry no range tests
template <bool SP, bool SC, bool WHOLE = false>
__global__ void __launch_bounds__(kLWarps * 32) ssm_bwd_local_warp_kernel(const BwdParams p, const WarpSched sc) {
  constexpr int H = 8;   // float2 pairs of states per thread
  using Smem = LocalWarpSmem<SP, SC>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  Smem& sm = reinterpret_cast<Smem*>(smem_raw)[warp];
  const int D = p.D;
  const int worker = blockIdx.x * kLWarps + warp;
  const bool has_z = p.z != nullptr;

  const __nv_bfloat16* __restrict__ gd = static_cast<const __nv_bfloat16*>(p.delta);
  const __nv_bfloat16* __restrict__ gz = static_cast<const __nv_bfloat16*>(p.z);
  const __nv_bfloat16* __restrict__ gg = static_cast<const __nv_bfloat16*>(p.dout);
  const __nv_bfloat16* __restrict__ gC = static_cast<const __nv_bfloat16*>(p.C);
  auto bf16_at = [&](const uint32_t* row, int c) {
    return __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(row)[c] << 16);
  };

  const int groups = (D + 31) / 32;
  const int nsegs = p.nseg - 1;   // segments 1 .. nseg - 1
  const WorkList wl = make_worklist(sc, worker);
  for (int pi = 0; pi < wl.count; ++pi) {
    int chain, from, to;
    get_piece(wl, sc.tiles, pi, chain, from, to);
    const int grp = chain % groups;
    const int bs = chain / groups;
    const int seg = 1 + bs % nsegs, b = bs / nsegs;
    const int d_w = grp * 32;
    const int t_seg0 = seg * p.seg_steps;
    const int t_seg_end = min(p.L, t_seg0 + p.seg_steps);
    const int live_tiles = (t_seg_end - t_seg0 + kLT - 1) / kLT;
    // positions [from, to) of the chain in processing order are tiles tile_hi down to tile_lo (time runs backwards)
    const int tile_lo = sc.tiles - to;
    int tile_hi = sc.tiles - 1 - from;
    if (tile_hi > live_tiles - 1) tile_hi = live_tiles - 1;
    const int ntiles = tile_hi >= tile_lo ? tile_hi - tile_lo + 1 : 0;
    const bool gives_out = to < sc.tiles;

    // ---- staging (this lane's chunks of a tile: rows lane / 4 + 8 k of delta, z, dout; rows lane / 2 + 16 k of C);
    // tile number i of the piece is tile tile_hi - i of the segment
    const int xrow = lane >> 2, xcc = lane & 3;
    const bool xcol_ok = d_w + xcc * 8 < D;
    const int brow = lane >> 1, bhc = lane & 1;
    auto issue_tile = [&](int i) {
      if (i < ntiles) {
        const int st = i % kLStages;
        const int t0 = t_seg0 + (tile_hi - i) * kLT;
        const size_t row0 = (size_t)b * p.L + t0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int tt = xrow + 8 * k;
          const bool ok = WHOLE || (xcol_ok && (t0 + tt < t_seg_end));
          const size_t go = ok ? (row0 + tt) * D + d_w + xcc * 8 : 0;
          cp_async16(&sm.d[st][tt][xcc * 4], gd + go, ok);
          cp_async16(&sm.z[st][tt][xcc * 4], (has_z ? gz : gd) + go, ok && has_z);
          cp_async16(&sm.g[st][tt][xcc * 4], gg + go, ok);
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int tt = brow + 16 * k;
          const bool ok = WHOLE || t0 + tt < t_seg_end;
          const size_t go = ok ? (row0 + tt) * 16 + bhc * 8 : 0;
          if constexpr (!SC) cp_async16(&sm.rC[st][tt][bhc * 4], gC + go, ok);
        }
      }
      cp_async_commit();
    };
    issue_tile(0);
    issue_tile(1);

    // ---- per-thread constants and the carried adjoint
    const int c_own = d_w + lane;
    const bool valid = c_own < D;
    float2 A2[H], mu[H];
    bool ap = !p.general_A;
    {
      float av[16];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid) a = *reinterpret_cast<const float4*>(p.A + (size_t)c_own * 16 + 4 * k);
        av[4 * k] = a.x; av[4 * k + 1] = a.y; av[4 * k + 2] = a.z; av[4 * k + 3] = a.w;
      }
      const float step = av[1] - av[0];
      const float tol = 1e-6f * fabsf(av[15]);
#pragma unroll
      for (int k = 2; k < 16; ++k) ap = ap && fabsf(av[k] - (av[0] + (float)k * step)) <= tol;
#pragma unroll
      for (int k = 0; k < H; ++k) A2[k] = make_float2(av[2 * k] * kLog2e, av[2 * k + 1] * kLog2e);
    }
    ap = __all_sync(0xffffffffu, ap);
    float2 Cst[SC ? H : 1];   // C as a parameter: this channel's row
    if constexpr (SC) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid) v = *reinterpret_cast<const float4*>(static_cast<const float*>(p.C) + (size_t)c_own * 16 + 4 * k);
        Cst[2 * k] = make_float2(v.x, v.y);
        Cst[2 * k + 1] = make_float2(v.z, v.w);
      }
    }
    const float a0s = A2[0].x, rs = A2[0].y - A2[0].x;
    const float bias_own = (SP && p.delta_bias != nullptr && valid) ? p.delta_bias[c_own] : 0.f;
    float dsum = 0.f;
    if (from > 0) {
      if (!wait_handoff(sc, worker, lane)) {
        cp_async_wait_all();
        return;
      }
      const float4* hb = sc.handoff + ((size_t)worker * 32 + lane) * kLocalHandoffVec;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float4 v = __ldcg(hb + k);
        mu[2 * k] = make_float2(v.x, v.y);
        mu[2 * k + 1] = make_float2(v.z, v.w);
      }
      dsum = __ldcg(hb + 4).x;
    } else {
#pragma unroll
      for (int k = 0; k < H; ++k) mu[k] = make_float2(0.f, 0.f);
    }

    // ---- 8 steps of the tile in stage st, rows r0 + 7 down to r0; the step sizes, gate terms and exponentials of all 8
    // steps first (independent work for a lone warp), then the recurrence
    const float gate_off = has_z ? 0.f : 1.f;
    auto eight_steps = [&](int st, int r0, auto ap_tag) {
      constexpr bool AP = decltype(ap_tag)::value;
      float dt[8], dsv[8], e0[AP ? 8 : 1], e1[AP ? 8 : 1];
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const int r = SSM_TILE_ROW(r0 + t, kLT, sc.abort);
        dt[t] = SP ? sm.dF[SP ? r : 0][lane] : bf16_at(sm.d[st][r], lane);
        // ds = dout * silu(z) with the hardware tanh; without z its tile is zero-filled (silu(0) = 0) and gate_off = 1
        // takes its place.  Rows past the end of the segment were zero-filled: dout = 0 gives ds = 0 and delta = 0
        // gives a = 1, so they leave the adjoint untouched.
        const float hz = 0.5f * bf16_at(sm.z[st][r], lane);
        dsv[t] = bf16_at(sm.g[st][r], lane) * (fmaf(hz, tanh_approx(hz), hz) + gate_off);
        if constexpr (AP) {
          e0[t] = ex2_approx(dt[t] * a0s);
          e1[t] = ex2_approx(dt[t] * rs);
        }
        dsum += dt[t];
      }
#pragma unroll
      for (int t = 7; t >= 0; --t) {
        const int r = SSM_TILE_ROW(r0 + t, kLT, sc.abort);
        float2 a[H];
        if constexpr (AP) {
          const float rr = e1[t], r2 = rr * rr, r4 = r2 * r2, r8 = r4 * r4;
          a[0] = make_float2(e0[t], e0[t] * rr);
          a[1] = f2mul(a[0], f2dup(r2));
          a[2] = f2mul(a[0], f2dup(r4));
          a[3] = f2mul(a[1], f2dup(r4));
#pragma unroll
          for (int k = 0; k < 4; ++k) a[4 + k] = f2mul(a[k], f2dup(r8));
        } else {
#pragma unroll
          for (int k = 0; k < H; ++k) {
            const float2 e = f2mul(f2dup(dt[t]), A2[k]);
            a[k] = make_float2(ex2_approx(e.x), ex2_approx(e.y));
          }
        }
        const float2 ds2 = f2dup(dsv[t]);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          float4 c;
          if constexpr (SC) c = make_float4(Cst[2 * k].x, Cst[2 * k].y, Cst[2 * k + 1].x, Cst[2 * k + 1].y);
          else c = *reinterpret_cast<const float4*>(&sm.fC[r][4 * k]);
          mu[2 * k] = f2mul(a[2 * k], f2fma(make_float2(c.x, c.y), ds2, mu[2 * k]));
          mu[2 * k + 1] = f2mul(a[2 * k + 1], f2fma(make_float2(c.z, c.w), ds2, mu[2 * k + 1]));
        }
      }
    };

    for (int i = 0; i < ntiles; ++i) {
      cp_async_wait_but_one();
      __syncwarp();             // tile i landed for all lanes; all lanes are done with tile i - 1
      issue_tile(i + 2);        // into the stage tile i - 1 used
      const int st = i % kLStages;
      const int t0 = t_seg0 + (tile_hi - i) * kLT;
      {
        if constexpr (!SC) {
          // C of the tile to float, one row per lane
          const uint4 c0 = *reinterpret_cast<const uint4*>(&sm.rC[st][lane][0]), c1 = *reinterpret_cast<const uint4*>(&sm.rC[st][lane][4]);
          const uint32_t wc[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
          for (int k = 0; k < 4; ++k)
            *reinterpret_cast<float4*>(&sm.fC[lane][4 * k]) =
                make_float4(bf16lo(wc[2 * k]), bf16hi(wc[2 * k]), bf16lo(wc[2 * k + 1]), bf16hi(wc[2 * k + 1]));
        }
        if constexpr (SP) {
          // step sizes of the tile, once per element; rows past the end of the segment stay identity steps
#pragma unroll 8
          for (int r = 0; r < kLT; ++r) {
            float v = bf16_at(sm.d[st][r], lane) + bias_own;
            if (p.softplus) v = softplus_fast(v);
            sm.dF[r][lane] = (WHOLE || t0 + r < t_seg_end) ? v : 0.f;
          }
        }
      }
      __syncwarp();
#pragma unroll 1
      for (int sb = kLT / 8 - 1; sb >= 0; --sb) {
        if (!WHOLE && t0 + sb * 8 >= t_seg_end) continue;   // identity steps
        if (ap) eight_steps(st, sb * 8, std::true_type{});
        else eight_steps(st, sb * 8, std::false_type{});
      }
    }
    cp_async_wait_all();
    __syncwarp();

    if (gives_out) {
      // the earlier part of this chain (in time) belongs to the next worker
      float4* hb = sc.handoff + ((size_t)(worker + 1) * 32 + lane) * kLocalHandoffVec;
#pragma unroll
      for (int k = 0; k < 4; ++k) __stcg(hb + k, make_float4(mu[2 * k].x, mu[2 * k].y, mu[2 * k + 1].x, mu[2 * k + 1].y));
      __stcg(hb + 4, make_float4(dsum, 0.f, 0.f, 0.f));
      publish_handoff(sc, worker, lane);
    } else if (valid) {
      const size_t sg = (size_t)b * p.nseg + seg;
      // (as inflow: what leaves segment 1 enters segment 0, and nothing enters segment 1)
      const size_t so = p.local_as_inflow ? sg - 1 : sg;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        *reinterpret_cast<float4*>(p.seg_local + (so * D + c_own) * 16 + 4 * k) =
            make_float4(mu[2 * k].x, mu[2 * k].y, mu[2 * k + 1].x, mu[2 * k + 1].y);
        if (p.local_as_inflow)
          *reinterpret_cast<float4*>(p.seg_local + (sg * D + c_own) * 16 + 4 * k) = make_float4(0.f, 0.f, 0.f, 0.f);
      }
      if (!p.local_as_inflow) p.seg_dsum[sg * D + c_own] = dsum;
    }
  }
}

bool bwd_local_fast_applicable(const ssm_problem_t& prob, const BwdParams& p) {
  auto al16 = [](const void* q) { return q == nullptr || (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
  return prob.io_dtype == SSM_BF16 && prob.N == 16 && prob.D % 8 == 0 && p.seg_steps % kLT == 0 && al16(p.delta) &&
         al16(p.z) && al16(p.dout) && al16(p.C) && al16(p.A) && al16(p.seg_local) && al16(p.handoff);
}

namespace {

template <bool SP, bool SC>
cudaError_t launch_local(const Plan& plan, const BwdParams& p, cudaStream_t s) {
  const size_t smem = sizeof(LocalWarpSmem<SP, SC>) * kLWarps;
  auto kern = ssm_bwd_local_warp_kernel<SP, SC>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 0, per_sm = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kLWarps * 32, smem)) != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  WarpSched sc{};
  sc.chains = p.batch * (plan.nseg - 1) * ((p.D + 31) / 32);
  sc.tiles = (plan.seg_steps + kLT - 1) / kLT;
  const bool can_share = p.abort != nullptr && p.flags != nullptr && p.handoff != nullptr && p.max_workers > 0;
  sc.workers = warp_workers(sc.chains, sms, per_sm * kLWarps, can_share ? p.max_workers : 0);
  const long long total = (long long)sc.chains * sc.tiles;
  sc.quota = (int)((total + sc.workers - 1) / sc.workers);
  sc.spin_limit = 1 << 22;
  sc.flags = p.flags + (p.max_workers + 1);   // second half of the flag array: the first belongs to the backward kernel
  sc.abort = p.abort;
  sc.handoff = p.handoff;                     // (the hand-off slots are shared: the two kernels run one after the other)
  const unsigned grid = (unsigned)((sc.workers + kLWarps - 1) / kLWarps);
  {
    // no ragged tile or channel group anywhere: the instantiation without range tests (same launch shape)
    if (p.L % kLT == 0 && plan.seg_steps % kLT == 0 && p.D % 32 == 0) {
      auto whole = ssm_bwd_local_warp_kernel<SP, SC, true>;
      if ((e = cudaFuncSetAttribute(whole, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
      whole<<<grid, kLWarps * 32, smem, s>>>(p, sc);
      return cudaGetLastError();
    }
  }
  kern<<<grid, kLWarps * 32, smem, s>>>(p, sc);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_bwd_local_fast(const Plan& plan, const BwdParams& p, cudaStream_t s) {
  if (plan.nseg < 2) return cudaSuccess;
  const bool sp = p.softplus || p.delta_bias != nullptr;
  if (p.static_C) return sp ? launch_local<true, true>(plan, p, s) : launch_local<false, true>(plan, p, s);
  return sp ? launch_local<true, false>(plan, p, s) : launch_local<false, false>(plan, p, s);
}

}  // namespace ssm
