// Forward selective scan, tuned path: bf16 io, N = 16, D % 8 == 0, 16-byte aligned pointers.
// Same mathematics and modes as ssm_fwd.cu (Algorithm 2 steps 5-6; Eq. 2a/2b; Eq. 4's A-bar; fused skip and gate).
//
// Mapping.  A compute thread owns 4 states of 2 adjacent channels (8 recurrences, held as packed float2 pairs so that
// the multiply-adds issue as two-wide FP32 instructions); the 4 lanes of a quad cover the 16 states of the channel
// pair; a warp covers 16 channels and sweeps time sequentially.  The sum over n of the readout is completed inside
// the quad by a batched two-step exchange, after which every lane holds the totals of two (step, channel) pairs.
//
// Warp roles.  A block has WARPS compute warps and one service warp.  The service warp issues the 16-byte cp.async
// copies of x, delta, z, B, C into a three-stage ring of [32 steps x channels] tiles, widens B and C to float, and
// finishes the previous tile: it adds the skip term to the readout totals the compute warps left in shared memory,
// applies the SiLU gate, rounds to bf16 and writes the output tile with 16-byte stores -- all while the compute warps
// run the recurrence of the current tile.  The two roles meet at one block-wide barrier per tile.
//
// Step size.  With a bias and/or the softplus of Algorithm 2 step 4 fused in (template flag SP), every compute warp
// turns the staged pre-activations of its own 16 channels into float step sizes, half a tile at a time and once per
// element, in a strip of shared memory of its own; its lanes then read those instead of unpacking bf16.
//
// Discretization.  a = 2^(delta * A * log2 e) with the hardware ex2.  When the four A values of a thread form an
// arithmetic progression (as in the S4D-Real initialisation A_n = -(n+1)) the four decays are built from two
// exponentials, a_k = a_0 r^k with r = 2^(delta * step * log2 e); the test is made per warp at run time and can
// be disabled by SSM_FLAG_GENERAL_A.
#include <type_traits>

#include "ssm_common.cuh"

namespace ssm {

namespace {

constexpr int kTT = 32;    // steps per tile
constexpr int kNST = 3;    // ring stages
constexpr int kHalf = 16;  // steps whose fused step sizes a compute warp prepares at a time

template <int WARPS, bool FULL, bool SP>
struct FastSmem {
  static constexpr int CH = 16 * WARPS;
  uint32_t x[kNST][kTT][CH / 2];
  uint32_t d[kNST][kTT][CH / 2];
  uint32_t z[FULL ? kNST : 1][FULL ? kTT : 1][CH / 2];
  uint32_t rawB[2][kTT][8];                        // widened one tile ahead: two stages
  uint32_t rawC[FULL ? 2 : 1][FULL ? kTT : 1][8];
  float4 fB[2][kTT][4];
  float4 fC[FULL ? 2 : 1][FULL ? kTT : 1][4];
  float dF[SP ? WARPS : 1][SP ? kHalf : 1][16];    // SP: step sizes after bias and softplus of half a tile, per warp
  float yp[FULL ? 2 : 1][FULL ? kTT : 1][CH];      // readout totals sum_n C h of a tile, per (step, channel)
  uint32_t o[FULL ? kTT : 1][CH / 2];              // output tile (bf16 pairs), owned by the service warp
  float Dsk[CH];                                   // D_skip of the block's channels
};

__device__ __forceinline__ void block_barrier(int nthreads) {
  asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}
__device__ __forceinline__ void cp_async_wait_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

}  // namespace

template <int WARPS, int MODE, bool SP, bool ZOH>
__global__ void __launch_bounds__((WARPS + 1) * 32) ssm_fwd_fast_kernel(const FwdParams p) {
  constexpr bool FULL = (MODE == kFwdFull);
  constexpr int THREADS = (WARPS + 1) * 32;
  constexpr int CH = 16 * WARPS;
  constexpr int CHUNKS = CH / 8;              // 16-byte chunks per tile row
  using Smem = FastSmem<WARPS, FULL, SP>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);

  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int d_cta = blockIdx.x * CH;
  const int seg = blockIdx.y;
  const int b = blockIdx.z;
  const int D = p.D;
  const int t_begin = seg * p.seg_steps;
  const int t_end = min(p.L, t_begin + p.seg_steps);
  const int ntiles = (t_end - t_begin + kTT - 1) / kTT;
  const bool has_z = FULL && p.z != nullptr;

  if (warp == WARPS) {
    // ================================================================== service warp
    const __nv_bfloat16* __restrict__ gx = static_cast<const __nv_bfloat16*>(p.x);
    const __nv_bfloat16* __restrict__ gd = static_cast<const __nv_bfloat16*>(p.delta);
    const __nv_bfloat16* __restrict__ gz = static_cast<const __nv_bfloat16*>(p.z);
    const __nv_bfloat16* __restrict__ gB = static_cast<const __nv_bfloat16*>(p.B);
    const __nv_bfloat16* __restrict__ gC = static_cast<const __nv_bfloat16*>(p.C);
    __nv_bfloat16* __restrict__ gout = static_cast<__nv_bfloat16*>(p.out);
    const size_t seg_row0 = (size_t)b * p.L + t_begin;

    auto issue_tile = [&](int i) {
      if (i < ntiles) {
        const int st = i % kNST;
        const int t0 = t_begin + i * kTT;
        const size_t row0 = seg_row0 + (size_t)i * kTT;
#pragma unroll
        for (int c = lane; c < kTT * CHUNKS; c += 32) {
          const int tt = c / CHUNKS, cc = c % CHUNKS;
          const bool ok = (d_cta + cc * 8 < D) && (t0 + tt < t_end);
          const size_t g = ok ? (row0 + tt) * D + d_cta + cc * 8 : 0;
          cp_async16(&sm.x[st][tt][cc * 4], gx + g, ok);
          cp_async16(&sm.d[st][tt][cc * 4], gd + g, ok);
          if (FULL) cp_async16(&sm.z[st][tt][cc * 4], (has_z ? gz : gx) + g, ok && has_z);
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int c = lane + 32 * k;
          const int tt = c >> 1, hc = c & 1;
          const bool ok = t0 + tt < t_end;
          const size_t g = ok ? (row0 + tt) * 16 + hc * 8 : 0;
          cp_async16(&sm.rawB[i & 1][tt][hc * 4], gB + g, ok);
          if (FULL) cp_async16(&sm.rawC[i & 1][tt][hc * 4], gC + g, ok);
        }
      }
      cp_async_commit();
    };
    auto widen_BC = [&](int i) {  // tile i: bf16 -> float
      if (i >= ntiles) return;
      const int fb = i & 1;
#pragma unroll
      for (int k = 0; k < kTT * 8 / 32; ++k) {
        const int c = lane + 32 * k;
        const int tt = c >> 3, w = c & 7;
        const uint32_t vb = sm.rawB[fb][tt][w];
        reinterpret_cast<float2*>(&sm.fB[fb][tt][0])[w] = make_float2(bf16lo(vb), bf16hi(vb));
        if (FULL) {
          const uint32_t vc = sm.rawC[fb][tt][w];
          reinterpret_cast<float2*>(&sm.fC[fb][tt][0])[w] = make_float2(bf16lo(vc), bf16hi(vc));
        }
      }
    };
    // skip term, gate and rounding of tile i (its readout totals are complete), then the 16-byte stores
    for (int c = lane; c < CH; c += 32)
      if (FULL) sm.Dsk[c] = (p.Dskip != nullptr && d_cta + c < D) ? p.Dskip[d_cta + c] : 0.f;
    __syncwarp();
    auto finish_tile = [&](int i) {
      if (!FULL) return;
      const int st = i % kNST, yb = i & 1;
#pragma unroll 4
      for (int c = lane; c < kTT * (CH / 2); c += 32) {
        const int tt = c / (CH / 2), eslot = c % (CH / 2);
        const float2 y = *reinterpret_cast<const float2*>(&sm.yp[yb][tt][2 * eslot]);
        const float2 Dk2 = *reinterpret_cast<const float2*>(&sm.Dsk[2 * eslot]);
        const uint32_t xw = sm.x[st][tt][eslot];
        float2 s2 = f2fma(Dk2, make_float2(bf16lo(xw), bf16hi(xw)), y);
        if (has_z) {
          const uint32_t zw = sm.z[st][tt][eslot];
          s2 = gate_pair_tanh(s2, make_float2(bf16lo(zw), bf16hi(zw)));
        }
        const __nv_bfloat162 r = __floats2bfloat162_rn(s2.x, s2.y);
        sm.o[tt][eslot] = *reinterpret_cast<const uint32_t*>(&r);
      }
      __syncwarp();
      const int t0 = t_begin + i * kTT;
      const size_t row0 = seg_row0 + (size_t)i * kTT;
#pragma unroll
      for (int c = lane; c < kTT * CHUNKS; c += 32) {
        const int tt = c / CHUNKS, cc = c % CHUNKS;
        if (d_cta + cc * 8 < D && t0 + tt < t_end)
          *reinterpret_cast<uint4*>(gout + (row0 + tt) * D + d_cta + cc * 8) =
              *reinterpret_cast<const uint4*>(&sm.o[tt][cc * 4]);
      }
      __syncwarp();
    };

    issue_tile(0);
    issue_tile(1);
    cp_async_wait_but_one();
    __syncwarp();
    widen_BC(0);
    for (int i = 0; i < ntiles; ++i) {
      block_barrier(THREADS);  // tile i is staged; the compute warps are done with tile i-1
      if (i >= 1) finish_tile(i - 1);  // reads x and z of the ring stage that tile i+2 is about to overwrite
      issue_tile(i + 2);
      cp_async_wait_but_one();
      __syncwarp();
      widen_BC(i + 1);
    }
    cp_async_wait_all();
    block_barrier(THREADS);
    finish_tile(ntiles - 1);
    return;
  }

  // ==================================================================== compute warps
  const int j = lane & 3;
  const int slot = warp * 8 + (lane >> 2);  // channel pair within the block
  const int d0 = d_cta + 2 * slot;  // first channel of this quad's pair (D is even, so both are valid or neither)
  const bool valid = d0 < D;
  const int pq = j & 1, gq = j >> 1;
  // A lane keeps the readout of channel pq of the pair and hands the other channel's partial sum to its neighbour,
  // so it numbers its own channels q = 0 (channel pq) and q = 1 (channel 1 - pq); the byte-permute selectors below
  // pick the matching half of a packed bf16 pair and widen it to float in one instruction.
  const uint32_t selA = pq ? 0x3244u : 0x1044u, selB = pq ? 0x1044u : 0x3244u;
  auto chan = [&](int q) { return d0 + (q ^ pq); };

  // ---- per-thread constants and state
  float2 A2[2][2];   // A * log2(e), states (4j, 4j+1) and (4j+2, 4j+3) of each channel
  float2 h[2][2];
  // ZOH: B-bar = E B with the input gain E = (a - 1) / A (Eq. 4), and E = delta where A = 0: 1 / A (0 where A = 0)
  // and the indicator of A = 0
  float2 invA[ZOH ? 2 : 1][2], zeroA[ZOH ? 2 : 1][2];
  float dsum[2] = {0.f, 0.f};
  bool ap = !p.general_A;
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), hs = a;
    if (valid) {
      a = *reinterpret_cast<const float4*>(p.A + (size_t)chan(q) * 16 + 4 * j);
      if (p.h_start != nullptr)
        hs = *reinterpret_cast<const float4*>(p.h_start + (((size_t)b * p.nseg + seg) * D + chan(q)) * 16 + 4 * j);
    }
    const float step = a.y - a.x;
    const float tol = 1e-6f * fabsf(a.w);
    ap = ap && fabsf(a.z - (a.x + 2.f * step)) <= tol && fabsf(a.w - (a.x + 3.f * step)) <= tol;
    A2[q][0] = make_float2(a.x * kLog2e, a.y * kLog2e);
    A2[q][1] = make_float2(a.z * kLog2e, a.w * kLog2e);
    h[q][0] = make_float2(hs.x, hs.y);
    h[q][1] = make_float2(hs.z, hs.w);
    if (ZOH) {
      auto inv = [](float v) { return v != 0.f ? 1.f / v : 0.f; };
      auto isz = [](float v) { return v != 0.f ? 0.f : 1.f; };
      invA[q][0] = make_float2(inv(a.x), inv(a.y));
      invA[q][1] = make_float2(inv(a.z), inv(a.w));
      zeroA[q][0] = make_float2(isz(a.x), isz(a.y));
      zeroA[q][1] = make_float2(isz(a.z), isz(a.w));
    }
  }
  ap = __all_sync(0xffffffffu, ap);
  // SP: in the step-size stage below a lane always handles channel pair (lane % 8) of its warp
  float bias0 = 0.f, bias1 = 0.f;
  if (SP && p.delta_bias != nullptr) {
    const int c = d_cta + warp * 16 + 2 * (lane & 7);
    if (c < D) {
      bias0 = p.delta_bias[c];
      bias1 = p.delta_bias[c + 1];
    }
  }


  // One tile of kTT steps, in sub-blocks of 4 steps: the loads of the next sub-block are issued before the
  // shared-memory stores of the current one, and the readout sums of 4 steps x 2 channels are exchanged inside the
  // quad in one batch, after which every lane leaves the totals of two (step, channel) pairs in shared memory for the service warp.  Rows past the end of the
  // segment were zero-filled: delta = 0 gives a = 1 and no input, so they leave the state untouched.
  auto compute_tile = [&](int i, auto ap_tag) {
    constexpr bool AP = decltype(ap_tag)::value;
    constexpr int SB = 4;  // the quad exchange below is written for exactly 4 steps
    const int st = i % kNST, fb = i & 1;
    float a0s[2], rs[2];  // AP path: A2 of the first state and of the step
    if (AP) {
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        a0s[q] = A2[q][0].x;
        rs[q] = A2[q][0].y - A2[q][0].x;
      }
    }
    uint32_t dw[SB], xw[SB];
    float2 dfv[SB];   // SP: the step sizes of the channel pair, float
    float4 Bq[SB], Cq[SB];
    // SP: step sizes of steps [half * kHalf, +kHalf) of this warp's 16 channels: bf16 pre-activation + bias, softplus,
    // float, into the warp's own strip (4 pairs per lane); rows past the end of the segment stay identity steps
    auto prepare_dt = [&](int half) {
      __syncwarp();
#pragma unroll
      for (int k = 0; k < kHalf / 4; ++k) {
        const int tt = (lane >> 3) + 4 * k, sl = lane & 7;
        const uint32_t w = sm.d[st][half * kHalf + tt][warp * 8 + sl];
        float v0 = bf16lo(w) + bias0, v1 = bf16hi(w) + bias1;
        if (p.softplus) {
          v0 = softplus_fast(v0);
          v1 = softplus_fast(v1);
        }
        const bool live = t_begin + i * kTT + half * kHalf + tt < t_end;
        *reinterpret_cast<float2*>(&sm.dF[warp][tt][2 * sl]) = live ? make_float2(v0, v1) : make_float2(0.f, 0.f);
      }
      __syncwarp();
    };
    auto load_sb = [&](int tb) {
      if (SP && tb % kHalf == 0) prepare_dt(tb / kHalf);
#pragma unroll
      for (int t = 0; t < SB; ++t) {
        if (SP) dfv[t] = *reinterpret_cast<const float2*>(&sm.dF[warp][(tb + t) % kHalf][2 * (lane >> 2)]);
        else dw[t] = sm.d[st][tb + t][slot];
        xw[t] = sm.x[st][tb + t][slot];
        Bq[t] = sm.fB[fb][tb + t][j];
        if (FULL) Cq[t] = sm.fC[fb][tb + t][j];
      }
    };
    load_sb(0);
#pragma unroll
    for (int tb = 0; tb < kTT; tb += SB) {
      // pass 1: discretization of the whole sub-block (independent work: decays a and inputs bx for 4 steps)
      float2 a01[SB][2], a23[SB][2], bx01[SB][2], bx23[SB][2];
#pragma unroll
      for (int t = 0; t < SB; ++t) {
        // q = 0 is this lane's kept channel (channel pq of the pair), q = 1 the one it hands to its neighbour
        const float dt[2] = {SP ? (pq ? dfv[t].y : dfv[t].x) : __uint_as_float(__byte_perm(dw[t], 0, selA)),
                             SP ? (pq ? dfv[t].x : dfv[t].y) : __uint_as_float(__byte_perm(dw[t], 0, selB))};
        const float u[2] = {__uint_as_float(__byte_perm(xw[t], 0, selA)), __uint_as_float(__byte_perm(xw[t], 0, selB))};
        const float2 du = f2mul(make_float2(dt[0], dt[1]), make_float2(u[0], u[1]));
        const float duq[2] = {du.x, du.y};
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          if (AP) {
            const float a0 = ex2_approx(dt[q] * a0s[q]);
            const float r = ex2_approx(dt[q] * rs[q]);
            const float r2 = r * r;
            a01[t][q] = make_float2(a0, a0 * r);
            a23[t][q] = f2mul(a01[t][q], make_float2(r2, r2));
          } else {
            const float2 dd = make_float2(dt[q], dt[q]);
            const float2 e01 = f2mul(dd, A2[q][0]), e23 = f2mul(dd, A2[q][1]);
            a01[t][q] = make_float2(ex2_approx(e01.x), ex2_approx(e01.y));
            a23[t][q] = make_float2(ex2_approx(e23.x), ex2_approx(e23.y));
          }
          if (ZOH) {
            const float2 dd = f2dup(dt[q]), uu = f2dup(u[q]), m1 = f2dup(-1.f), one = f2dup(1.f);
            const float2 E01 = f2fma(f2fma(a01[t][q], one, m1), invA[q][0], f2mul(zeroA[q][0], dd));
            const float2 E23 = f2fma(f2fma(a23[t][q], one, m1), invA[q][1], f2mul(zeroA[q][1], dd));
            bx01[t][q] = f2mul(f2mul(E01, uu), make_float2(Bq[t].x, Bq[t].y));
            bx23[t][q] = f2mul(f2mul(E23, uu), make_float2(Bq[t].z, Bq[t].w));
          } else {
            const float2 dq = make_float2(duq[q], duq[q]);
            bx01[t][q] = f2mul(dq, make_float2(Bq[t].x, Bq[t].y));
            bx23[t][q] = f2mul(dq, make_float2(Bq[t].z, Bq[t].w));
          }
          if (MODE == kFwdSummary) dsum[q] += dt[q];
        }
      }
      // pass 2: the recurrence (4 independent packed chains) and the readout
      float y[SB][2];
#pragma unroll
      for (int t = 0; t < SB; ++t) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          h[q][0] = f2fma(a01[t][q], h[q][0], bx01[t][q]);
          h[q][1] = f2fma(a23[t][q], h[q][1], bx23[t][q]);
          if (FULL) {
            float2 yv = f2mul(make_float2(Cq[t].x, Cq[t].y), h[q][0]);
            yv = f2fma(make_float2(Cq[t].z, Cq[t].w), h[q][1], yv);
            y[t][q] = yv.x + yv.y;
          }
        }
      }
      if (tb + SB < kTT) load_sb(tb + SB);
      if (FULL) {
        float w[SB];
#pragma unroll
        for (int t = 0; t < SB; ++t) w[t] = y[t][0] + __shfl_xor_sync(0xffffffffu, y[t][1], 1);
        // lanes j and j^2 hold the same channel: the lower one finishes steps 0,1 of the sub-block, the upper 2,3
        float tot[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float keep = gq ? w[2 + e] : w[e], send = gq ? w[e] : w[2 + e];
          tot[e] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
        }
        sm.yp[fb][tb + 2 * gq][2 * slot + pq] = tot[0];
        sm.yp[fb][tb + 2 * gq + 1][2 * slot + pq] = tot[1];
      }
    }
  };

  for (int i = 0; i < ntiles; ++i) {
    block_barrier(THREADS);
    const int t0 = t_begin + i * kTT;
    if (MODE != kFwdSummary && p.ckpt != nullptr && (t0 % kCkptSteps) == 0 && valid) {
#pragma unroll
      for (int q = 0; q < 2; ++q)
        *reinterpret_cast<float4*>(p.ckpt + (((size_t)b * p.nck + t0 / kCkptSteps) * D + chan(q)) * 16 + 4 * j) =
            make_float4(h[q][0].x, h[q][0].y, h[q][1].x, h[q][1].y);
    }
    if (ap) compute_tile(i, std::true_type{});
    else compute_tile(i, std::false_type{});
  }
  block_barrier(THREADS);
  if (MODE == kFwdFull && p.h_last != nullptr && seg == p.nseg - 1 && valid) {
#pragma unroll
    for (int q = 0; q < 2; ++q)
      *reinterpret_cast<float4*>(p.h_last + ((size_t)b * D + chan(q)) * 16 + 4 * j) =
          make_float4(h[q][0].x, h[q][0].y, h[q][1].x, h[q][1].y);
  }
  if (MODE == kFwdSummary && valid) {
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      *reinterpret_cast<float4*>(p.seg_end + (((size_t)b * p.nseg + seg) * D + chan(q)) * 16 + 4 * j) =
          make_float4(h[q][0].x, h[q][0].y, h[q][1].x, h[q][1].y);
      if (j < 2 && q == 0) p.seg_dsum[((size_t)b * p.nseg + seg) * D + chan(0)] = dsum[0];
    }
  }
}

template <int WARPS, int MODE, bool SP, bool ZOH>
static cudaError_t launch_fast_variant(const Plan& plan, const FwdParams& p, cudaStream_t s) {
  constexpr size_t smem = sizeof(FastSmem<WARPS, MODE == kFwdFull, SP>);
  constexpr int CH = 16 * WARPS;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(ssm_fwd_fast_kernel<WARPS, MODE, SP, ZOH>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  dim3 grid((p.D + CH - 1) / CH, plan.nseg, p.batch);
  ssm_fwd_fast_kernel<WARPS, MODE, SP, ZOH><<<grid, (WARPS + 1) * 32, smem, s>>>(p);
  return cudaGetLastError();
}

// ZOH: the zero-order-hold B-bar of Eq. 4 instead of delta * B
template <int WARPS, int MODE, bool SP>
static cudaError_t launch_fast_sp(const Plan& plan, const FwdParams& p, cudaStream_t s) {
  if (p.zoh) return launch_fast_variant<WARPS, MODE, SP, true>(plan, p, s);
  return launch_fast_variant<WARPS, MODE, SP, false>(plan, p, s);
}

// SP: the step size goes through the bias / softplus stage of the service warp
template <int WARPS, int MODE>
static cudaError_t launch_fast(const Plan& plan, const FwdParams& p, cudaStream_t s) {
  if (p.softplus || p.delta_bias != nullptr) return launch_fast_sp<WARPS, MODE, true>(plan, p, s);
  return launch_fast_sp<WARPS, MODE, false>(plan, p, s);
}

bool fwd_fast_applicable(const ssm_problem_t& prob, const FwdParams& p) {
  auto al16 = [](const void* q) { return q == nullptr || (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
  if (p.static_B || p.static_C) return false;  // input-dependent B, C only
  return prob.io_dtype == SSM_BF16 && prob.N == 16 && prob.D % 8 == 0 && al16(p.x) && al16(p.delta) && al16(p.z) &&
         al16(p.B) && al16(p.C) && al16(p.out) && al16(p.A) && al16(p.h_start) && al16(p.ckpt) && al16(p.seg_end) && al16(p.h_last);
}

// Two compute warps (32 channels) per block measured best on all three layer shapes (1, 3 and 4 were 3-35 % slower).
constexpr int kFwdFastWarps = 2;

cudaError_t launch_fwd_fast(const Plan& plan, const FwdParams& p, int mode, cudaStream_t s) {
  switch (mode) {
    case kFwdFull: return launch_fast<kFwdFastWarps, kFwdFull>(plan, p, s);
    case kFwdSummary: return launch_fast<kFwdFastWarps, kFwdSummary>(plan, p, s);
    default: return launch_fast<kFwdFastWarps, kFwdCkptOnly>(plan, p, s);
  }
}

}  // namespace ssm
