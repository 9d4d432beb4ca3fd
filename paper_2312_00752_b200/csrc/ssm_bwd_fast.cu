// Backward selective scan, tuned path: bf16 io, N = 16, D % 8 == 0, 16-byte aligned pointers.
// Same mathematics as ssm_bwd.cu (adjoint of Eq. 2a/2b with skip term and gate; states recomputed, Section 3.3).
//
// Mapping (as in the tuned forward kernel).  A thread owns 4 states of 2 adjacent channels as packed float2 pairs;
// the 4 lanes of a quad cover the 16 states of the channel pair; a warp covers 16 channels, a block 32.
//
// Recomputation in two levels.  The block walks its segment backwards in tiles of 32 steps (one checkpoint block).
// For a tile it first re-runs the recurrence from the checkpoint state over steps 0..23, parking the states at steps
// 8, 16 and 24 in shared memory; then, for the sub-blocks of 8 steps from last to first, it re-runs the 8 steps keeping
// every h_t in registers and walks them backwards with the adjoint recurrence.
//
// Registers are the scarce resource (255 per thread, 4 blocks per SM, and almost no L1 left beside 54 KB of shared
// memory per block, so a spill costs an L2 round trip): whatever can wait in shared memory does -- the input words of a
// step are read again in the reverse pass, the checkpoint state waits in a staging buffer that is dead by then, and
// the readout is finished before the reverse pass starts.
//
// Scheduling.  The kernel is persistent: blocks claim work items (channel group, tile) from a global counter in an
// order in which the tile that a tile depends on (the next tile in time of the same channel group) is always claimed
// earlier, so whoever holds it is already running; the adjoint mu and the dA / dD accumulators cross from one tile
// to the next through a small hand-off buffer in L2 and a release/acquire flag per channel group.  This keeps every
// SM busy to the end whatever the ratio of blocks to SMs is.  Every wait is bounded: after a fixed number of polls a
// block raises an abort word that all blocks observe, and the host reports SSM_ERR_TIMEOUT.
//
// Sums.  The three per-(step, channel) sums over n (readout for dz, sum lam*B for dx and ddelta, sum w*A for
// ddelta) are exchanged inside the quad in batches per sub-block, after which every lane finalises 4 steps of one
// channel (the readout and dz before the reverse pass, dx and ddelta after it).  dB and dC are summed over the two
// channels of a thread in registers, over the 8 quads of a warp through
// a shared-memory transpose with a fixed order, over the 2 warps in ascending order, and leave the block as partial
// sums that ssm_bwd_reduce_kernel adds in ascending block order.  dA and dD accumulate in registers over the whole
// segment.  Everything is deterministic; there are no floating-point atomics.
#include <type_traits>

#include "ssm_common.cuh"

namespace ssm {

namespace {

constexpr int kBT = 32;   // steps per tile = checkpoint spacing
constexpr int kSB = 8;    // steps per register-resident sub-block
constexpr int kRB = 4;    // steps between two dB/dC transposes
static_assert(kBT == kCkptSteps, "the tuned backward kernel restarts from one checkpoint per tile");
constexpr int kBwdFastWarps = 2;
constexpr int kBwdFastThreads = kBwdFastWarps * 32;
constexpr int kBwdFastCH = 16 * kBwdFastWarps;
constexpr float kInvLog2e = 0.6931471805599453f;
constexpr int kHandoffVec = 5;            // float4 per thread: mu (2), dA (2), dD (1)
constexpr int kSpinLimit = 1 << 22;       // polls of a dependency flag before giving up (each poll sleeps ~100 ns)

struct BwdFastSmem {
  uint32_t x[2][kBT][kBwdFastCH / 2];   // bf16 pairs; the rows of a finished sub-block are reused for dx
  uint32_t d[2][kBT][kBwdFastCH / 2];   // ... for ddelta
  uint32_t z[2][kBT][kBwdFastCH / 2];   // ... for dz
  uint32_t g[2][kBT][kBwdFastCH / 2];
  uint32_t rawB[2][kBT][8];
  uint32_t rawC[2][kBT][8];
  float4 fB[kBT][4];
  float4 fC[kBT][4];
  float ds[kBT][kBwdFastCH];            // dout * silu(z)
  float gsp[kBT][kBwdFastCH];           // dout * silu'(z); with the fused step size: the step size itself, float
  float4 red[kBwdFastWarps][kRB][8][4][2];   // [warp][step][quad][lane in quad][dB quad | dC quad]
  float acc[kBwdFastWarps][kBT][32];    // per-warp sums over its 16 channels: [step][dB 0..15 | dC 0..15]
  int sched[4];                         // [0] current item, [1] next item, [2] abort
  float4 hsave[kBT / kSB - 1][2][kBwdFastThreads];  // states at steps 8, 16, 24 of the tile, per thread and channel
};


__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

}  // namespace

// ZOH: B-bar = E B with E = (a - 1) / A (Eq. 4; E = delta where A = 0) instead of delta * B
template <bool SP, bool ZOH>
__global__ void __launch_bounds__(kBwdFastThreads) ssm_bwd_fast_kernel(const BwdParams p) {
  constexpr int THREADS = kBwdFastThreads;
  constexpr int CH = kBwdFastCH;
  constexpr int CHUNKS = CH / 8;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  BwdFastSmem& sm = *reinterpret_cast<BwdFastSmem*>(smem_raw);

  const __nv_bfloat16* __restrict__ gx = static_cast<const __nv_bfloat16*>(p.x);
  const __nv_bfloat16* __restrict__ gd = static_cast<const __nv_bfloat16*>(p.delta);
  const __nv_bfloat16* __restrict__ gz = static_cast<const __nv_bfloat16*>(p.z);
  const __nv_bfloat16* __restrict__ gg = static_cast<const __nv_bfloat16*>(p.dout);
  const __nv_bfloat16* __restrict__ gB = static_cast<const __nv_bfloat16*>(p.B);
  const __nv_bfloat16* __restrict__ gC = static_cast<const __nv_bfloat16*>(p.C);
  __nv_bfloat16* __restrict__ gdx = static_cast<__nv_bfloat16*>(p.dx);
  __nv_bfloat16* __restrict__ gdd = static_cast<__nv_bfloat16*>(p.ddelta);
  __nv_bfloat16* __restrict__ gdz = static_cast<__nv_bfloat16*>(p.dz);

  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  const int j = lane & 3, quad = lane >> 2;
  const int slot = warp * 8 + quad;      // channel pair within the block
  const int D = p.D;
  const bool has_z = gz != nullptr;
  // q = 0 is the channel whose sums this lane keeps (channel pq of the pair), q = 1 the one it hands to its neighbour
  const int pq = j & 1, gq = j >> 1;
  const uint32_t selA = pq ? 0x3244u : 0x1044u, selB = pq ? 0x1044u : 0x3244u;

  // ---- work items: chain = (batch, segment, channel group); item = (order within the chain, chain), order-major
  const int groups = (D + CH - 1) / CH;
  const int chains = p.batch * p.nseg * groups;
  const int tiles_max = p.seg_steps / kBT;
  const int total_items = chains * tiles_max;
  int* const sched_counter = p.sched;
  int* const sched_abort = p.sched + 1;
  int* const sched_flags = p.sched + 64;

  struct Item {
    int chain, ord, b, seg, grp, d_cta, t_begin, t_end, ntiles, tile, t0;
    bool live;   // false: the chain has fewer tiles than tiles_max and this order does not exist
  };
  auto decode = [&](int id) {
    Item it;
    it.ord = id / chains;
    it.chain = id - it.ord * chains;
    it.grp = it.chain % groups;
    const int bs = it.chain / groups;
    it.seg = bs % p.nseg;
    it.b = bs / p.nseg;
    it.d_cta = it.grp * CH;
    it.t_begin = it.seg * p.seg_steps;
    it.t_end = min(p.L, it.t_begin + p.seg_steps);
    it.ntiles = (it.t_end - it.t_begin + kBT - 1) / kBT;
    it.live = id < total_items && it.ord < it.ntiles;
    it.tile = it.ntiles - 1 - it.ord;               // tiles run from last to first
    it.t0 = it.t_begin + it.tile * kBT;
    return it;
  };
  auto issue_item = [&](const Item& it, int st) {   // inputs of one tile into ring stage st
    if (it.live) {
      const size_t row0 = (size_t)it.b * p.L + it.t0;
      for (int c = tid; c < kBT * CHUNKS; c += THREADS) {
        const int tt = c / CHUNKS, cc = c % CHUNKS;
        const bool ok = (it.t0 + tt < it.t_end) && (it.d_cta + cc * 8 < D);
        const size_t g = ok ? (row0 + tt) * D + it.d_cta + cc * 8 : 0;
        cp_async16(&sm.x[st][tt][cc * 4], gx + g, ok);
        cp_async16(&sm.d[st][tt][cc * 4], gd + g, ok);
        cp_async16(&sm.z[st][tt][cc * 4], (has_z ? gz : gx) + g, ok && has_z);
        cp_async16(&sm.g[st][tt][cc * 4], gg + g, ok);
      }
      for (int c = tid; c < kBT * 2; c += THREADS) {
        const int tt = c >> 1, cc = c & 1;
        const bool ok = it.t0 + tt < it.t_end;
        const size_t g = ok ? (row0 + tt) * 16 + cc * 8 : 0;
        cp_async16(&sm.rawB[st][tt][cc * 4], gB + g, ok);
        cp_async16(&sm.rawC[st][tt][cc * 4], gC + g, ok);
      }
    }
    cp_async_commit();
  };

  // ---- state of the chain being processed (set per item)
  float2 A2[2][2], mu[2][2], dA2[2][2];
  float2 invA[ZOH ? 2 : 1][2];   // ZOH: 1 / A (0 where A = 0)
  bool zeroA = false;            // ZOH: some A of this warp is exactly 0 (then the slower exact form of E is used)
  float Dk = 0.f, dD_acc = 0.f;
  float bias_pq = 0.f, dbias_acc = 0.f;   // SP: bias of the kept channel, sum of the pre-activation gradient
  int d0 = 0;
  bool valid = false;
  auto chan = [&](int q) { return d0 + (q ^ pq); };

  // decays of one step for channel q: general A or arithmetic-progression A (two exponentials)
  auto decays = [&](float dt, int q, auto ap_tag, float2& a01, float2& a23) {
    if (decltype(ap_tag)::value) {
      const float a0 = ex2_approx(dt * A2[q][0].x);
      const float r = ex2_approx(dt * (A2[q][0].y - A2[q][0].x));
      const float r2 = r * r;
      a01 = make_float2(a0, a0 * r);
      a23 = f2mul(a01, f2dup(r2));
    } else {
      const float2 e01 = f2mul(f2dup(dt), A2[q][0]), e23 = f2mul(f2dup(dt), A2[q][1]);
      a01 = make_float2(ex2_approx(e01.x), ex2_approx(e01.y));
      a23 = make_float2(ex2_approx(e23.x), ex2_approx(e23.y));
    }
  };

  // ZOH input gain of channel q: E = (a - 1) / A, and E = dt where A = 0
  auto gain = [&](float dt, int q, float2 a01, float2 a23, float2& E01, float2& E23) {
    E01 = f2mul(f2fma(a01, f2dup(1.f), f2dup(-1.f)), invA[ZOH ? q : 0][0]);
    E23 = f2mul(f2fma(a23, f2dup(1.f), f2dup(-1.f)), invA[ZOH ? q : 0][1]);
    if (zeroA) {
      if (A2[q][0].x == 0.f) E01.x = dt;
      if (A2[q][0].y == 0.f) E01.y = dt;
      if (A2[q][1].x == 0.f) E23.x = dt;
      if (A2[q][1].y == 0.f) E23.y = dt;
    }
  };
  // dE/dA = (dt a - E) / A, and dt^2 / 2 where A = 0
  auto gain_dA = [&](float dt, int q, float2 a01, float2 a23, float2 E01, float2 E23, float2& G01, float2& G23) {
    const float2 dd = f2dup(dt);
    G01 = f2mul(f2fma(dd, a01, f2mul(E01, f2dup(-1.f))), invA[ZOH ? q : 0][0]);
    G23 = f2mul(f2fma(dd, a23, f2mul(E23, f2dup(-1.f))), invA[ZOH ? q : 0][1]);
    if (zeroA) {
      const float hv = 0.5f * dt * dt;
      if (A2[q][0].x == 0.f) G01.x = hv;
      if (A2[q][0].y == 0.f) G01.y = hv;
      if (A2[q][1].x == 0.f) G23.x = hv;
      if (A2[q][1].y == 0.f) G23.y = hv;
    }
  };
  // input term of the recurrence for channel q: bx = delta x B, or E x B under ZOH
  auto input_term = [&](float dt, float xu, float dxu, int q, float2 a01, float2 a23, float4 Bq, float2& b01, float2& b23) {
    if (ZOH) {
      float2 E01, E23;
      gain(dt, q, a01, a23, E01, E23);
      b01 = f2mul(f2mul(E01, f2dup(xu)), make_float2(Bq.x, Bq.y));
      b23 = f2mul(f2mul(E23, f2dup(xu)), make_float2(Bq.z, Bq.w));
    } else {
      b01 = f2mul(f2dup(dxu), make_float2(Bq.x, Bq.y));
      b23 = f2mul(f2dup(dxu), make_float2(Bq.z, Bq.w));
    }
  };

  // step sizes of the lane's channel pair at tile row tt as (kept channel, handed channel)
  auto step_sizes = [&](int st, int tt, uint32_t dw) {
    if (SP) {
      const float2 f = *reinterpret_cast<const float2*>(&sm.gsp[tt][2 * slot]);
      return pq ? make_float2(f.y, f.x) : f;
    }
    (void)st;
    return make_float2(bf16sel(dw, selA), bf16sel(dw, selB));
  };

  // nlive: rows of the tile inside the segment (the rest were zero-filled and are identity steps)
  auto process_tile = [&](int st, auto ap_tag, const float4 (&ck)[2], int nlive) {
    // The raw B / C rows of this ring stage were widened by the staging pass and are dead until the stage is refilled
    // two tiles from now: the checkpoint state waits there (one float4 per thread and channel) until the first
    // sub-block needs it again, instead of in registers.
    float4* const park[2] = {reinterpret_cast<float4*>(&sm.rawB[st][0][0]), reinterpret_cast<float4*>(&sm.rawC[st][0][0])};
    static_assert(sizeof(sm.rawB[0]) == sizeof(float4) * kBwdFastThreads, "one float4 per thread fits a raw B stage");
    // start state of sub-block sb, from where level 1 (or the checkpoint) left it
    auto start_state = [&](int sb, int q) { return sb > 0 ? sm.hsave[sb - 1][q][tid] : park[q][tid]; };
    // ---- level 1: states at the sub-block boundaries (steps 0, 8, 16, 24 of the tile), parked in shared memory
    {
      float2 h[2][2];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        park[q][tid] = ck[q];
        h[q][0] = make_float2(ck[q].x, ck[q].y);
        h[q][1] = make_float2(ck[q].z, ck[q].w);
      }
#pragma unroll 1
    for (int sb = 0; sb < kBT / kSB - 1; ++sb) {
#pragma unroll
      for (int t = 0; t < kSB; ++t) {
        const int tt = sb * kSB + t;
        const uint32_t dw = SP ? 0u : sm.d[st][tt][slot], xw = sm.x[st][tt][slot];
        const float4 Bq = sm.fB[tt][j];
        const float2 dt2 = step_sizes(st, tt, dw);
        const float2 u2 = make_float2(bf16sel(xw, selA), bf16sel(xw, selB));
        const float2 du = f2mul(dt2, u2);
        const float dtq[2] = {dt2.x, dt2.y}, uq[2] = {u2.x, u2.y}, duq[2] = {du.x, du.y};
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float2 a01, a23, b01, b23;
          decays(dtq[q], q, ap_tag, a01, a23);
          input_term(dtq[q], uq[q], duq[q], q, a01, a23, Bq, b01, b23);
          h[q][0] = f2fma(a01, h[q][0], b01);
          h[q][1] = f2fma(a23, h[q][1], b23);
        }
      }
#pragma unroll
      for (int q = 0; q < 2; ++q) sm.hsave[sb][q][tid] = make_float4(h[q][0].x, h[q][0].y, h[q][1].x, h[q][1].y);
    }
    }
    // ---- level 2: sub-blocks from last to first
#pragma unroll 1
    for (int sb = kBT / kSB - 1; sb >= 0; --sb) {
      float2 hist[kSB][2][2];
      // (the x and step-size words are re-read from shared memory in the reverse pass: registers are the scarce resource)
      float yw[kSB], dxw[kSB], ddw[kSB];  // quad-pair sums of: readout, delta * sum lam B, sum w A + x sum lam B
      {
        float2 h[2][2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const float4 v = start_state(sb, q);
          h[q][0] = make_float2(v.x, v.y);
          h[q][1] = make_float2(v.z, v.w);
        }
#pragma unroll
        for (int t = 0; t < kSB; ++t) {
          const int tt = sb * kSB + t;
          const uint32_t xw = sm.x[st][tt][slot];
          const float4 Bq = sm.fB[tt][j], Cq = sm.fC[tt][j];
          const float2 dt2 = step_sizes(st, tt, SP ? 0u : sm.d[st][tt][slot]);
          const float2 u2 = make_float2(bf16sel(xw, selA), bf16sel(xw, selB));
          const float2 du = f2mul(dt2, u2);
          const float dtq[2] = {dt2.x, dt2.y}, uq[2] = {u2.x, u2.y}, duq[2] = {du.x, du.y};
          float y[2];
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            float2 a01, a23, b01, b23;
            decays(dtq[q], q, ap_tag, a01, a23);
            input_term(dtq[q], uq[q], duq[q], q, a01, a23, Bq, b01, b23);
            h[q][0] = f2fma(a01, h[q][0], b01);
            h[q][1] = f2fma(a23, h[q][1], b23);
            hist[t][q][0] = h[q][0];
            hist[t][q][1] = h[q][1];
            float2 yv = f2mul(make_float2(Cq.x, Cq.y), h[q][0]);
            yv = f2fma(make_float2(Cq.z, Cq.w), h[q][1], yv);
            y[q] = yv.x + yv.y;
          }
          yw[t] = y[0] + __shfl_xor_sync(0xffffffffu, y[1], 1);
        }
      }
      // The readout totals are complete: finish them now (second exchange: lanes j and j^2 hold sums of the same
      // channel, the lower keeps steps 0..3, the upper 4..7) and write dz, so that they do not occupy registers
      // during the reverse recurrence.  The z rows of the tile were consumed by the staging pass.
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float ky = gq ? yw[4 + e] : yw[e], sy = gq ? yw[e] : yw[4 + e];
        const float ytot = ky + __shfl_xor_sync(0xffffffffu, sy, 2);
        const int tt = sb * kSB + 4 * gq + e;
        const float u = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(&sm.x[st][tt][slot])[pq] << 16);
        const float s = fmaf(Dk, u, ytot);
        float gsp;
        if (SP) {
          // the gate derivative is rebuilt here (its array holds the step sizes)
          const float gf = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(&sm.g[st][tt][slot])[pq] << 16);
          const float zf = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(&sm.z[st][tt][slot])[pq] << 16);
          const float sg = sigmoid_fast(zf);
          gsp = has_z ? gf * sg * fmaf(zf, 1.f - sg, 1.f) : 0.f;
        } else {
          gsp = sm.gsp[tt][2 * slot + pq];
        }
        reinterpret_cast<__nv_bfloat16*>(&sm.z[st][tt][slot])[pq] = __float2bfloat16_rn(gsp * s);
      }
      // reverse recurrence over the sub-block
#pragma unroll
      for (int t = kSB - 1; t >= 0; --t) {
        const int tt = sb * kSB + t;
        const float4 Bq = sm.fB[tt][j], Cq = sm.fC[tt][j];
        const float2 dt2 = step_sizes(st, tt, SP ? 0u : sm.d[st][tt][slot]);
        const uint32_t xw = sm.x[st][tt][slot];
        const float2 u2 = make_float2(bf16sel(xw, selA), bf16sel(xw, selB));
        const float2 du = f2mul(dt2, u2);
        const float dtq[2] = {dt2.x, dt2.y}, uq[2] = {u2.x, u2.y}, duq[2] = {du.x, du.y};
        const float dsq[2] = {sm.ds[tt][2 * slot + pq], sm.ds[tt][2 * slot + (pq ^ 1)]};
        float2 dB01, dB23, dC01, dC23;
        float dxp[2], ddp[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float2 a01, a23;
          decays(dtq[q], q, ap_tag, a01, a23);
          const float2 ds2 = f2dup(dsq[q]), du2 = f2dup(duq[q]);
          const float2 lam01 = f2fma(make_float2(Cq.x, Cq.y), ds2, mu[q][0]);
          const float2 lam23 = f2fma(make_float2(Cq.z, Cq.w), ds2, mu[q][1]);
          // with ZOH the input weight of a state is E x instead of delta x: lE = lam E takes the place of lam below
          float2 E01, E23, lw01 = lam01, lw23 = lam23, xw2 = du2;
          if (ZOH) {
            gain(dtq[q], q, a01, a23, E01, E23);
            lw01 = f2mul(lam01, E01);
            lw23 = f2mul(lam23, E23);
            xw2 = f2dup(uq[q]);
          }
          if (q == 0) {
            dC01 = f2mul(ds2, hist[t][q][0]);
            dC23 = f2mul(ds2, hist[t][q][1]);
            dB01 = f2mul(lw01, xw2);
            dB23 = f2mul(lw23, xw2);
          } else {
            dC01 = f2fma(ds2, hist[t][q][0], dC01);
            dC23 = f2fma(ds2, hist[t][q][1], dC23);
            dB01 = f2fma(lw01, xw2, dB01);
            dB23 = f2fma(lw23, xw2, dB23);
          }
          float2 lb = f2mul(lw01, make_float2(Bq.x, Bq.y));
          lb = f2fma(lw23, make_float2(Bq.z, Bq.w), lb);
          const float lamB = lb.x + lb.y;   // sum lam B (default rule), sum lam E B (ZOH)
          mu[q][0] = f2mul(a01, lam01);
          mu[q][1] = f2mul(a23, lam23);
          float2 hp0, hp1;   // h_{t-1}: the step before in registers, or the sub-block's start state (read again)
          if (t > 0) {
            hp0 = hist[t > 0 ? t - 1 : 0][q][0];
            hp1 = hist[t > 0 ? t - 1 : 0][q][1];
          } else {
            const float4 v = start_state(sb, q);
            hp0 = make_float2(v.x, v.y);
            hp1 = make_float2(v.z, v.w);
          }
          const float2 w01 = f2mul(mu[q][0], hp0), w23 = f2mul(mu[q][1], hp1);
          float2 wa = f2mul(w01, A2[q][0]);
          wa = f2fma(w23, A2[q][1], wa);
          dA2[q][0] = f2fma(w01, f2dup(dtq[q]), dA2[q][0]);
          dA2[q][1] = f2fma(w23, f2dup(dtq[q]), dA2[q][1]);
          if (ZOH) {
            // dE/ddelta = a: the step-size gradient through E is x sum mu B; dE/dA adds lam (dE/dA) B x to dA
            float2 mb = f2mul(mu[q][0], make_float2(Bq.x, Bq.y));
            mb = f2fma(mu[q][1], make_float2(Bq.z, Bq.w), mb);
            float2 G01, G23;
            gain_dA(dtq[q], q, a01, a23, E01, E23, G01, G23);
            const float2 uu = f2dup(uq[q]);
            dA2[q][0] = f2fma(f2mul(lam01, G01), f2mul(make_float2(Bq.x, Bq.y), uu), dA2[q][0]);
            dA2[q][1] = f2fma(f2mul(lam23, G23), f2mul(make_float2(Bq.z, Bq.w), uu), dA2[q][1]);
            dxp[q] = lamB;
            ddp[q] = fmaf(uq[q], mb.x + mb.y, (wa.x + wa.y) * kInvLog2e);
          } else {
            dxp[q] = dtq[q] * lamB;
            ddp[q] = fmaf(uq[q], lamB, (wa.x + wa.y) * kInvLog2e);
          }
        }
        sm.red[warp][t % kRB][quad][j][0] = make_float4(dB01.x, dB01.y, dB23.x, dB23.y);
        sm.red[warp][t % kRB][quad][j][1] = make_float4(dC01.x, dC01.y, dC23.x, dC23.y);
        dxw[t] = dxp[0] + __shfl_xor_sync(0xffffffffu, dxp[1], 1);
        ddw[t] = ddp[0] + __shfl_xor_sync(0xffffffffu, ddp[1], 1);
        if (t % kRB == 0) {
          // dB / dC of steps t .. t+kRB-1: sum over the 8 quads of this warp in ascending order;
          // lane -> (step = lane / 8, state quad = (lane / 2) % 4, dB or dC = lane % 2)
          __syncwarp();
          const int tr = lane >> 3, jr = (lane >> 1) & 3, hf = lane & 1;
          float4 acc4 = sm.red[warp][tr][0][jr][hf];
#pragma unroll
          for (int qd = 1; qd < 8; ++qd) {
            const float4 v = sm.red[warp][tr][qd][jr][hf];
            acc4.x += v.x; acc4.y += v.y; acc4.z += v.z; acc4.w += v.w;
          }
          *reinterpret_cast<float4*>(&sm.acc[warp][sb * kSB + t + tr][16 * hf + 4 * jr]) = acc4;
          __syncwarp();
        }
      }
      // second exchange: lanes j and j^2 hold sums of the same channel; the lower keeps steps 0..3, the upper 4..7
      float dxtot[4], ddtot[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float kx = gq ? dxw[4 + e] : dxw[e], sx = gq ? dxw[e] : dxw[4 + e];
        const float kd = gq ? ddw[4 + e] : ddw[e], sd = gq ? ddw[e] : ddw[4 + e];
        dxtot[e] = kx + __shfl_xor_sync(0xffffffffu, sx, 2);
        ddtot[e] = kd + __shfl_xor_sync(0xffffffffu, sd, 2);
      }
      // finalise 4 steps of channel pq: the rows of this sub-block are no longer read as inputs by this quad
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int tt = sb * kSB + 4 * gq + e;
        const float u = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(&sm.x[st][tt][slot])[pq] << 16);
        const float ds = sm.ds[tt][2 * slot + pq];
        dD_acc = fmaf(ds, u, dD_acc);
        reinterpret_cast<__nv_bfloat16*>(&sm.x[st][tt][slot])[pq] = __float2bfloat16_rn(fmaf(ds, Dk, dxtot[e]));
        float ddv = ddtot[e];
        if (SP) {
          // the gradient goes to the pre-activation v: d softplus(v) / dv = sigmoid(v)
          if (p.softplus) {
            const float v = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(&sm.d[st][tt][slot])[pq] << 16) + bias_pq;
            ddv *= sigmoid_fast(v);
          }
          // (a padded row still sees the adjoint that flows through it, so its value is not zero)
          if (tt < nlive) dbias_acc += ddv;
        }
        reinterpret_cast<__nv_bfloat16*>(&sm.d[st][tt][slot])[pq] = __float2bfloat16_rn(ddv);
      }
    }
  };


  // ---- persistent loop over claimed items
  if (tid == 0) {
    sm.sched[0] = atomicAdd(sched_counter, 1);
    sm.sched[2] = 0;
  }
  __syncthreads();
  Item cur = decode(sm.sched[0]);
  int st = 0;
  issue_item(cur, st);
  while (cur.chain + cur.ord * chains < total_items) {
    if (tid == 0) sm.sched[1] = atomicAdd(sched_counter, 1);   // claim ahead: its inputs are prefetched below
    if (cur.live) {
      d0 = cur.d_cta + 2 * slot;
      valid = d0 < D;
    }
    float4 ck[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
    bool ap = !p.general_A;
    if (cur.live) {
      // per-chain constants and the checkpoint state of this tile
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid) {
          a = *reinterpret_cast<const float4*>(p.A + (size_t)chan(q) * 16 + 4 * j);
          ck[q] = *reinterpret_cast<const float4*>(p.ckpt + (((size_t)cur.b * p.nck + cur.t0 / kCkptSteps) * D + chan(q)) * 16 + 4 * j);
        }
        const float step = a.y - a.x, tol = 1e-6f * fabsf(a.w);
        ap = ap && fabsf(a.z - (a.x + 2.f * step)) <= tol && fabsf(a.w - (a.x + 3.f * step)) <= tol;
        A2[q][0] = make_float2(a.x * kLog2e, a.y * kLog2e);
        A2[q][1] = make_float2(a.z * kLog2e, a.w * kLog2e);
        if (ZOH) {
          auto inv = [](float v) { return v != 0.f ? 1.f / v : 0.f; };
          invA[q][0] = make_float2(inv(a.x), inv(a.y));
          invA[q][1] = make_float2(inv(a.z), inv(a.w));
          zeroA = zeroA || a.x == 0.f || a.y == 0.f || a.z == 0.f || a.w == 0.f;
        }
      }
      Dk = (valid && p.Dskip != nullptr) ? p.Dskip[d0 + pq] : 0.f;
      if (SP) bias_pq = (valid && p.delta_bias != nullptr) ? p.delta_bias[d0 + pq] : 0.f;
      // carried values: from the segment's inflow for the first tile in order, else from the tile before in order
      if (cur.ord == 0) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          float4 m = make_float4(0.f, 0.f, 0.f, 0.f);
          if (valid && p.mu_in != nullptr)
            m = *reinterpret_cast<const float4*>(p.mu_in + (((size_t)cur.b * p.nseg + cur.seg) * D + chan(q)) * 16 + 4 * j);
          mu[q][0] = make_float2(m.x, m.y);
          mu[q][1] = make_float2(m.z, m.w);
          dA2[q][0] = dA2[q][1] = make_float2(0.f, 0.f);
        }
        dD_acc = 0.f;
        dbias_acc = 0.f;
      } else {
        if (tid == 0) {
          int spins = 0;
          while (ld_acquire(sched_flags + cur.chain) < cur.ord) {
            __nanosleep(100);
            if (++spins > (p.test_withhold ? 1000 : kSpinLimit) || ld_acquire(sched_abort) != 0) {
              atomicExch(sched_abort, 1);
              sm.sched[2] = 1;
              break;
            }
          }
        }
      }
    }
    ap = __all_sync(0xffffffffu, ap);
    if (ZOH) zeroA = __any_sync(0xffffffffu, zeroA);
    cp_async_wait_all();
    __syncthreads();                       // inputs of this tile landed; sched[1], sched[2] and the dependency are visible
    if (sm.sched[2] != 0) {                // a bounded wait gave up somewhere: every block leaves
      cp_async_wait_all();
      return;
    }
    const Item nxt = decode(sm.sched[1]);
    issue_item(nxt, st ^ 1);
    if (nxt.live) {
      // the checkpoint state of the next tile is needed the moment that tile starts: pull it into L2 now
      const int dn = nxt.d_cta + 2 * slot;
      if (dn < D) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const float* ckp = p.ckpt + (((size_t)nxt.b * p.nck + nxt.t0 / kCkptSteps) * D + dn + q) * 16 + 4 * j;
          asm volatile("prefetch.global.L2 [%0];" ::"l"(ckp));
        }
      }
    }
    if (cur.live) {
      if (cur.ord > 0) {
        const float4* hb = p.handoff + ((size_t)cur.chain * THREADS + tid) * kHandoffVec;
        const float4 m0 = __ldcg(hb), m1 = __ldcg(hb + 1), a0 = __ldcg(hb + 2), a1 = __ldcg(hb + 3), dd = __ldcg(hb + 4);
        mu[0][0] = make_float2(m0.x, m0.y); mu[0][1] = make_float2(m0.z, m0.w);
        mu[1][0] = make_float2(m1.x, m1.y); mu[1][1] = make_float2(m1.z, m1.w);
        dA2[0][0] = make_float2(a0.x, a0.y); dA2[0][1] = make_float2(a0.z, a0.w);
        dA2[1][0] = make_float2(a1.x, a1.y); dA2[1][1] = make_float2(a1.z, a1.w);
        dD_acc = dd.x;
        if (SP) dbias_acc = dd.y;
      }
      const size_t row0 = (size_t)cur.b * p.L + cur.t0;
      // widen B, C; per-element gate terms ds = dout * silu(z), gsp = dout * silu'(z)
      for (int c = tid; c < kBT * 8; c += THREADS) {
        const int tt = c >> 3, w = c & 7;
        const uint32_t vb = sm.rawB[st][tt][w], vc = sm.rawC[st][tt][w];
        reinterpret_cast<float2*>(&sm.fB[tt][0])[w] = make_float2(bf16lo(vb), bf16hi(vb));
        reinterpret_cast<float2*>(&sm.fC[tt][0])[w] = make_float2(bf16lo(vc), bf16hi(vc));
      }
      for (int c = tid; c < kBT * (CH / 2); c += THREADS) {
        const int tt = c / (CH / 2), w = c % (CH / 2);
        const uint32_t zw = sm.z[st][tt][w], gw = sm.g[st][tt][w];
        float2 dsv, gpv;
        const float g0 = bf16lo(gw), g1 = bf16hi(gw);
        if (has_z) {
          const float z0 = bf16lo(zw), z1 = bf16hi(zw);
          const float s0 = sigmoid_fast(z0), s1 = sigmoid_fast(z1);
          dsv = make_float2(g0 * z0 * s0, g1 * z1 * s1);
          gpv = make_float2(g0 * s0 * fmaf(z0, 1.f - s0, 1.f), g1 * s1 * fmaf(z1, 1.f - s1, 1.f));
        } else {
          dsv = make_float2(g0, g1);
          gpv = make_float2(0.f, 0.f);
        }
        *reinterpret_cast<float2*>(&sm.ds[tt][2 * w]) = dsv;
        if (SP) {
          // step size of Algorithm 2 step 4 from the pre-activation; rows past the end stay identity steps
          const uint32_t dw = sm.d[st][tt][w];
          const int c0 = cur.d_cta + 2 * w;
          const bool chan_ok = c0 < D && p.delta_bias != nullptr;
          float v0 = bf16lo(dw) + (chan_ok ? p.delta_bias[c0] : 0.f), v1 = bf16hi(dw) + (chan_ok ? p.delta_bias[c0 + 1] : 0.f);
          if (p.softplus) {
            v0 = softplus_fast(v0);
            v1 = softplus_fast(v1);
          }
          gpv = (cur.t0 + tt < cur.t_end) ? make_float2(v0, v1) : make_float2(0.f, 0.f);
        }
        *reinterpret_cast<float2*>(&sm.gsp[tt][2 * w]) = gpv;
      }
      __syncthreads();
      if (ap) process_tile(st, std::true_type{}, ck, cur.t_end - cur.t0);
      else process_tile(st, std::false_type{}, ck, cur.t_end - cur.t0);
      __syncthreads();
      // results of the tile: 16-byte stores of dx, ddelta, dz; block partial sums of dB, dC
      for (int c = tid; c < kBT * CHUNKS; c += THREADS) {
        const int tt = c / CHUNKS, cc = c % CHUNKS;
        if (cur.t0 + tt < cur.t_end && cur.d_cta + cc * 8 < D) {
          const size_t g = (row0 + tt) * D + cur.d_cta + cc * 8;
          *reinterpret_cast<uint4*>(gdx + g) = *reinterpret_cast<const uint4*>(&sm.x[st][tt][cc * 4]);
          *reinterpret_cast<uint4*>(gdd + g) = *reinterpret_cast<const uint4*>(&sm.d[st][tt][cc * 4]);
          if (gdz != nullptr) *reinterpret_cast<uint4*>(gdz + g) = *reinterpret_cast<const uint4*>(&sm.z[st][tt][cc * 4]);
        }
      }
      const size_t bln = (size_t)p.batch * p.L * 16;
      for (int c = tid; c < kBT * 8; c += THREADS) {  // float4 granules: [step][dB 0..15 | dC 0..15]
        const int tt = c >> 3, f = c & 7;
        if (cur.t0 + tt < cur.t_end) {
          float4 v = *reinterpret_cast<const float4*>(&sm.acc[0][tt][4 * f]);
#pragma unroll
          for (int w = 1; w < kBwdFastWarps; ++w) {
            const float4 o = *reinterpret_cast<const float4*>(&sm.acc[w][tt][4 * f]);
            v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
          }
          const int which = f >> 2;
          *reinterpret_cast<float4*>(p.dBC_part + ((size_t)cur.grp * 2 + which) * bln + (row0 + tt) * 16 + 4 * (f & 3)) = v;
        }
      }
      if (cur.ord + 1 < cur.ntiles) {
        // hand the carried values to whoever runs the next tile of this chain
        float4* hb = p.handoff + ((size_t)cur.chain * THREADS + tid) * kHandoffVec;
        __stcg(hb, make_float4(mu[0][0].x, mu[0][0].y, mu[0][1].x, mu[0][1].y));
        __stcg(hb + 1, make_float4(mu[1][0].x, mu[1][0].y, mu[1][1].x, mu[1][1].y));
        __stcg(hb + 2, make_float4(dA2[0][0].x, dA2[0][0].y, dA2[0][1].x, dA2[0][1].y));
        __stcg(hb + 3, make_float4(dA2[1][0].x, dA2[1][0].y, dA2[1][1].x, dA2[1][1].y));
        __stcg(hb + 4, make_float4(dD_acc, SP ? dbias_acc : 0.f, 0.f, 0.f));
        __threadfence();
        __syncthreads();
        if (tid == 0 && !p.test_withhold) st_release(sched_flags + cur.chain, cur.ord + 1);
      } else {
        // first tile in time: the chain is complete
        if (valid) {
          const size_t part = (size_t)cur.b * p.nseg + cur.seg;
#pragma unroll
          for (int q = 0; q < 2; ++q)
            *reinterpret_cast<float4*>(p.dA_part + (part * D + chan(q)) * 16 + 4 * j) =
                make_float4(dA2[q][0].x, dA2[q][0].y, dA2[q][1].x, dA2[q][1].y);
        }
        if (valid && cur.seg == 0 && p.dh0 != nullptr) {
          // the adjoint that leaves the first step is the gradient of the initial state
#pragma unroll
          for (int q = 0; q < 2; ++q)
            *reinterpret_cast<float4*>(p.dh0 + ((size_t)cur.b * D + chan(q)) * 16 + 4 * j) =
                make_float4(mu[q][0].x, mu[q][0].y, mu[q][1].x, mu[q][1].y);
        }
        // dD: lanes j and j^2 accumulated disjoint steps of the same channel
        const float dsum2 = dD_acc + __shfl_xor_sync(0xffffffffu, dD_acc, 2);
        if (valid && j < 2) p.dD_part[((size_t)cur.b * p.nseg + cur.seg) * D + d0 + pq] = dsum2;
        if (SP) {
          const float bsum2 = dbias_acc + __shfl_xor_sync(0xffffffffu, dbias_acc, 2);
          if (valid && j < 2 && p.dbias_part != nullptr)
            p.dbias_part[((size_t)cur.b * p.nseg + cur.seg) * D + d0 + pq] = bsum2;
        }
      }
    }
    cur = nxt;
    st ^= 1;
  }
  cp_async_wait_all();
}

bool bwd_fast_applicable(const ssm_problem_t& prob, const BwdParams& p) {
  auto al16 = [](const void* q) { return q == nullptr || (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
  if (p.static_B || p.static_C) return false;  // input-dependent B, C only
  // work items are numbered with 32-bit integers (one spare bit for the claims that run past the end)
  const long long items = (long long)p.batch * p.nseg * ((p.D + kBwdFastCH - 1) / kBwdFastCH) * (p.seg_steps / kBT);
  if (items > (1LL << 30)) return false;
  return prob.io_dtype == SSM_BF16 && prob.N == 16 && prob.D % 8 == 0 && p.seg_steps % kBT == 0 && al16(p.x) &&
         al16(p.delta) && al16(p.z) && al16(p.B) && al16(p.C) && al16(p.dout) && al16(p.dx) && al16(p.ddelta) &&
         al16(p.dz) && al16(p.A) && al16(p.ckpt) && al16(p.mu_in) && al16(p.dh0) && al16(p.dBC_part) && al16(p.dA_part) &&
         p.sched != nullptr && p.handoff != nullptr;
}

int bwd_fast_channels_per_block() { return kBwdFastCH; }
size_t bwd_fast_handoff_bytes_per_chain() { return sizeof(float4) * kHandoffVec * kBwdFastThreads; }

template <bool SP, bool ZOH>
static cudaError_t launch_bwd_fast_sp(const Plan& plan, const BwdParams& p, cudaStream_t s) {
  constexpr size_t smem = sizeof(BwdFastSmem);
  cudaError_t e = cudaFuncSetAttribute(ssm_bwd_fast_kernel<SP, ZOH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 0, per_sm = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ssm_bwd_fast_kernel<SP, ZOH>, kBwdFastThreads, smem)) != cudaSuccess)
    return e;
  const int groups = (p.D + kBwdFastCH - 1) / kBwdFastCH;
  const long long chains = (long long)p.batch * plan.nseg * groups;
  const long long items = chains * (plan.seg_steps / kBT);
  const long long resident = (long long)sms * (per_sm > 0 ? per_sm : 1);
  const unsigned grid = (unsigned)(items < resident ? items : resident);
  // the claim counter, the abort word and the flag of every chain were zeroed by the caller (ssm_scan_bwd)
  ssm_bwd_fast_kernel<SP, ZOH><<<grid, kBwdFastThreads, smem, s>>>(p);
  return cudaGetLastError();
}

// SP: the step size is bias + pre-activation, through the softplus if asked (Algorithm 2 step 4)
cudaError_t launch_bwd_fast(const Plan& plan, const BwdParams& p, cudaStream_t s) {
  const bool sp = p.softplus || p.delta_bias != nullptr;
  if (p.zoh) return sp ? launch_bwd_fast_sp<true, true>(plan, p, s) : launch_bwd_fast_sp<false, true>(plan, p, s);
  return sp ? launch_bwd_fast_sp<true, false>(plan, p, s) : launch_bwd_fast_sp<false, false>(plan, p, s);
}

}  // namespace ssm
