// Backward selective scan, tuned path: bf16 io, N = 16, D % 8 == 0, 16-byte aligned pointers.
// Same mathematics as ssm_bwd.cu (adjoint of Eq. 2a/2b with skip term and gate; states recomputed, Section 3.3).
//
// One warp is one worker, as in the tuned forward kernel (ssm_fwd_warp.cu): it owns CW adjacent channels of one batch
// entry, walks its part of the sequence backwards in tiles of 8 steps, stages its own tiles with cp.async and shares
// nothing with the other warps of its block.  A thread holds S states of CPT channels as packed float2 pairs; the
// LPC = 16 / S lanes of a group cover the 16 states of the group's channels.  With CPT = LPC (16 recurrences per thread,
// CW = 32) local channel q of lane j (j = lane % LPC) is channel j ^ q of the group, so the sums over n are
// reduce-scattered with xor-shuffles and every lane finishes exactly one channel per step (channel `lane`).  With
// S = 8, CPT = 1 (8 recurrences per thread, CW = 16) the two lanes of a group share one channel, the sums are completed
// in both, and lane j finishes the steps of parity j; this mapping needs half the registers, so twice as many warps are
// resident, and a problem has twice as many chains to give them.
//
// Recomputation.  The forward pass left the state at the start of every block of 8 steps, so a sub-block of 8 steps is
// rebuilt directly from its checkpoint: a forward sweep keeps the states after the odd steps in registers (64
// registers), the reverse sweep walks the steps in pairs and rebuilds the state after the even step of a pair from the
// one before it (one multiply-add per state), which is also the h_{t-1} of the odd step.
//
// Sums.  The sums over n (readout for dz, sum lam B for dx and ddelta, sum w A for ddelta) are reduce-scattered over
// the lane group.  dB and dC are summed over the CPT channels of a thread in registers and over the lane groups of
// the warp through a transposing pass over shared memory every 4 steps, in a fixed order, and leave the warp as partial
// sums per group of 32 channels that ssm_bwd_reduce_kernel adds in ascending group order.  dA and dD accumulate in
// registers along the chain.  Everything is deterministic; there are no floating-point atomics.
//
// Schedule.  As in the forward kernel (WarpSched in ssm_common.cuh), in reverse time: a chain that two workers share
// hands the adjoint mu and the dA / dD accumulators from one to the other once, through L2, behind a bounded wait.
#include <cstdlib>
#include <type_traits>

#include "ssm_common.cuh"

namespace ssm {

int warp_workers(int chains, int sms, int per_sm, int max_workers);

namespace {

constexpr int kBT = 8;             // steps per tile (one sub-block: 8 warps per SM need small tiles)
constexpr int kSB = kCkptSteps;    // steps per sub-block = checkpoint spacing
constexpr int kRB = 4;             // steps between two dB / dC transposes
constexpr int kBwdWarps = 4;       // warps per block
constexpr int kBwdFastChannels = 32;   // channels per warp of the mapping the launcher picks
// float4 per lane of a hand-off: mu (4), dA (4), dD and dbias (1), and 4 more for each of dB / dC that is a parameter
__host__ __device__ constexpr int bwd_handoff_vec(int bc) { return 9 + 4 * ((bc & 1) + ((bc >> 1) & 1)); }
constexpr float kInvLog2e = 0.6931471805599453f;
static_assert(kSB == 8 && kBT % kSB == 0, "sub-blocks of 8 steps, whole sub-blocks per tile");

template <int S, int CPT, bool SP>
struct BwdWarpSmem {
  static constexpr int CW = (32 / (16 / S)) * CPT;   // channels per warp
  uint32_t x[2][kBT][CW / 2];    // bf16 pairs
  uint32_t d[2][kBT][CW / 2];
  uint32_t z[2][kBT][CW / 2];
  uint32_t g[2][kBT][CW / 2];
  uint32_t rB[2][kBT][8];        // bf16 pairs, 16 states
  uint32_t rC[2][kBT][8];
  float4 ck[2][kBT / kSB][CPT * S / 4][32];   // checkpoint states: [sub-block][float4 of the thread][lane]
  float fB[kBT][16];             // B and C of the tile widened to float
  float fC[kBT][16];
  float ds[kBT][CW];             // dout * silu(z)
  float gp[kBT][CW];             // dout * silu'(z)
  float dF[SP ? kBT : 1][CW];    // SP: step sizes after bias and softplus
  uint32_t ox[kBT][CW / 2];      // dx, ddelta, dz of the tile (bf16 pairs)
  uint32_t od[kBT][CW / 2];
  uint32_t oz[kBT][CW / 2];
  float4 red[kRB][32][S / 2];    // dB / dC terms of 4 steps: [step][lane][dB float4s | dC float4s], swizzled
};


template <int S, int CPT_>
struct Lane {
  static constexpr int LPC = 16 / S, CPT = CPT_, H = S / 2, V = S / 2;   // V: float4 of dB / dC terms per thread and step
  static constexpr int CW = (32 / LPC) * CPT;       // channels per warp
  static constexpr bool OWN = (CPT == LPC);          // every lane finishes its own channel (else: parity of the step)
  static_assert(OWN || (CPT == 1 && LPC == 2), "supported mappings");
  int lane, j, g, co;    // co: the channel (within the warp) this lane finishes
  uint32_t sel0, sel1;
  __device__ __forceinline__ explicit Lane(int l) : lane(l), j(l % LPC), g(l / LPC) {
    co = OWN ? lane : g;
    sel0 = (j & 1) ? 0x3244u : 0x1044u;
    sel1 = (j & 1) ? 0x1044u : 0x3244u;
  }
  // the CPT values of a tile row (CW channels as bf16 pairs) that belong to this thread, by local channel
  __device__ __forceinline__ void unpack_row(const uint32_t* row, float (&v)[CPT]) const {
    if constexpr (!OWN) {
      v[0] = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(row)[g] << 16);
    } else if constexpr (CPT == 1) {
      v[0] = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(row)[lane] << 16);
    } else if constexpr (CPT == 2) {
      const uint32_t w = row[g];
      v[0] = bf16sel(w, sel0);
      v[1] = bf16sel(w, sel1);
    } else {
      const uint2 w = *reinterpret_cast<const uint2*>(row + 2 * g);
      const uint32_t wa = (j & 2) ? w.y : w.x, wb = (j & 2) ? w.x : w.y;
      v[0] = bf16sel(wa, sel0);
      v[1] = bf16sel(wa, sel1);
      v[2] = bf16sel(wb, sel0);
      v[3] = bf16sel(wb, sel1);
    }
  }
  // the same from a row of CW floats
  __device__ __forceinline__ void pick_row(const float* row, float (&v)[CPT]) const {
    if constexpr (!OWN) {
      v[0] = row[g];
    } else if constexpr (CPT == 1) {
      v[0] = row[lane];
    } else if constexpr (CPT == 2) {
      const float2 f = *reinterpret_cast<const float2*>(row + 2 * g);
      v[0] = (j & 1) ? f.y : f.x;
      v[1] = (j & 1) ? f.x : f.y;
    } else {
      const float4 f = *reinterpret_cast<const float4*>(row + 4 * g);
      const float a0 = (j & 2) ? f.z : f.x, a1 = (j & 2) ? f.w : f.y, b0 = (j & 2) ? f.x : f.z, b1 = (j & 2) ? f.y : f.w;
      v[0] = (j & 1) ? a1 : a0;
      v[1] = (j & 1) ? a0 : a1;
      v[2] = (j & 1) ? b1 : b0;
      v[3] = (j & 1) ? b0 : b1;
    }
  }
  // this thread's S states of a row of 16 floats
  __device__ __forceinline__ void load_states_f(const float* row, float2 (&v)[H]) const {
#pragma unroll
    for (int k = 0; k < H / 2; ++k) {
      const float4 a = *reinterpret_cast<const float4*>(row + S * j + 4 * k);
      v[2 * k] = make_float2(a.x, a.y);
      v[2 * k + 1] = make_float2(a.z, a.w);
    }
  }
  // this thread's S states of a packed B or C row (16 states as 8 bf16 pairs), widened
  __device__ __forceinline__ void load_states(const uint32_t* row, float2 (&v)[H]) const {
    if constexpr (H == 8) {
      const uint4 a = *reinterpret_cast<const uint4*>(row), b = *reinterpret_cast<const uint4*>(row + 4);
      const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = make_float2(bf16lo(w[k]), bf16hi(w[k]));
    } else if constexpr (H == 4) {
      const uint4 a = *reinterpret_cast<const uint4*>(row + 4 * j);
      const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
      for (int k = 0; k < 4; ++k) v[k] = make_float2(bf16lo(w[k]), bf16hi(w[k]));
    } else {
      const uint2 a = *reinterpret_cast<const uint2*>(row + 2 * j);
      v[0] = make_float2(bf16lo(a.x), bf16hi(a.x));
      v[1] = make_float2(bf16lo(a.y), bf16hi(a.y));
    }
  }
};

// Decays of one (step, channel): general A (one exponential per state) or arithmetic-progression A (two exponentials)
template <int H, bool AP>
__device__ __forceinline__ void decays(float dt, const float2 (&A2)[H], float a0s, float rs, float2 (&a)[H]) {
  if constexpr (AP) {
    const float a0 = ex2_approx(dt * a0s);
    const float rr = ex2_approx(dt * rs);
    const float r2 = rr * rr;
    a[0] = make_float2(a0, a0 * rr);
    if constexpr (H > 1) a[1] = f2mul(a[0], f2dup(r2));
    if constexpr (H > 2) {
      const float r4 = r2 * r2;
      a[2] = f2mul(a[0], f2dup(r4));
      a[3] = f2mul(a[1], f2dup(r4));
      if constexpr (H > 4) {
        const float r8 = r4 * r4;
#pragma unroll
        for (int k = 0; k < 4; ++k) a[4 + k] = f2mul(a[k], f2dup(r8));
      }
    }
  } else {
#pragma unroll
    for (int k = 0; k < H; ++k) {
      const float2 e = f2mul(f2dup(dt), A2[k]);
      a[k] = make_float2(ex2_approx(e.x), ex2_approx(e.y));
    }
  }
}

// Per-thread state that lives along a chain
// BC: bit 0 = B is a per-channel parameter [D][16] (Algorithm 1's non-selective B), bit 1 = the same for C
template <int S, int CPT, bool ZOH, int BC>
struct ChainRegs {
  static constexpr int H = S / 2;
  static constexpr bool SB = BC & 1, SC = BC & 2;
  float2 Bst[SB ? CPT : 1][SB ? H : 1], dBs[SB ? CPT : 1][SB ? H : 1];   // the parameter and its gradient over time
  float2 Cst[SC ? CPT : 1][SC ? H : 1], dCs[SC ? CPT : 1][SC ? H : 1];
  float2 A2[CPT][H];    // A * log2(e)
  // ZOH: B-bar = E B with the input gain E = (a - 1) / A (Eq. 4): 1 / A (0 where A = 0)
  float2 invA[ZOH ? CPT : 1][ZOH ? H : 1];
  float minA;           // ZOH: smallest |A| among this thread's states
  float a0s[CPT], rs[CPT];
  float2 mu[CPT][H];    // adjoint flowing backwards in time
  float2 dA[CPT][H];
  float Dk, dD, dbias;
};

// One sub-block of 8 steps: rows [r0, r0 + 8) of the tile; nlive = rows of the tile inside the segment.
// ZS (ZOH only): some |delta A| of the sub-block is too small for the closed form of the input gain.
template <int S, int CPT, bool SP, bool AP, bool ZOH, bool ZS, int BC>
__device__ __forceinline__ void sub_block(const Lane<S, CPT>& ln, ChainRegs<S, CPT, ZOH, BC>& cr, int r0, int nlive, float gate_on,
                                          bool softplus, const uint32_t* tx, const uint32_t* td, const float* tfB,
                                          const float* tfC, const float* tds, const float* tgp, const float* tdF,
                                          const float4* tck, uint32_t* tox, uint32_t* tod, uint32_t* toz, float4* tred,
                                          float* part_dB, float* part_dC, int* abort_word) {
  using LN = Lane<S, CPT>;
  constexpr int LPC = LN::LPC, H = LN::H, V = LN::V, CW = LN::CW, WPR = CW / 2;
  constexpr bool OWN = LN::OWN;
  constexpr bool SB = BC & 1, SC = BC & 2;
  const int lane = ln.lane;
  // B / C of a (step, channel, state pair): the staged row, or the channel's parameter
  auto Bof = [&](const float2 (&Bv)[H], int q, int k) { return SB ? cr.Bst[SB ? q : 0][SB ? k : 0] : Bv[k]; };
  auto Cof = [&](const float2 (&Cv)[H], int q, int k) { return SC ? cr.Cst[SC ? q : 0][SC ? k : 0] : Cv[k]; };
  // ZOH input gain E = (a - 1) / A and its derivative dE/dA = (delta a - E) / A, each with its series for small
  // delta A (which covers A = 0); dE/ddelta = a
  auto gain = [&](int q, int k, float2 a, float dtq) {
    const float2 invA = cr.invA[ZOH ? q : 0][ZOH ? k : 0];
    if constexpr (ZS) return zoh_gain_pair(a, f2mul(f2dup(dtq), cr.A2[q][k]), dtq, invA);
    else return zoh_gain_closed(a, invA);
  };
  auto gain_dA = [&](int q, int k, float2 a, float2 E, float dtq) {
    const float2 invA = cr.invA[ZOH ? q : 0][ZOH ? k : 0];
    if constexpr (ZS) return zoh_gain_dA_pair(a, E, f2mul(f2dup(dtq), cr.A2[q][k]), dtq, invA);
    else return zoh_gain_dA_closed(a, E, dtq, invA);
  };
  // ---- forward sweep from the checkpoint: the states after the odd steps stay in registers
  float2 hist[kSB / 2][CPT][H];
  {
    float2 h[CPT][H];
#pragma unroll
    for (int q = 0; q < CPT; ++q)
#pragma unroll
      for (int k = 0; k < S / 4; ++k) {
        const float4 v = tck[(q * (S / 4) + k) * 32 + lane];
        h[q][2 * k] = make_float2(v.x, v.y);
        h[q][2 * k + 1] = make_float2(v.z, v.w);
      }
    float dt[kSB][CPT], u[kSB][CPT];
#pragma unroll
    for (int t = 0; t < kSB; ++t) {
      const int r = SSM_TILE_ROW(r0 + t, kBT, abort_word);
      if constexpr (SP) ln.pick_row(tdF + r * CW, dt[t]);
      else ln.unpack_row(td + r * WPR, dt[t]);
      ln.unpack_row(tx + r * WPR, u[t]);
    }
#pragma unroll
    for (int t = 0; t < kSB; ++t) {
      const int r = SSM_TILE_ROW(r0 + t, kBT, abort_word);
      float2 Bv[H];
      if constexpr (!SB) ln.load_states_f(tfB + r * 16, Bv);
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        float2 a[H];
        decays<H, AP>(dt[t][q], cr.A2[q], cr.a0s[q], cr.rs[q], a);
        const float2 du2 = f2dup(dt[t][q] * u[t][q]);
#pragma unroll
        for (int k = 0; k < H; ++k) {
          const float2 Bk = Bof(Bv, q, k);
          const float2 bx = ZOH ? f2mul(f2mul(gain(q, k, a[k], dt[t][q]), f2dup(u[t][q])), Bk) : f2mul(du2, Bk);
          h[q][k] = f2fma(a[k], h[q][k], bx);
          if (t & 1) hist[t >> 1][q][k] = h[q][k];
        }
      }
    }
  }
  // ---- reverse sweep in pairs of steps (2m + 1, 2m)
#pragma unroll
  for (int m = kSB / 2 - 1; m >= 0; --m) {
    // ======== odd step t1 = 2m + 1: its state is hist[m]; its w = mu h_{t-1} waits for the even step's state
    const int r1 = SSM_TILE_ROW(r0 + 2 * m + 1, kBT, abort_word);
    float dt1[CPT], u1[CPT], ds1[CPT];
    if constexpr (SP) ln.pick_row(tdF + r1 * CW, dt1);
    else ln.unpack_row(td + r1 * WPR, dt1);
    ln.unpack_row(tx + r1 * WPR, u1);
    ln.pick_row(tds + r1 * CW, ds1);
    const float gp1 = tgp[r1 * CW + ln.co];
    float y1[CPT], lb1[CPT], mb1[ZOH ? CPT : 1];   // mb: sum mu B (ZOH: the step-size gradient through E)
    {
      float2 Bv[H], Cv[H];
      if constexpr (!SB) ln.load_states_f(tfB + r1 * 16, Bv);
      if constexpr (!SC) ln.load_states_f(tfC + r1 * 16, Cv);
      float2 dBt[H], dCt[H];
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        float2 a[H];
        decays<H, AP>(dt1[q], cr.A2[q], cr.a0s[q], cr.rs[q], a);
        // with ZOH the input weight of a state is E x instead of delta x: lw = lam E takes the place of lam below
        const float2 ds2 = f2dup(ds1[q]), du2 = f2dup(ZOH ? u1[q] : dt1[q] * u1[q]);
        float2 yv = make_float2(0.f, 0.f), lb = yv, mb = yv;
#pragma unroll
        for (int k = 0; k < H; ++k) {
          const float2 hc = hist[m][q][k];
          const float2 Bk = Bof(Bv, q, k), Ck = Cof(Cv, q, k);
          const float2 lam = f2fma(Ck, ds2, cr.mu[q][k]);
          float2 lw = lam;
          if constexpr (ZOH) {
            const float2 E = gain(q, k, a[k], dt1[q]);
            lw = f2mul(lam, E);
            // dE/dA adds lam (dE/dA) B x to dA
            cr.dA[q][k] = f2fma(f2mul(lam, gain_dA(q, k, a[k], E, dt1[q])), f2mul(Bk, f2dup(u1[q])), cr.dA[q][k]);
          }
          // dB / dC terms: summed over the thread's channels for the cross-lane sum, or over time per channel
          if constexpr (SC) cr.dCs[SC ? q : 0][SC ? k : 0] = f2fma(ds2, hc, cr.dCs[SC ? q : 0][SC ? k : 0]);
          else if (q == 0) dCt[k] = f2mul(ds2, hc);
          else dCt[k] = f2fma(ds2, hc, dCt[k]);
          if constexpr (SB) cr.dBs[SB ? q : 0][SB ? k : 0] = f2fma(lw, du2, cr.dBs[SB ? q : 0][SB ? k : 0]);
          else if (q == 0) dBt[k] = f2mul(lw, du2);
          else dBt[k] = f2fma(lw, du2, dBt[k]);
          lb = f2fma(lw, Bk, lb);
          yv = f2fma(Ck, hc, yv);
          cr.mu[q][k] = f2mul(a[k], lam);
          if constexpr (ZOH) mb = f2fma(cr.mu[q][k], Bk, mb);
        }
        y1[q] = yv.x + yv.y;
        lb1[q] = lb.x + lb.y;
        if constexpr (ZOH) mb1[q] = mb.x + mb.y;
      }
      // dB / dC terms of this step into the transposing buffer (swizzled: conflict-free 16-byte stores)
      float4* rrow = tred + ((2 * m + 1) & (kRB - 1)) * 32 * V + lane * V;
      const int swz = (lane / (8 / V)) & (V - 1);
#pragma unroll
      for (int v = 0; v < V / 2; ++v) {
        if constexpr (!SB) rrow[v ^ swz] = make_float4(dBt[2 * v].x, dBt[2 * v].y, dBt[2 * v + 1].x, dBt[2 * v + 1].y);
        if constexpr (!SC)
          rrow[(V / 2 + v) ^ swz] = make_float4(dCt[2 * v].x, dCt[2 * v].y, dCt[2 * v + 1].x, dCt[2 * v + 1].y);
      }
    }
    if constexpr (OWN) {
#pragma unroll
      for (int mm = 1; mm < LPC; mm <<= 1) {
#pragma unroll
        for (int q = 0; q < CPT; ++q)
          if ((q & (2 * mm - 1)) == 0) {
            y1[q] += __shfl_xor_sync(0xffffffffu, y1[q + mm], mm);
            lb1[q] += __shfl_xor_sync(0xffffffffu, lb1[q + mm], mm);
            if constexpr (ZOH) mb1[q] += __shfl_xor_sync(0xffffffffu, mb1[q + mm], mm);
          }
      }
    } else {
      y1[0] += __shfl_xor_sync(0xffffffffu, y1[0], 1);
      lb1[0] += __shfl_xor_sync(0xffffffffu, lb1[0], 1);
      if constexpr (ZOH) mb1[0] += __shfl_xor_sync(0xffffffffu, mb1[0], 1);
    }

    // ======== even step t0 = 2m: its state is rebuilt from the one before it
    const int r0e = SSM_TILE_ROW(r0 + 2 * m, kBT, abort_word);
    float dt0[CPT], u0[CPT], ds0[CPT];
    if constexpr (SP) ln.pick_row(tdF + r0e * CW, dt0);
    else ln.unpack_row(td + r0e * WPR, dt0);
    ln.unpack_row(tx + r0e * WPR, u0);
    ln.pick_row(tds + r0e * CW, ds0);
    const float gp0 = tgp[r0e * CW + ln.co];
    float y0[CPT], lb0[CPT], wa0[CPT], wa1[CPT], mb0[ZOH ? CPT : 1];
    {
      float2 Bv[H], Cv[H];
      if constexpr (!SB) ln.load_states_f(tfB + r0e * 16, Bv);
      if constexpr (!SC) ln.load_states_f(tfC + r0e * 16, Cv);
      float2 dBt[H], dCt[H];
#pragma unroll
      for (int q = 0; q < CPT; ++q) {
        float2 a[H];
        decays<H, AP>(dt0[q], cr.A2[q], cr.a0s[q], cr.rs[q], a);
        const float2 ds2 = f2dup(ds0[q]), du2 = f2dup(ZOH ? u0[q] : dt0[q] * u0[q]), dt02 = f2dup(dt0[q]), dt12 = f2dup(dt1[q]);
        float2 yv = make_float2(0.f, 0.f), lb = yv, w0a = yv, w1a = yv, mb = yv;
#pragma unroll
        for (int k = 0; k < H; ++k) {
          float2 hpp;   // the state before the even step: the history entry before, or the checkpoint
          if (m > 0) {
            hpp = hist[m > 0 ? m - 1 : 0][q][k];
          } else {
            const float4 v = tck[(q * (S / 4) + (k >> 1)) * 32 + lane];
            hpp = (k & 1) ? make_float2(v.z, v.w) : make_float2(v.x, v.y);
          }
          float2 E = make_float2(0.f, 0.f);
          if constexpr (ZOH) E = gain(q, k, a[k], dt0[q]);
          const float2 Bk = Bof(Bv, q, k), Ck = Cof(Cv, q, k);
          const float2 he = f2fma(a[k], hpp, f2mul(ZOH ? f2mul(E, du2) : du2, Bk));      // h after the even step
          const float2 w1 = f2mul(cr.mu[q][k], he);                   // the odd step's w = mu_{t1} h_{t1 - 1}
          w1a = f2fma(w1, cr.A2[q][k], w1a);
          cr.dA[q][k] = f2fma(w1, dt12, cr.dA[q][k]);
          const float2 lam = f2fma(Ck, ds2, cr.mu[q][k]);
          float2 lw = lam;
          if constexpr (ZOH) {
            lw = f2mul(lam, E);
            cr.dA[q][k] = f2fma(f2mul(lam, gain_dA(q, k, a[k], E, dt0[q])), f2mul(Bk, f2dup(u0[q])), cr.dA[q][k]);
          }
          if constexpr (SC) cr.dCs[SC ? q : 0][SC ? k : 0] = f2fma(ds2, he, cr.dCs[SC ? q : 0][SC ? k : 0]);
          else if (q == 0) dCt[k] = f2mul(ds2, he);
          else dCt[k] = f2fma(ds2, he, dCt[k]);
          if constexpr (SB) cr.dBs[SB ? q : 0][SB ? k : 0] = f2fma(lw, du2, cr.dBs[SB ? q : 0][SB ? k : 0]);
          else if (q == 0) dBt[k] = f2mul(lw, du2);
          else dBt[k] = f2fma(lw, du2, dBt[k]);
          lb = f2fma(lw, Bk, lb);
          yv = f2fma(Ck, he, yv);
          cr.mu[q][k] = f2mul(a[k], lam);
          if constexpr (ZOH) mb = f2fma(cr.mu[q][k], Bk, mb);
          const float2 w0 = f2mul(cr.mu[q][k], hpp);
          w0a = f2fma(w0, cr.A2[q][k], w0a);
          cr.dA[q][k] = f2fma(w0, dt02, cr.dA[q][k]);
        }
        y0[q] = yv.x + yv.y;
        lb0[q] = lb.x + lb.y;
        wa0[q] = w0a.x + w0a.y;
        wa1[q] = w1a.x + w1a.y;
        if constexpr (ZOH) mb0[q] = mb.x + mb.y;
      }
      float4* rrow = tred + ((2 * m) & (kRB - 1)) * 32 * V + lane * V;
      const int swz = (lane / (8 / V)) & (V - 1);
#pragma unroll
      for (int v = 0; v < V / 2; ++v) {
        if constexpr (!SB) rrow[v ^ swz] = make_float4(dBt[2 * v].x, dBt[2 * v].y, dBt[2 * v + 1].x, dBt[2 * v + 1].y);
        if constexpr (!SC)
          rrow[(V / 2 + v) ^ swz] = make_float4(dCt[2 * v].x, dCt[2 * v].y, dCt[2 * v + 1].x, dCt[2 * v + 1].y);
      }
    }
    if constexpr (OWN) {
#pragma unroll
      for (int mm = 1; mm < LPC; mm <<= 1) {
#pragma unroll
        for (int q = 0; q < CPT; ++q)
          if ((q & (2 * mm - 1)) == 0) {
            y0[q] += __shfl_xor_sync(0xffffffffu, y0[q + mm], mm);
            lb0[q] += __shfl_xor_sync(0xffffffffu, lb0[q + mm], mm);
            wa0[q] += __shfl_xor_sync(0xffffffffu, wa0[q + mm], mm);
            wa1[q] += __shfl_xor_sync(0xffffffffu, wa1[q + mm], mm);
            if constexpr (ZOH) mb0[q] += __shfl_xor_sync(0xffffffffu, mb0[q + mm], mm);
          }
      }
      // ---- finish both steps of the pair for this lane's own channel
      const float dz1 = gp1 * fmaf(cr.Dk, u1[0], y1[0]);
      // default rule: dx = delta sum lam B, ddelta = x sum lam B + sum w A; ZOH: dx = sum lam E B, ddelta = x sum mu B + sum w A
      const float dx1 = ZOH ? fmaf(ds1[0], cr.Dk, lb1[0]) : fmaf(dt1[0], lb1[0], ds1[0] * cr.Dk);
      const float dz0 = gp0 * fmaf(cr.Dk, u0[0], y0[0]);
      const float dx0 = ZOH ? fmaf(ds0[0], cr.Dk, lb0[0]) : fmaf(dt0[0], lb0[0], ds0[0] * cr.Dk);
      cr.dD = fmaf(ds1[0], u1[0], cr.dD);
      cr.dD = fmaf(ds0[0], u0[0], cr.dD);
      float dd1 = fmaf(u1[0], ZOH ? mb1[0] : lb1[0], wa1[0] * kInvLog2e);
      float dd0 = fmaf(u0[0], ZOH ? mb0[0] : lb0[0], wa0[0] * kInvLog2e);
      if constexpr (SP) {
        // the gradient goes to the pre-activation v: d softplus(v) / dv = sigmoid(v); the bias gets the sum over time
        if (softplus) {
          dd1 *= sigmoid_from_softplus(dt1[0]);
          dd0 *= sigmoid_from_softplus(dt0[0]);
        }
        if (r0 + 2 * m + 1 < nlive) cr.dbias += dd1;
        if (r0 + 2 * m < nlive) cr.dbias += dd0;
      }
      reinterpret_cast<__nv_bfloat16*>(tox + r1 * WPR)[lane] = __float2bfloat16_rn(dx1);
      reinterpret_cast<__nv_bfloat16*>(tod + r1 * WPR)[lane] = __float2bfloat16_rn(dd1);
      reinterpret_cast<__nv_bfloat16*>(toz + r1 * WPR)[lane] = __float2bfloat16_rn(dz1 * gate_on);
      reinterpret_cast<__nv_bfloat16*>(tox + r0e * WPR)[lane] = __float2bfloat16_rn(dx0);
      reinterpret_cast<__nv_bfloat16*>(tod + r0e * WPR)[lane] = __float2bfloat16_rn(dd0);
      reinterpret_cast<__nv_bfloat16*>(toz + r0e * WPR)[lane] = __float2bfloat16_rn(dz0 * gate_on);
    } else {
      // both lanes of the group complete the sums; lane 1 finishes the odd step of the pair, lane 0 the even one
      y0[0] += __shfl_xor_sync(0xffffffffu, y0[0], 1);
      lb0[0] += __shfl_xor_sync(0xffffffffu, lb0[0], 1);
      wa0[0] += __shfl_xor_sync(0xffffffffu, wa0[0], 1);
      wa1[0] += __shfl_xor_sync(0xffffffffu, wa1[0], 1);
      if constexpr (ZOH) mb0[0] += __shfl_xor_sync(0xffffffffu, mb0[0], 1);
      const bool odd = ln.j != 0;
      const float ym = odd ? y1[0] : y0[0], lbm = odd ? lb1[0] : lb0[0], wam = odd ? wa1[0] : wa0[0];
      const float um = odd ? u1[0] : u0[0], dtm = odd ? dt1[0] : dt0[0], dsm = odd ? ds1[0] : ds0[0];
      const float gpm = odd ? gp1 : gp0;
      const int rm = odd ? r1 : r0e;
      const float dzm = gpm * fmaf(cr.Dk, um, ym);
      const float dxm = ZOH ? fmaf(dsm, cr.Dk, lbm) : fmaf(dtm, lbm, dsm * cr.Dk);
      cr.dD = fmaf(dsm, um, cr.dD);
      float ddm = fmaf(um, ZOH ? (odd ? mb1[0] : mb0[0]) : lbm, wam * kInvLog2e);
      if constexpr (SP) {
        if (softplus) ddm *= sigmoid_from_softplus(dtm);
        if (r0 + 2 * m + (odd ? 1 : 0) < nlive) cr.dbias += ddm;
      }
      reinterpret_cast<__nv_bfloat16*>(tox + rm * WPR)[ln.co] = __float2bfloat16_rn(dxm);
      reinterpret_cast<__nv_bfloat16*>(tod + rm * WPR)[ln.co] = __float2bfloat16_rn(ddm);
      reinterpret_cast<__nv_bfloat16*>(toz + rm * WPR)[ln.co] = __float2bfloat16_rn(dzm * gate_on);
    }

    if (BC != 3 && (2 * m) % kRB == 0) {
      // dB / dC of steps 2m .. 2m + 3: every lane sums one float4 of one step over the lane groups, ascending
      // (a half that is a parameter has nothing in the buffer: its lanes idle)
      __syncwarp();
      const int s = lane >> 3, o = lane & 7;
      const int which = o >> 2, n0 = 4 * (o & 3);
      if (!(which ? SC : SB)) {
        const int jo = n0 / S, v = which * (S / 4) + (n0 % S) / 4;
        const float4* rs_ = tred + s * 32 * V;
        float4 acc;
#pragma unroll
        for (int gg = 0; gg < 32 / LPC; ++gg) {
          const int l = gg * LPC + jo;
          const float4 t4 = rs_[l * V + (v ^ ((l / (8 / V)) & (V - 1)))];
          if (gg == 0) acc = t4;
          else { acc.x += t4.x; acc.y += t4.y; acc.z += t4.z; acc.w += t4.w; }
        }
        const int row = r0 + 2 * m + s;
        if (row < nlive && SSM_IN_RANGE(row < kBT && n0 + 4 <= 16, abort_word))
          *reinterpret_cast<float4*>((which ? part_dC : part_dB) + (size_t)row * 16 + n0) = acc;
      }
      __syncwarp();
    }
  }
}

}  // namespace

// WHOLE: every tile and every channel group of the problem is whole (L and the segment length are multiples of the tile,
// D of the chain width), so the staging, the sub-blocks and the output copy carry no range tests
template <int S, int CPT, bool SP, bool ZOH, int BC, bool WHOLE = false>
__global__ void __launch_bounds__(kBwdWarps * 32, (CPT == 16 / S) ? 2 : 3)
    ssm_bwd_warp_kernel(const BwdParams p, const WarpSched sc) {
  constexpr bool SB = BC & 1, SC = BC & 2;
  constexpr int HV = bwd_handoff_vec(BC);
  using LN = Lane<S, CPT>;
  constexpr int H = S / 2, CW = LN::CW, WPR = CW / 2, NV = CPT * S / 4;   // NV: float4 of a thread's states
  constexpr bool OWN = LN::OWN;
  using Smem = BwdWarpSmem<S, CPT, SP>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  Smem& sm = reinterpret_cast<Smem*>(smem_raw)[warp];
  const LN ln(lane);
  const int j = ln.j, g = ln.g;
  const int D = p.D;
  const int worker = blockIdx.x * kBwdWarps + warp;
  const bool has_z = p.z != nullptr;

  const __nv_bfloat16* __restrict__ gx = static_cast<const __nv_bfloat16*>(p.x);
  const __nv_bfloat16* __restrict__ gd = static_cast<const __nv_bfloat16*>(p.delta);
  const __nv_bfloat16* __restrict__ gz = static_cast<const __nv_bfloat16*>(p.z);
  const __nv_bfloat16* __restrict__ gg = static_cast<const __nv_bfloat16*>(p.dout);
  const __nv_bfloat16* __restrict__ gB = static_cast<const __nv_bfloat16*>(p.B);
  const __nv_bfloat16* __restrict__ gC = static_cast<const __nv_bfloat16*>(p.C);
  __nv_bfloat16* __restrict__ gdx = static_cast<__nv_bfloat16*>(p.dx);
  __nv_bfloat16* __restrict__ gdd = static_cast<__nv_bfloat16*>(p.ddelta);
  __nv_bfloat16* __restrict__ gdz = static_cast<__nv_bfloat16*>(p.dz);

  const int groups = (D + CW - 1) / CW;
  const size_t bln = (size_t)p.batch * p.L * 16;
  const WorkList wl = make_worklist(sc, worker);
  for (int pi = 0; pi < wl.count; ++pi) {
    int chain, from, to;
    get_piece(wl, sc.tiles, pi, chain, from, to);
    const int grp = chain % groups;
    const int bs = chain / groups;
    const int seg = bs % p.nseg, b = bs / p.nseg;
    const int d_w = grp * CW;
    const int t_seg0 = seg * p.seg_steps;
    const int t_seg_end = min(p.L, t_seg0 + p.seg_steps);
    const int live_tiles = (t_seg_end - t_seg0 + kBT - 1) / kBT;
    // positions [from, to) of the chain in processing order are tiles tile_hi down to tile_lo (time runs backwards)
    const int tile_lo = sc.tiles - to;
    int tile_hi = sc.tiles - 1 - from;
    if (tile_hi > live_tiles - 1) tile_hi = live_tiles - 1;
    const bool gives_out = to < sc.tiles;

    // ---- staging: 16-byte chunks of the tile rows (CW / 8 per row of x, delta, z, dout; 2 per row of B, C)
    constexpr int CPR = CW / 8;                 // chunks per row
    constexpr int XCH = kBT * CPR;              // chunks per tensor and tile
    const int c_grp = d_w + g * CPT;            // first channel of this lane group
    const bool valid = WHOLE || c_grp < D;      // (CPT channels: all valid or none, D is a multiple of 8)
    auto chan = [&](int q) { return OWN ? c_grp + (j ^ q) : c_grp; };
    auto issue_tile = [&](int tile, int st) {
      if (tile >= tile_lo && tile >= 0) {
        const int t0 = t_seg0 + tile * kBT;
        const size_t row0 = (size_t)b * p.L + t0;
#pragma unroll
        for (int k = 0; k < (XCH + 31) / 32; ++k) {
          const int c = lane + 32 * k;
          if (XCH % 32 == 0 || c < XCH) {
            const int tt = c / CPR, cc = c % CPR;
            const bool ok = WHOLE || ((d_w + cc * 8 < D) && (t0 + tt < t_seg_end));
            const size_t go = ok ? (row0 + tt) * D + d_w + cc * 8 : 0;
            cp_async16(&sm.x[st][tt][cc * 4], gx + go, ok);
            cp_async16(&sm.d[st][tt][cc * 4], gd + go, ok);
            cp_async16(&sm.z[st][tt][cc * 4], (has_z ? gz : gx) + go, ok && has_z);
            cp_async16(&sm.g[st][tt][cc * 4], gg + go, ok);
          }
        }
        if (lane < kBT * 2) {
          const int tt = lane >> 1, hc = lane & 1;
          const bool ok = WHOLE || t0 + tt < t_seg_end;
          const size_t go = ok ? (row0 + tt) * 16 + hc * 8 : 0;
          if constexpr (!SB) cp_async16(&sm.rB[st][tt][hc * 4], gB + go, ok);
          if constexpr (!SC) cp_async16(&sm.rC[st][tt][hc * 4], gC + go, ok);
        }
#pragma unroll
        for (int sb = 0; sb < kBT / kSB; ++sb) {
          const bool ok = WHOLE || (valid && (t0 + sb * kSB < t_seg_end));
#pragma unroll
          for (int q = 0; q < CPT; ++q)
#pragma unroll
            for (int k = 0; k < S / 4; ++k) {
              const size_t go = ok ? ckpt_offset(1, b, p.nck, (t0 + sb * kSB) / kCkptSteps, D, 16, chan(q), S * j + 4 * k) : 0;
              cp_async16(&sm.ck[st][sb][q * (S / 4) + k][lane], p.ckpt + go, ok);
            }
        }
      }
      cp_async_commit();
    };
    issue_tile(tile_hi, 0);

    // ---- per-thread constants and carried values
    ChainRegs<S, CPT, ZOH, BC> cr;
    bool ap = !p.general_A;
    cr.minA = 3.0e38f;
#pragma unroll
    for (int q = 0; q < CPT; ++q) {
      float av[S];
#pragma unroll
      for (int k = 0; k < S / 4; ++k) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        if (valid) a = *reinterpret_cast<const float4*>(p.A + (size_t)chan(q) * 16 + S * j + 4 * k);
        av[4 * k] = a.x; av[4 * k + 1] = a.y; av[4 * k + 2] = a.z; av[4 * k + 3] = a.w;
      }
      const float step = av[1] - av[0];
      const float tol = 1e-6f * fabsf(av[S - 1]);
#pragma unroll
      for (int k = 2; k < S; ++k) ap = ap && fabsf(av[k] - (av[0] + (float)k * step)) <= tol;
      if (ZOH && valid) {
#pragma unroll
        for (int k = 0; k < S; ++k) cr.minA = fminf(cr.minA, fabsf(av[k]));
      }
#pragma unroll
      for (int k = 0; k < H; ++k) {
        cr.A2[q][k] = make_float2(av[2 * k] * kLog2e, av[2 * k + 1] * kLog2e);
        if constexpr (ZOH) {
          auto inv = [](float v) { return v != 0.f ? 1.f / v : 0.f; };
          cr.invA[q][k] = make_float2(inv(av[2 * k]), inv(av[2 * k + 1]));
        }
      }
      cr.a0s[q] = cr.A2[q][0].x;
      cr.rs[q] = cr.A2[q][0].y - cr.A2[q][0].x;
      if constexpr (SB || SC) {
#pragma unroll
        for (int k = 0; k < S / 4; ++k) {
          const size_t at = (size_t)chan(q) * 16 + S * j + 4 * k;
          if constexpr (SB) {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (valid) v = *reinterpret_cast<const float4*>(static_cast<const float*>(p.B) + at);
            cr.Bst[q][2 * k] = make_float2(v.x, v.y);
            cr.Bst[q][2 * k + 1] = make_float2(v.z, v.w);
            cr.dBs[q][2 * k] = cr.dBs[q][2 * k + 1] = make_float2(0.f, 0.f);
          }
          if constexpr (SC) {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (valid) v = *reinterpret_cast<const float4*>(static_cast<const float*>(p.C) + at);
            cr.Cst[q][2 * k] = make_float2(v.x, v.y);
            cr.Cst[q][2 * k + 1] = make_float2(v.z, v.w);
            cr.dCs[q][2 * k] = cr.dCs[q][2 * k + 1] = make_float2(0.f, 0.f);
          }
        }
      }
    }
    ap = __all_sync(0xffffffffu, ap);
    const int c_own = d_w + ln.co;
    cr.Dk = (p.Dskip != nullptr && c_own < D) ? p.Dskip[c_own] : 0.f;
    cr.dD = 0.f;
    cr.dbias = 0.f;
    if (from > 0) {
      if (!wait_handoff(sc, worker, lane)) {
        cp_async_wait_all();
        return;
      }
      const float4* hb = sc.handoff + ((size_t)worker * 32 + lane) * HV;
      float4 v[2 * NV];
#pragma unroll
      for (int k = 0; k < 2 * NV; ++k) v[k] = __ldcg(hb + k);
      const float4 dv = __ldcg(hb + 2 * NV);
      if constexpr (SB || SC) {
        // the gradient sums of the parameters B / C ride along like dA
#pragma unroll
        for (int q = 0; q < CPT; ++q)
#pragma unroll
          for (int k = 0; k < S / 4; ++k) {
            if constexpr (SB) {
              const float4 w = __ldcg(hb + 2 * NV + 1 + q * (S / 4) + k);
              cr.dBs[q][2 * k] = make_float2(w.x, w.y);
              cr.dBs[q][2 * k + 1] = make_float2(w.z, w.w);
            }
            if constexpr (SC) {
              const float4 w = __ldcg(hb + 2 * NV + 1 + (SB ? NV : 0) + q * (S / 4) + k);
              cr.dCs[q][2 * k] = make_float2(w.x, w.y);
              cr.dCs[q][2 * k + 1] = make_float2(w.z, w.w);
            }
          }
      }
      const float* f = reinterpret_cast<const float*>(v);
#pragma unroll
      for (int q = 0; q < CPT; ++q)
#pragma unroll
        for (int k = 0; k < H; ++k) {
          cr.mu[q][k] = make_float2(f[(q * H + k) * 2], f[(q * H + k) * 2 + 1]);
          cr.dA[q][k] = make_float2(f[4 * NV + (q * H + k) * 2], f[4 * NV + (q * H + k) * 2 + 1]);
        }
      cr.dD = dv.x;
      cr.dbias = dv.y;
    } else {
#pragma unroll
      for (int q = 0; q < CPT; ++q)
#pragma unroll
        for (int k = 0; k < S / 4; ++k) {
          float4 m4 = make_float4(0.f, 0.f, 0.f, 0.f);
          if (valid && p.mu_in != nullptr)
            m4 = *reinterpret_cast<const float4*>(p.mu_in + (((size_t)b * p.nseg + seg) * D + chan(q)) * 16 + S * j + 4 * k);
          cr.mu[q][2 * k] = make_float2(m4.x, m4.y);
          cr.mu[q][2 * k + 1] = make_float2(m4.z, m4.w);
          cr.dA[q][2 * k] = cr.dA[q][2 * k + 1] = make_float2(0.f, 0.f);
        }
    }

    // The sweep over the tiles exists once per kind of A (arithmetic progression or general), chosen once per chain, so
    // that neither body carries the registers of the other.
    auto sweep = [&](auto ap_tag) {
    constexpr bool AP_ = decltype(ap_tag)::value;
    int st = 0;
    for (int tile = tile_hi; tile >= tile_lo; --tile, st ^= 1) {
      cp_async_wait_all();
      __syncwarp();                   // this tile landed for all lanes; all lanes are done with the previous one
      issue_tile(tile - 1, st ^ 1);   // prefetch the tile before in time
      const int t0 = t_seg0 + tile * kBT;
      const int nlive = WHOLE ? kBT : min(kBT, t_seg_end - t0);
      {
        // B and C of the tile to float: lane -> (row lane / 4, states 4 (lane % 4) ..)
#pragma unroll
        for (int k = 0; k < (kBT * 4 + 31) / 32; ++k) {
          const int c = lane + 32 * k, rr = c >> 2, qq = c & 3;
          if (kBT * 4 % 32 == 0 || rr < kBT) {
            if constexpr (!SB) {
              const uint2 wb = *reinterpret_cast<const uint2*>(&sm.rB[st][rr][2 * qq]);
              *reinterpret_cast<float4*>(&sm.fB[rr][4 * qq]) = make_float4(bf16lo(wb.x), bf16hi(wb.x), bf16lo(wb.y), bf16hi(wb.y));
            }
            if constexpr (!SC) {
              const uint2 wc = *reinterpret_cast<const uint2*>(&sm.rC[st][rr][2 * qq]);
              *reinterpret_cast<float4*>(&sm.fC[rr][4 * qq]) = make_float4(bf16lo(wc.x), bf16hi(wc.x), bf16lo(wc.y), bf16hi(wc.y));
            }
          }
        }
        // per-element gate terms of the tile: ds = dout silu(z), gp = dout silu'(z); element e = lane + 32 i
        constexpr int EPL = kBT * CW / 32;   // elements per lane
        float zf[EPL], gf[EPL], df[SP ? EPL : 1];
#pragma unroll
        for (int i = 0; i < EPL; ++i) {
          const int e = lane + 32 * i, r = e / CW, c = e % CW;
          zf[i] = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(sm.z[st][r])[c] << 16);
          gf[i] = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(sm.g[st][r])[c] << 16);
          if constexpr (SP) df[i] = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(sm.d[st][r])[c] << 16);
        }
        // (with 32 channels per warp an element's channel is this lane's own; with 16 it is lane % 16)
        const int c_el = d_w + lane % CW;
        const float bias_el = (SP && p.delta_bias != nullptr && c_el < D) ? p.delta_bias[c_el] : 0.f;
#pragma unroll
        for (int i = 0; i < EPL; ++i) {
          const int e = lane + 32 * i, r = e / CW, c = e % CW;
          float dsv = gf[i], gpv = 0.f;
          if (has_z) {
            const float sg = sigmoid_fast(zf[i]);
            dsv = gf[i] * zf[i] * sg;
            gpv = gf[i] * sg * fmaf(zf[i], 1.f - sg, 1.f);
          }
          sm.ds[r][c] = dsv;
          sm.gp[r][c] = gpv;
          if constexpr (SP) {
            float v = df[i] + bias_el;
            if (p.softplus) v = softplus_fast(v);
            sm.dF[r][c] = r < nlive ? v : 0.f;   // rows past the end stay identity steps
          }
        }
      }
      __syncwarp();
      const size_t row0 = (size_t)b * p.L + t0;
      float* part_dB = p.dBC_part + ((size_t)grp * 2 + 0) * bln + row0 * 16;
      float* part_dC = p.dBC_part + ((size_t)grp * 2 + 1) * bln + row0 * 16;
#pragma unroll 1
      for (int sb = kBT / kSB - 1; sb >= 0; --sb) {
        if (sb * kSB >= nlive) continue;   // a sub-block of identity steps
        bool zs = false;
        if constexpr (ZOH) {
          // smallest step size of the live rows of the sub-block among this thread's channels
          float dmin = 3.0e38f;
          for (int t = 0; t < kSB && sb * kSB + t < nlive; ++t) {
            float dv[CPT];
            if constexpr (SP) ln.pick_row(&sm.dF[0][0] + (sb * kSB + t) * LN::CW, dv);
            else ln.unpack_row(&sm.d[st][0][0] + (sb * kSB + t) * (LN::CW / 2), dv);
#pragma unroll
            for (int q = 0; q < CPT; ++q) dmin = fminf(dmin, fabsf(dv[q]));
          }
          zs = __any_sync(0xffffffffu, dmin * cr.minA < kZohSmall);
        }
#define SSM_SUB_BLOCK(ZS_)                                                                                          \
  sub_block<S, CPT, SP, AP_, ZOH, ZS_, BC>(ln, cr, sb * kSB, nlive, has_z ? 1.f : 0.f, p.softplus != 0, &sm.x[st][0][0], \
                                       &sm.d[st][0][0], &sm.fB[0][0], &sm.fC[0][0], &sm.ds[0][0], &sm.gp[0][0],      \
                                       &sm.dF[0][0], &sm.ck[st][sb][0][0], &sm.ox[0][0], &sm.od[0][0], &sm.oz[0][0], \
                                       &sm.red[0][0][0], part_dB, part_dC, sc.abort)
        if constexpr (ZOH) {
          if (zs) SSM_SUB_BLOCK(true);
          else SSM_SUB_BLOCK(false);
        } else {
          SSM_SUB_BLOCK(false);
        }
#undef SSM_SUB_BLOCK
      }
      __syncwarp();
      // ---- results of the tile: 16-byte stores of dx, ddelta, dz
#pragma unroll
      for (int k = 0; k < (XCH + 31) / 32; ++k) {
        const int c = lane + 32 * k;
        const int tt = c / CPR, cc = c % CPR;
        if ((XCH % 32 == 0 || c < XCH) && (WHOLE || (d_w + cc * 8 < D && tt < nlive)) &&
            SSM_IN_RANGE(row0 + tt < (size_t)p.batch * p.L && d_w + cc * 8 + 8 <= D, sc.abort)) {
          const size_t go = (row0 + tt) * D + d_w + cc * 8;
          *reinterpret_cast<uint4*>(gdx + go) = *reinterpret_cast<const uint4*>(&sm.ox[tt][cc * 4]);
          *reinterpret_cast<uint4*>(gdd + go) = *reinterpret_cast<const uint4*>(&sm.od[tt][cc * 4]);
          if (gdz != nullptr) *reinterpret_cast<uint4*>(gdz + go) = *reinterpret_cast<const uint4*>(&sm.oz[tt][cc * 4]);
        }
      }
    }
    };
    if (ap) sweep(std::true_type{});
    else sweep(std::false_type{});
    cp_async_wait_all();
    __syncwarp();

    if (gives_out) {
      // the earlier part of this chain (in time) belongs to the next worker
      float4* hb = sc.handoff + ((size_t)(worker + 1) * 32 + lane) * HV;
      if constexpr (SB || SC) {
#pragma unroll
        for (int q = 0; q < CPT; ++q)
#pragma unroll
          for (int k = 0; k < S / 4; ++k) {
            if constexpr (SB)
              __stcg(hb + 2 * NV + 1 + q * (S / 4) + k, make_float4(cr.dBs[q][2 * k].x, cr.dBs[q][2 * k].y,
                                                                    cr.dBs[q][2 * k + 1].x, cr.dBs[q][2 * k + 1].y));
            if constexpr (SC)
              __stcg(hb + 2 * NV + 1 + (SB ? NV : 0) + q * (S / 4) + k,
                     make_float4(cr.dCs[q][2 * k].x, cr.dCs[q][2 * k].y, cr.dCs[q][2 * k + 1].x, cr.dCs[q][2 * k + 1].y));
          }
      }
      float f[8 * NV];
#pragma unroll
      for (int q = 0; q < CPT; ++q)
#pragma unroll
        for (int k = 0; k < H; ++k) {
          f[(q * H + k) * 2] = cr.mu[q][k].x;
          f[(q * H + k) * 2 + 1] = cr.mu[q][k].y;
          f[4 * NV + (q * H + k) * 2] = cr.dA[q][k].x;
          f[4 * NV + (q * H + k) * 2 + 1] = cr.dA[q][k].y;
        }
#pragma unroll
      for (int k = 0; k < 2 * NV; ++k) __stcg(hb + k, make_float4(f[4 * k], f[4 * k + 1], f[4 * k + 2], f[4 * k + 3]));
      __stcg(hb + 2 * NV, make_float4(cr.dD, cr.dbias, 0.f, 0.f));
      publish_handoff(sc, worker, lane);
    } else {
      // first step in time done: the chain is complete
      float dD_tot = cr.dD, dbias_tot = cr.dbias;
      if constexpr (!OWN) {   // the two lanes of a group summed the steps of one parity each
        dD_tot += __shfl_xor_sync(0xffffffffu, dD_tot, 1);
        dbias_tot += __shfl_xor_sync(0xffffffffu, dbias_tot, 1);
      }
      if (valid) {
        const size_t part = (size_t)b * p.nseg + seg;
#pragma unroll
        for (int q = 0; q < CPT; ++q)
#pragma unroll
          for (int k = 0; k < S / 4; ++k) {
            *reinterpret_cast<float4*>(p.dA_part + (part * D + chan(q)) * 16 + S * j + 4 * k) =
                make_float4(cr.dA[q][2 * k].x, cr.dA[q][2 * k].y, cr.dA[q][2 * k + 1].x, cr.dA[q][2 * k + 1].y);
            if constexpr (SB)
              *reinterpret_cast<float4*>(p.dBs_part + (part * D + chan(q)) * 16 + S * j + 4 * k) =
                  make_float4(cr.dBs[q][2 * k].x, cr.dBs[q][2 * k].y, cr.dBs[q][2 * k + 1].x, cr.dBs[q][2 * k + 1].y);
            if constexpr (SC)
              *reinterpret_cast<float4*>(p.dCs_part + (part * D + chan(q)) * 16 + S * j + 4 * k) =
                  make_float4(cr.dCs[q][2 * k].x, cr.dCs[q][2 * k].y, cr.dCs[q][2 * k + 1].x, cr.dCs[q][2 * k + 1].y);
            if (seg == 0 && p.dh0 != nullptr)   // the adjoint that leaves the first step is the gradient of the initial state
              *reinterpret_cast<float4*>(p.dh0 + ((size_t)b * D + chan(q)) * 16 + S * j + 4 * k) =
                  make_float4(cr.mu[q][2 * k].x, cr.mu[q][2 * k].y, cr.mu[q][2 * k + 1].x, cr.mu[q][2 * k + 1].y);
          }
        if (OWN || j == 0) {
          p.dD_part[part * D + c_own] = dD_tot;
          if (SP && p.dbias_part != nullptr) p.dbias_part[part * D + c_own] = dbias_tot;
        }
      }
    }
  }
}

namespace {

template <int S, int CPT, bool SP, bool ZOH, int BC = 0>
cudaError_t launch_bwd_variant(const Plan& plan, const BwdParams& p, cudaStream_t s) {
  constexpr int CW = Lane<S, CPT>::CW;
  const size_t smem = sizeof(BwdWarpSmem<S, CPT, SP>) * kBwdWarps;
  auto kern = ssm_bwd_warp_kernel<S, CPT, SP, ZOH, BC>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 0, per_sm = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kBwdWarps * 32, smem)) != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  WarpSched sc{};
  sc.chains = p.batch * plan.nseg * ((p.D + CW - 1) / CW);
  sc.tiles = (plan.seg_steps + kBT - 1) / kBT;
  const bool can_share = p.abort != nullptr && p.flags != nullptr && p.handoff != nullptr && p.max_workers > 0;
  sc.workers = warp_workers(sc.chains, sms, per_sm * kBwdWarps, can_share ? p.max_workers : 0);
  if (p.test_withhold && can_share) {
    // test hook: make neighbouring workers share chains whatever the shape (all of them must be resident)
    sc.workers = p.max_workers < per_sm * kBwdWarps * sms ? p.max_workers : per_sm * kBwdWarps * sms;
  }
  const long long total = (long long)sc.chains * sc.tiles;
  sc.quota = (int)((total + sc.workers - 1) / sc.workers);
  sc.spin_limit = p.test_withhold ? 1000 : (1 << 22);
  sc.withhold = p.test_withhold;
  sc.flags = p.flags;
  sc.abort = p.abort;
  sc.handoff = p.handoff;
  const unsigned grid = (unsigned)((sc.workers + kBwdWarps - 1) / kBwdWarps);
  {
    // no ragged tile or channel group anywhere: the instantiation without range tests (same launch shape)
    if (p.L % kBT == 0 && plan.seg_steps % kBT == 0 && p.D % CW == 0) {
      auto whole = ssm_bwd_warp_kernel<S, CPT, SP, ZOH, BC, true>;
      if ((e = cudaFuncSetAttribute(whole, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
      whole<<<grid, kBwdWarps * 32, smem, s>>>(p, sc);
      return cudaGetLastError();
    }
  }
  kern<<<grid, kBwdWarps * 32, smem, s>>>(p, sc);
  return cudaGetLastError();
}

}  // namespace

bool bwd_fast_applicable(const ssm_problem_t& prob, const BwdParams& p) {
  auto al16 = [](const void* q) { return q == nullptr || (reinterpret_cast<uintptr_t>(q) & 15) == 0; };
  if ((p.static_B || p.static_C) && p.zoh) return false;  // non-selective B / C: default B-bar rule only
  if ((p.static_B && !al16(p.dBs_part)) || (p.static_C && !al16(p.dCs_part))) return false;
  return prob.io_dtype == SSM_BF16 && prob.N == 16 && prob.D % 8 == 0 && p.seg_steps % kBT == 0 && al16(p.x) &&
         al16(p.delta) && al16(p.z) && al16(p.B) && al16(p.C) && al16(p.dout) && al16(p.dx) && al16(p.ddelta) &&
         al16(p.dz) && al16(p.A) && al16(p.ckpt) && al16(p.mu_in) && al16(p.dh0) && al16(p.dBC_part) && al16(p.dA_part) &&
         al16(p.handoff) && (p.groups == (p.D + 31) / 32 || p.groups == (p.D + 15) / 16);
}

size_t bwd_handoff_bytes_per_worker(bool static_B, bool static_C) {
  return sizeof(float4) * bwd_handoff_vec((static_B ? 1 : 0) | (static_C ? 2 : 0)) * 32;
}
// channels per warp of the tuned kernel = the channel-group size of the dB / dC partial sums
int bwd_fast_channels_per_warp() { return kBwdFastChannels; }

cudaError_t launch_bwd_fast(const Plan& plan, const BwdParams& p, cudaStream_t s) {
  const bool sp = p.softplus || p.delta_bias != nullptr;
  if (p.static_B || p.static_C) {   // (never with ZOH: bwd_fast_applicable)
    const int bc = (p.static_B ? 1 : 0) | (p.static_C ? 2 : 0);
    if (bc == 3) return sp ? launch_bwd_variant<8, 2, true, false, 3>(plan, p, s) : launch_bwd_variant<8, 2, false, false, 3>(plan, p, s);
    if (bc == 1) return sp ? launch_bwd_variant<8, 2, true, false, 1>(plan, p, s) : launch_bwd_variant<8, 2, false, false, 1>(plan, p, s);
    return sp ? launch_bwd_variant<8, 2, true, false, 2>(plan, p, s) : launch_bwd_variant<8, 2, false, false, 2>(plan, p, s);
  }
  if (p.zoh) return sp ? launch_bwd_variant<8, 2, true, true>(plan, p, s) : launch_bwd_variant<8, 2, false, true>(plan, p, s);
  return sp ? launch_bwd_variant<8, 2, true, false>(plan, p, s) : launch_bwd_variant<8, 2, false, false>(plan, p, s);
}

}  // namespace ssm
