// Forward + backward of a batch that lives in HOST memory (the paper has no counterpart: its kernels start from
// tensors already in HBM).  One call copies the inputs to the device, runs ssm_scan_fwd (saving checkpoint states)
// and ssm_scan_bwd, and copies every result back.
//
// The batch entries of the selective scan are independent (Section 2, "Structure and Dimensions"), so the call cuts
// the batch into up to kMaxChunks pieces and pipelines them over three streams: while piece c is computed on the
// caller's stream, piece c+1 is on its way in on a copy-in stream and piece c-1 on its way out on a copy-out stream;
// PCIe is full duplex, so the three overlap.  Device buffers are double-buffered per direction and come from an arena
// the caller provides; events order the reuse of a buffer.  dA and dD are sums over the batch: every piece leaves its
// own partial sum and a last kernel adds the pieces in ascending order (fixed order, no atomics).
//
// The two helper streams are created once per device and kept; events are created per call.  Every copy is a plain
// cudaMemcpyAsync (one per tensor and piece).  With pageable host memory the copies still work but do not overlap.
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>
#include <vector>

#include "ssm_scan.h"

namespace {

constexpr int kMaxChunks = 8;
constexpr int kMaxDevices = 64;

std::mutex g_stream_mutex;
cudaStream_t g_in_stream[kMaxDevices] = {};
cudaStream_t g_out_stream[kMaxDevices] = {};
bool g_streams_ready[kMaxDevices] = {};

cudaError_t helper_streams(cudaStream_t* in, cudaStream_t* out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_stream_mutex);
  if (!g_streams_ready[dev]) {
    if ((e = cudaStreamCreateWithFlags(&g_in_stream[dev], cudaStreamNonBlocking)) != cudaSuccess) return e;
    if ((e = cudaStreamCreateWithFlags(&g_out_stream[dev], cudaStreamNonBlocking)) != cudaSuccess) return e;
    g_streams_ready[dev] = true;
  }
  *in = g_in_stream[dev];
  *out = g_out_stream[dev];
  return cudaSuccess;
}

inline size_t align_up(size_t v) { return (v + 255) & ~(size_t)255; }

struct HostPlan {
  int nchunks, chunk_batch;          // pieces and batch entries per piece (the last piece may be smaller)
  ssm_problem_t chunk;               // the problem of a full piece
  size_t e;                          // bytes per io element
  size_t bld, bln;                   // bytes of one (chunk_batch, L, D) / (chunk_batch, L, N) tensor
  // arena offsets
  size_t in[2], out[2];              // double-buffered piece inputs (x, delta, z, dout, B, C) and outputs
  size_t A, Dskip, dA_part, dD_part, dA, dD, saved, ws;
  size_t ws_bytes, total;
};

bool make_host_plan(const ssm_problem_t* p, HostPlan* hp) {
  if (p == nullptr || p->batch < 1 || p->L < 1 || p->D < 1 || p->N < 1) return false;
  if (p->io_dtype != SSM_F32 && p->io_dtype != SSM_BF16) return false;
  HostPlan h{};
  h.nchunks = std::min<int>(p->batch, kMaxChunks);
  h.chunk_batch = (p->batch + h.nchunks - 1) / h.nchunks;
  h.nchunks = (p->batch + h.chunk_batch - 1) / h.chunk_batch;
  h.chunk = *p;
  h.chunk.batch = h.chunk_batch;
  h.chunk.flags = (p->flags & (SSM_FLAG_HAS_Z | SSM_FLAG_HAS_DSKIP | SSM_FLAG_GENERAL_A | SSM_FLAG_ZOH_BBAR)) |
                  SSM_FLAG_SAVE_STATES;
  h.e = p->io_dtype == SSM_BF16 ? 2 : 4;
  h.bld = align_up((size_t)h.chunk_batch * p->L * p->D * h.e);
  h.bln = align_up((size_t)h.chunk_batch * p->L * p->N * h.e);
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off += align_up(bytes);
    return at;
  };
  for (int b = 0; b < 2; ++b) h.in[b] = take(4 * h.bld + 2 * h.bln);
  for (int b = 0; b < 2; ++b) h.out[b] = take(4 * h.bld + 2 * h.bln);
  h.A = take((size_t)p->D * p->N * 4);
  h.Dskip = take((size_t)p->D * 4);
  h.dA_part = take((size_t)h.nchunks * p->D * p->N * 4);
  h.dD_part = take((size_t)h.nchunks * p->D * 4);
  h.dA = take((size_t)p->D * p->N * 4);
  h.dD = take((size_t)p->D * 4);
  h.saved = take(ssm_scan_saved_state_bytes(&h.chunk));
  h.ws_bytes = std::max(ssm_scan_fwd_workspace_bytes(&h.chunk), ssm_scan_bwd_workspace_bytes(&h.chunk));
  h.ws = take(h.ws_bytes);
  h.total = off;
  *hp = h;
  return true;
}

// out[i] = sum over pieces of part[c][i], ascending c
__global__ void sum_pieces_kernel(const float* __restrict__ part, int pieces, int n, float* __restrict__ out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float s = 0.f;
  for (int c = 0; c < pieces; ++c) s += part[(size_t)c * n + i];
  out[i] = s;
}

}  // namespace

extern "C" SSM_API size_t ssm_scan_host_arena_bytes(const ssm_problem_t* p) {
  HostPlan h;
  return make_host_plan(p, &h) ? h.total : 0;
}

extern "C" ssm_status_t ssm_scan_fwd_bwd_host(const ssm_problem_t* p, const void* x, const void* delta, const float* A,
                                              const void* B, const void* C, const float* D_skip, const void* z,
                                              const void* dout, void* out, void* dx, void* ddelta, float* dA, void* dB,
                                              void* dC, float* dD, void* dz, void* device_arena, size_t arena_bytes,
                                              void* stream) {
  HostPlan h;
  if (!make_host_plan(p, &h)) return SSM_ERR_INVALID_ARG;
  if (p->flags & SSM_FLAG_COMPLEX) return SSM_ERR_UNSUPPORTED;   // this entry point moves real-state buffers only
  const bool has_z = p->flags & SSM_FLAG_HAS_Z, has_d = p->flags & SSM_FLAG_HAS_DSKIP;
  if (!x || !delta || !A || !B || !C || !dout || !out || !dx || !ddelta || !dA || !dB || !dC) return SSM_ERR_INVALID_ARG;
  if ((has_z && (!z || !dz)) || (has_d && (!D_skip || !dD))) return SSM_ERR_INVALID_ARG;
  if (device_arena == nullptr || (reinterpret_cast<uintptr_t>(device_arena) & 255) != 0 || arena_bytes < h.total)
    return SSM_ERR_WORKSPACE;

  cudaStream_t s_run = static_cast<cudaStream_t>(stream), s_in = nullptr, s_out = nullptr;
  if (helper_streams(&s_in, &s_out) != cudaSuccess) return SSM_ERR_CUDA;
  char* arena = static_cast<char*>(device_arena);
  const size_t e = h.e;
  const size_t row_d = (size_t)p->L * p->D * e, row_n = (size_t)p->L * p->N * e;   // bytes of one batch entry

  // events: [0] entry, then per piece: inputs landed, computed, results drained
  std::vector<cudaEvent_t> ev(1 + 3 * (size_t)h.nchunks, nullptr);
  bool ok = true;
  for (auto& q : ev) ok = ok && cudaEventCreateWithFlags(&q, cudaEventDisableTiming) == cudaSuccess;
  auto landed = [&](int c) { return ev[1 + 3 * c]; };
  auto computed = [&](int c) { return ev[2 + 3 * c]; };
  auto drained = [&](int c) { return ev[3 + 3 * c]; };
  auto CK = [&](cudaError_t err) { ok = ok && err == cudaSuccess; };
  ssm_status_t status = SSM_OK;

  if (ok) {
    // everything the caller enqueued on `stream` before this call comes first
    CK(cudaEventRecord(ev[0], s_run));
    CK(cudaStreamWaitEvent(s_in, ev[0], 0));
    CK(cudaStreamWaitEvent(s_out, ev[0], 0));
    CK(cudaMemcpyAsync(arena + h.A, A, (size_t)p->D * p->N * 4, cudaMemcpyHostToDevice, s_in));
    if (has_d) CK(cudaMemcpyAsync(arena + h.Dskip, D_skip, (size_t)p->D * 4, cudaMemcpyHostToDevice, s_in));
  }
  for (int c = 0; ok && c < h.nchunks; ++c) {
    const int b0 = c * h.chunk_batch;
    const int nb = std::min(h.chunk_batch, p->batch - b0);
    ssm_problem_t cp = h.chunk;
    cp.batch = nb;
    char* in = arena + h.in[c & 1];
    char* ot = arena + h.out[c & 1];
    char *d_x = in, *d_dl = in + h.bld, *d_z = in + 2 * h.bld, *d_g = in + 3 * h.bld, *d_B = in + 4 * h.bld,
         *d_C = in + 4 * h.bld + h.bln;
    char *d_out = ot, *d_dx = ot + h.bld, *d_dd = ot + 2 * h.bld, *d_dz = ot + 3 * h.bld, *d_dB = ot + 4 * h.bld,
         *d_dC = ot + 4 * h.bld + h.bln;
    const size_t nd = (size_t)nb * row_d, nn = (size_t)nb * row_n, od = (size_t)b0 * row_d, on = (size_t)b0 * row_n;

    // ---- copy in: the input buffer is free once the piece that used it two pieces ago has been computed
    if (c >= 2) CK(cudaStreamWaitEvent(s_in, computed(c - 2), 0));
    CK(cudaMemcpyAsync(d_x, static_cast<const char*>(x) + od, nd, cudaMemcpyHostToDevice, s_in));
    CK(cudaMemcpyAsync(d_dl, static_cast<const char*>(delta) + od, nd, cudaMemcpyHostToDevice, s_in));
    if (has_z) CK(cudaMemcpyAsync(d_z, static_cast<const char*>(z) + od, nd, cudaMemcpyHostToDevice, s_in));
    CK(cudaMemcpyAsync(d_g, static_cast<const char*>(dout) + od, nd, cudaMemcpyHostToDevice, s_in));
    CK(cudaMemcpyAsync(d_B, static_cast<const char*>(B) + on, nn, cudaMemcpyHostToDevice, s_in));
    CK(cudaMemcpyAsync(d_C, static_cast<const char*>(C) + on, nn, cudaMemcpyHostToDevice, s_in));
    CK(cudaEventRecord(landed(c), s_in));

    // ---- compute: needs the inputs, and the output buffer drained by the piece that used it two pieces ago
    CK(cudaStreamWaitEvent(s_run, landed(c), 0));
    if (c >= 2) CK(cudaStreamWaitEvent(s_run, drained(c - 2), 0));
    if (!ok) break;
    const float* A_d = reinterpret_cast<const float*>(arena + h.A);
    const float* dk_d = has_d ? reinterpret_cast<const float*>(arena + h.Dskip) : nullptr;
    status = ssm_scan_fwd(&cp, d_x, d_dl, A_d, d_B, d_C, dk_d, has_z ? d_z : nullptr, d_out, arena + h.saved,
                          arena + h.ws, h.ws_bytes, s_run);
    if (status != SSM_OK) break;
    cp.flags &= ~(uint32_t)SSM_FLAG_SAVE_STATES;
    status = ssm_scan_bwd(&cp, d_x, d_dl, A_d, d_B, d_C, dk_d, has_z ? d_z : nullptr, d_g, arena + h.saved, d_dx, d_dd,
                          reinterpret_cast<float*>(arena + h.dA_part) + (size_t)c * p->D * p->N, d_dB, d_dC,
                          has_d ? reinterpret_cast<float*>(arena + h.dD_part) + (size_t)c * p->D : nullptr,
                          has_z ? d_dz : nullptr, arena + h.ws, h.ws_bytes, s_run);
    if (status != SSM_OK) break;
    CK(cudaEventRecord(computed(c), s_run));

    // ---- copy out
    CK(cudaStreamWaitEvent(s_out, computed(c), 0));
    CK(cudaMemcpyAsync(static_cast<char*>(out) + od, d_out, nd, cudaMemcpyDeviceToHost, s_out));
    CK(cudaMemcpyAsync(static_cast<char*>(dx) + od, d_dx, nd, cudaMemcpyDeviceToHost, s_out));
    CK(cudaMemcpyAsync(static_cast<char*>(ddelta) + od, d_dd, nd, cudaMemcpyDeviceToHost, s_out));
    if (has_z) CK(cudaMemcpyAsync(static_cast<char*>(dz) + od, d_dz, nd, cudaMemcpyDeviceToHost, s_out));
    CK(cudaMemcpyAsync(static_cast<char*>(dB) + on, d_dB, nn, cudaMemcpyDeviceToHost, s_out));
    CK(cudaMemcpyAsync(static_cast<char*>(dC) + on, d_dC, nn, cudaMemcpyDeviceToHost, s_out));
    CK(cudaEventRecord(drained(c), s_out));
  }
  if (ok && status == SSM_OK) {
    // dA, dD: pieces added in ascending order, then home; the caller's stream ends after every copy-out
    const int n_a = p->D * p->N;
    sum_pieces_kernel<<<(n_a + 255) / 256, 256, 0, s_run>>>(reinterpret_cast<const float*>(arena + h.dA_part), h.nchunks,
                                                            n_a, reinterpret_cast<float*>(arena + h.dA));
    CK(cudaGetLastError());
    CK(cudaMemcpyAsync(dA, arena + h.dA, (size_t)n_a * 4, cudaMemcpyDeviceToHost, s_run));
    if (has_d) {
      sum_pieces_kernel<<<(p->D + 255) / 256, 256, 0, s_run>>>(reinterpret_cast<const float*>(arena + h.dD_part),
                                                              h.nchunks, p->D, reinterpret_cast<float*>(arena + h.dD));
      CK(cudaGetLastError());
      CK(cudaMemcpyAsync(dD, arena + h.dD, (size_t)p->D * 4, cudaMemcpyDeviceToHost, s_run));
    }
  }
  // whatever happened, the caller's stream must not run ahead of work this call put on the helper streams
  if (ev[0] != nullptr) {
    cudaEvent_t tail_in = nullptr, tail_out = nullptr;
    if (cudaEventCreateWithFlags(&tail_in, cudaEventDisableTiming) == cudaSuccess &&
        cudaEventCreateWithFlags(&tail_out, cudaEventDisableTiming) == cudaSuccess) {
      cudaEventRecord(tail_in, s_in);
      cudaEventRecord(tail_out, s_out);
      cudaStreamWaitEvent(s_run, tail_in, 0);
      cudaStreamWaitEvent(s_run, tail_out, 0);
    } else {
      cudaStreamSynchronize(s_in);
      cudaStreamSynchronize(s_out);
    }
    if (tail_in) cudaEventDestroy(tail_in);
    if (tail_out) cudaEventDestroy(tail_out);
  }
  for (auto q : ev)
    if (q != nullptr) cudaEventDestroy(q);   // released by the runtime once the recorded work has completed
  if (status != SSM_OK) return status;
  return ok ? SSM_OK : SSM_ERR_CUDA;
}
