// Widening / narrowing of the state dimension, so that bf16 problems with fewer than 16 states per channel
// (Table 10 sweeps N = 1 ... 16) run on the tuned 16-state kernels: B and C get zero columns for the added states, so
// those states stay exactly zero (h = a h + delta B x with B = 0 from h = 0) and contribute nothing to the readout
// (C = 0) or to any gradient of the real inputs; their own gradient columns are dropped again on the way out.
//
// One kernel copies up to kRepackMax row-major arrays [rows][n_src] -> [rows][n_dst]: column j of the destination is
// column j of the source where j < n_src, else a fill value.  Narrowing (n_dst < n_src) is the same copy.
// The fill for A continues the arithmetic progression of the row's values (A_n = A_0 + n step, which keeps the
// two-exponential path of the tuned kernels) as long as the continued values stay <= 0, so that exp(delta A) cannot
// overflow in a state that only ever holds zero; otherwise it repeats the last value of the row.
#include <algorithm>

#include "ssm_common.cuh"

namespace ssm {

enum { kRepackBf16 = 0, kRepackF32 = 1, kRepackA = 2 };
constexpr int kRepackMax = 6;

struct RepackJob {
  const void* src;
  void* dst;
  int rows, n_src, n_dst, kind;
};
struct RepackJobs {
  RepackJob job[kRepackMax];
  int count;
};

namespace {

__global__ void __launch_bounds__(256) ssm_repack_kernel(const RepackJobs jobs) {
  const RepackJob jb = jobs.job[blockIdx.y];
  const long long total = (long long)jb.rows * jb.n_dst;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / jb.n_dst;
    const int j = (int)(i % jb.n_dst);
    if (jb.kind == kRepackBf16) {
      const __nv_bfloat16* s = static_cast<const __nv_bfloat16*>(jb.src);
      static_cast<__nv_bfloat16*>(jb.dst)[i] = j < jb.n_src ? s[r * jb.n_src + j] : __float2bfloat16(0.f);
    } else if (jb.kind == kRepackF32) {
      const float* s = static_cast<const float*>(jb.src);
      static_cast<float*>(jb.dst)[i] = j < jb.n_src ? s[r * jb.n_src + j] : 0.f;
    } else {
      const float* s = static_cast<const float*>(jb.src) + r * jb.n_src;
      float v;
      if (j < jb.n_src) {
        v = s[j];
      } else {
        const float a0 = s[0], last = s[jb.n_src - 1];
        const float step = jb.n_src >= 2 ? s[1] - s[0] : 0.f;
        bool ap = true;
        const float tol = 1e-6f * fabsf(last);
        for (int k = 2; k < jb.n_src; ++k) ap = ap && fabsf(s[k] - (a0 + (float)k * step)) <= tol;
        const float far = a0 + (float)(jb.n_dst - 1) * step;   // the progression is monotone: its ends bound it
        ap = ap && a0 <= 0.f && far <= 0.f && isfinite(far);
        v = ap ? a0 + (float)j * step : last;
      }
      static_cast<float*>(jb.dst)[i] = v;
    }
  }
}

}  // namespace

void repack_add(RepackJobs& jobs, const void* src, void* dst, long long rows, int n_src, int n_dst, int kind) {
  if (src == nullptr || dst == nullptr || jobs.count >= kRepackMax) return;
  jobs.job[jobs.count++] = RepackJob{src, dst, (int)rows, n_src, n_dst, kind};
}

cudaError_t repack_run(const RepackJobs& jobs, cudaStream_t s) {
  if (jobs.count == 0) return cudaSuccess;
  long long most = 1;
  for (int i = 0; i < jobs.count; ++i) most = std::max(most, (long long)jobs.job[i].rows * jobs.job[i].n_dst);
  const unsigned gx = (unsigned)std::min<long long>((most + 255) / 256, 4LL * kNumSMs);
  ssm_repack_kernel<<<dim3(gx, (unsigned)jobs.count), 256, 0, s>>>(jobs);
  return cudaGetLastError();
}

}  // namespace ssm
