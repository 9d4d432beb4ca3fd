/*
 * ssm_conv1d.h -- C ABI of the short causal depthwise convolution (+ SiLU) that feeds the selective scan
 * (Section 3.4 and Figure 3: on the SSM branch of the block the projected input passes a short convolution and the
 * SiLU activation before it becomes the scan's x).  A neighbour of the hot path, not part of the scan itself.
 *
 * Per batch b and channel d independently, with W taps per channel whose LAST tap multiplies the current step:
 *     pre[b,t,d] = bias[d] + sum_{k=0}^{W-1} w[d,k] * x[b, t-(W-1)+k, d]         (x before the sequence: x_prev or 0)
 *     y[b,t,d]   = pre * sigmoid(pre)   with SSM_CONV_FLAG_SILU, else pre
 * Backward for loss = sum(dy * y):  dpre = dy * silu'(pre);  dx[b,s,d] = sum_k w[d,k] dpre[b, s+(W-1)-k, d];
 *     dw[d,k] = sum_{b,t} dpre[b,t,d] x[b,t-(W-1)+k,d];  dbias[d] = sum_{b,t} dpre[b,t,d]   (fixed summation order).
 *
 * Conventions as in ssm_scan.h: plain C, no torch types; every pointer is caller-owned DEVICE memory valid for
 * `stream`; the library allocates nothing; calls enqueue and return; argument errors are reported before anything is
 * launched; outputs are overwritten; results are bitwise reproducible.
 * Layouts: x, y, dy, dx contiguous [batch][L][D] in io_dtype; x_prev, dx_prev [batch][W-1][D] in io_dtype;
 * w, dw float32 [D][W]; bias, dbias float32 [D].  Arithmetic is float32.  The vector path (4 elements per access)
 * needs D % 4 == 0 and x / y / dy / dx / x_prev / dx_prev aligned to 4 elements; otherwise a scalar path with the
 * same results runs.
 */
#ifndef SSM_CONV1D_H_
#define SSM_CONV1D_H_

#include "ssm_scan.h"

#ifdef __cplusplus
extern "C" {
#endif

enum {
  SSM_CONV_FLAG_SILU = 1u,     /* y = silu(pre); otherwise y = pre                  */
  SSM_CONV_FLAG_HAS_BIAS = 2u  /* bias is given; otherwise 0 and dbias not produced */
};

typedef struct {
  int32_t batch, L, D;   /* all >= 1 */
  int32_t width;         /* taps per channel, 1..4 */
  int32_t io_dtype;      /* ssm_dtype_t */
  uint32_t flags;        /* SSM_CONV_FLAG_* */
} ssm_conv_problem_t;

/*
 * Forward.  x, w, y required; bias required iff SSM_CONV_FLAG_HAS_BIAS; x_prev may be NULL (zeros): the W-1 inputs
 * that precede the first step when a sequence is processed in pieces.  Needs no workspace.
 */
SSM_API ssm_status_t ssm_conv1d_fwd(const ssm_conv_problem_t* p, const void* x, const float* w, const float* bias,
                                    const void* x_prev, void* y, void* stream /* cudaStream_t */);

/* Bytes of scratch ssm_conv1d_bwd needs (per-block partial sums of dw and dbias); 0 for an invalid problem. */
SSM_API size_t ssm_conv1d_bwd_workspace_bytes(const ssm_conv_problem_t* p);

/*
 * Backward.  The pre-activation is recomputed from x (nothing is saved by the forward call, in the spirit of the
 * block-level recomputation of Appendix D).  x, w, dy, dx, dw required; bias / x_prev as in the forward call;
 * dbias may be NULL; dx_prev may be NULL (gradient of x_prev, [batch][W-1][D] io_dtype).  workspace of at least
 * ssm_conv1d_bwd_workspace_bytes(p) bytes, 16-byte aligned.
 */
SSM_API ssm_status_t ssm_conv1d_bwd(const ssm_conv_problem_t* p, const void* x, const float* w, const float* bias,
                                    const void* x_prev, const void* dy, void* dx, float* dw, float* dbias,
                                    void* dx_prev, void* workspace, size_t workspace_bytes,
                                    void* stream /* cudaStream_t */);

#ifdef __cplusplus
}
#endif
#endif /* SSM_CONV1D_H_ */
