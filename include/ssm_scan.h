/*
 * ssm_scan.h -- C ABI of the B200 (sm_100a) selective-scan library.
 *
 * The library computes the selective state-space scan "S6" of Algorithm 2 (steps 5-6), forward and backward,
 * fused with the skip term and the SiLU gate of the block it sits in (Section 3.4).  For every batch index b and
 * channel d independently (Section 2, "Structure and Dimensions": diagonal A, one SSM per channel), with
 * t = 1..L and n = 1..N:
 *
 *     a[t,n]  = exp(delta[b,t,d] * A[d,n])                                   discretization, Eq. 4 (A-bar)
 *     h[t,n]  = a[t,n] * h[t-1,n] + delta[b,t,d] * B[b,t,n] * x[b,t,d]       recurrence, Eq. 2a; h[0,n] = 0
 *     s[t]    = sum_n C[b,t,n] * h[t,n] + D_skip[d] * x[b,t,d]               readout, Eq. 2b, plus skip term
 *     out[b,t,d] = s[t] * z[b,t,d] / (1 + exp(-z[b,t,d]))                    SiLU gate
 *
 * B-bar is delta*B unless SSM_FLAG_ZOH_BBAR asks for the zero-order-hold expression of Eq. 4.  delta is the positive
 * step size, i.e. the value AFTER the softplus of Algorithm 2 step 4 (the *_fused_dt calls take the pre-activation).
 * The (batch, L, D, N) tensors a, B-bar and h never exist in device memory (Section 3.3); long sequences are split in
 * time and the state is carried between the pieces (the chunked scan of Appendix D).  The backward pass recomputes the states from saved or
 * rebuilt checkpoint states instead of reading them (Section 3.3 and Appendix D, recomputation).
 *
 * Conventions common to all entry points
 *   - Every pointer except `p` is DEVICE memory owned by the caller (ssm_scan_fwd_bwd_host alone takes host
 *     buffers); the library never allocates, frees or keeps a pointer after the call returns.  Scratch memory is the caller's `workspace` (size from the *_workspace_bytes
 *     queries; at least 256-byte aligned; contents undefined between calls; calls that overlap on the GPU must not
 *     share a workspace).
 *   - Layouts are dense row-major: x, delta, z, out, dout, dx, ddelta, dz are [batch][L][D]; B, C, dB, dC are
 *     [batch][L][N] (float32 [D][N] with SSM_FLAG_STATIC_B / _C); A, dA are [D][N]; D_skip, dD are [D].
 *   - x, delta, B, C, z, out, dout, dx, ddelta, dB, dC, dz have the element type `io_dtype`; A, D_skip, dA, dD and
 *     every state are float32; all arithmetic and accumulation is float32; results are rounded once to io_dtype
 *     (round-to-nearest-even).
 *   - Outputs are overwritten, never accumulated.  Inputs must not alias outputs.
 *   - Calls enqueue work on `stream` and return without synchronising.  Argument errors are detected before
 *     anything is launched and reported by the return value; nothing is written in that case.  A failed kernel
 *     launch is reported as SSM_ERR_CUDA.
 *   - N must be 1, 2, 4, 8, 16 (the state sizes Table 10 ablates), 32 or 64 (larger states on the generic kernels;
 *     the tuned kernels are N = 16; bf16 problems with N < 16 and D % 8 == 0 run on them too, with A, B, C and the
 *     state arrays widened inside the workspace by columns that stay zero).  All io pointers must be
 *     aligned to the element size; 16-byte aligned pointers together with D % 8 == 0 select the vector path.
 *   - Results are bitwise reproducible for fixed inputs, shape, flags and library build: every reduction (over n,
 *     over channels for dB/dC, over batch and time for dA/dD) has a fixed order and no floating-point atomics
 *     are used.
 *   - NaN and Inf propagate; signs are not validated (A < 0 and delta > 0 are expected).
 */
#ifndef SSM_SCAN_H_
#define SSM_SCAN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define SSM_API __attribute__((visibility("default")))
#else
#define SSM_API
#endif

typedef enum {
  SSM_OK = 0,
  SSM_ERR_INVALID_ARG = 1,  /* null required pointer, non-positive dimension, misaligned pointer, bad flag      */
  SSM_ERR_UNSUPPORTED = 2,  /* N or dtype outside the supported set                                             */
  SSM_ERR_WORKSPACE = 3,    /* workspace null / misaligned / smaller than the query reports                     */
  SSM_ERR_CUDA = 4,         /* a CUDA runtime call or a kernel launch failed                                    */
  SSM_ERR_TIMEOUT = 5,      /* a bounded device-side wait gave up (reported by ssm_scan_check_status)           */
  SSM_ERR_BOUNDS = 6        /* bounds-checking build only: a tuned kernel computed a tile row or a global row /
                               channel outside its range; the access was clamped or skipped, nothing faulted
                               (reported by ssm_scan_check_status)                                              */
} ssm_status_t;

typedef enum { SSM_F32 = 0, SSM_BF16 = 1 } ssm_dtype_t;

enum {
  SSM_FLAG_HAS_Z = 1u,        /* z is given: out = s * silu(z); otherwise out = s and dz is not produced        */
  SSM_FLAG_HAS_DSKIP = 2u,    /* D_skip is given; otherwise the skip term is absent and dD is not produced      */
  SSM_FLAG_SAVE_STATES = 4u,  /* forward: also write the checkpoint states that backward starts its recomputation
                                 from (the scan states Appendix D keeps between chunks)                          */
  SSM_FLAG_GENERAL_A = 8u,    /* do not use the fast path for rows of A that are arithmetic progressions in n   */
  SSM_FLAG_DELTA_SOFTPLUS = 32u, /* ssm_scan_*_fused_dt: the step size is softplus(delta_pre + delta_bias[d])         */
  SSM_FLAG_ZOH_BBAR = 64u,    /* B-bar = (exp(delta A) - 1) / A * B, the zero-order hold of Eq. 4 (delta * B at A = 0),
                                 instead of the default delta * B; honoured by every call                        */
  SSM_FLAG_STATIC_B = 256u,   /* B is not input-dependent (Algorithm 1; the selective-parameter ablation, Table 7): B is a float32
                                 parameter [D][N] like A instead of io_dtype [batch][L][N], and dB is float32 [D][N],
                                 summed over batch and time.  Tuned kernels for bf16 / N = 16 with the default B-bar
                                 rule, generic kernels otherwise.                                                */
  SSM_FLAG_STATIC_C = 512u,   /* the same for C and dC                                                            */
  SSM_FLAG_COMPLEX = 1024u,   /* complex-valued state (Section 3.6): A and dA are float32 [D][N][2], B, C, dB, dC io_dtype
                                 [batch][L][N][2], every state array (saved_states, h0, h_last, dh_last, dh0, the h of
                                 ssm_step) float32 [..][N][2], all as interleaved (re, im) pairs; the readout is
                                 s = 2 Re(sum_n C h) + D_skip x (the N states stand for N conjugate pairs); a gradient
                                 of a complex quantity holds (dL/dRe, dL/dIm).  N <= 32.  Not combined with
                                 SSM_FLAG_ZOH_BBAR, SSM_FLAG_STATIC_B / _C, the *_fused_dt calls or
                                 ssm_scan_fwd_bwd_host (SSM_ERR_UNSUPPORTED).  Plain kernels, no time split.      */
  SSM_FLAG_TEST_WITHHOLD = 16u /* test hook for the bounded waits: the tuned backward kernel shares channel groups
                                 between neighbouring warps whatever the shape, never publishes a hand-off flag and
                                 polls only 1000 times, so every warp that continues a group gives up and
                                 ssm_scan_check_status reports SSM_ERR_TIMEOUT; the gradients are then undefined  */
};

typedef struct {
  int32_t batch, L, D, N;   /* all >= 1 */
  int32_t io_dtype;         /* ssm_dtype_t */
  uint32_t flags;           /* SSM_FLAG_* */
} ssm_problem_t;

/* Bytes of scratch memory ssm_scan_fwd / ssm_scan_bwd need for this problem (0 is possible).  Returns 0 for an
 * invalid problem; the call itself then reports the error. */
SSM_API size_t ssm_scan_fwd_workspace_bytes(const ssm_problem_t* p);
SSM_API size_t ssm_scan_bwd_workspace_bytes(const ssm_problem_t* p);

/* Bytes of the `saved_states` buffer: float32 states h at the start of every block of ssm_scan_checkpoint_steps()
 * time steps.  The buffer is opaque: its layout is the library's ([batch][ceil(L / steps)][D][N], or for bf16 io with
 * N = 16 and D % 8 == 0 a layout tiled by groups of 32 channels, D rounded up to a multiple of 32) and depends on the
 * problem (dimensions, dtype, SSM_FLAG_COMPLEX, the STATIC / ZOH flags); a buffer written by a forward call is valid
 * for backward calls with the same ssm_problem_t only. */
SSM_API size_t ssm_scan_saved_state_bytes(const ssm_problem_t* p);
SSM_API int32_t ssm_scan_checkpoint_steps(void);

/*
 * Forward (Algorithm 2 steps 5-6, Eq. 2a/2b, Eq. 4's A-bar, skip term, gate).
 *   x, delta, B, C        in, io_dtype, required
 *   A                     in, float32 [D][N], required
 *   D_skip                in, float32 [D]; required iff SSM_FLAG_HAS_DSKIP
 *   z                     in, io_dtype; required iff SSM_FLAG_HAS_Z
 *   out                   out, io_dtype [batch][L][D]
 *   saved_states          out, float32, ssm_scan_saved_state_bytes(p) bytes; required iff SSM_FLAG_SAVE_STATES
 *   workspace             scratch of at least ssm_scan_fwd_workspace_bytes(p) bytes (may be NULL if that is 0)
 */
SSM_API ssm_status_t ssm_scan_fwd(const ssm_problem_t* p, const void* x, const void* delta, const float* A, const void* B,
                          const void* C, const float* D_skip, const void* z, void* out, void* saved_states,
                          void* workspace, size_t workspace_bytes, void* stream /* cudaStream_t */);

/*
 * Forward with a carried-in and a carried-out state, for processing a long sequence in pieces or for handing a prompt
 * over to token-by-token generation (Appendix D: with the intermediate scan states one can continue the scan with the
 * next chunk; Section 2: the recurrent mode of Eq. 2).  Same as ssm_scan_fwd, plus
 *   h0        in, float32 [batch][D][N]: the state before the first step (NULL: zero)
 *   h_last    out, float32 [batch][D][N]: the state after the last step (NULL: not wanted)
 * Checkpoint states written with SSM_FLAG_SAVE_STATES include the effect of h0, so ssm_scan_bwd given those saved
 * states returns the gradients of this call's inputs; ssm_scan_bwd_state also returns the gradient with respect to
 * h0 and accepts h0 when it has to rebuild the checkpoints (plain ssm_scan_bwd without saved states assumes h0 = 0).
 */
SSM_API ssm_status_t ssm_scan_fwd_state(const ssm_problem_t* p, const void* x, const void* delta, const float* A,
                                        const void* B, const void* C, const float* D_skip, const void* z,
                                        const float* h0, void* out, float* h_last, void* saved_states,
                                        void* workspace, size_t workspace_bytes, void* stream /* cudaStream_t */);

/*
 * Forward and backward with the step-size activation fused in (Algorithm 2 step 4: Delta = tau_Delta(Parameter +
 * s_Delta(x)) with tau_Delta = softplus, Section 3.2; the bias initialisation of Section 3.6 is that Parameter).
 * `delta_pre` [batch][L][D] (io_dtype) is the output of the projection s_Delta, `delta_bias` float32 [D] the parameter
 * (NULL: zero); the step size used by the scan is
 *     delta = softplus(delta_pre + delta_bias[d])     with SSM_FLAG_DELTA_SOFTPLUS,
 *     delta = delta_pre + delta_bias[d]               without it,
 * evaluated in float32 and never rounded to io_dtype, which saves the separate elementwise pass over [batch][L][D] in
 * each direction.  Everything else is as in ssm_scan_fwd_state / ssm_scan_bwd.  The backward returns
 *     ddelta_pre   io_dtype [batch][L][D]: gradient of the pre-activation (ddelta * sigmoid(delta_pre + bias) with the
 *                  softplus),
 *     ddelta_bias  float32 [D], may be NULL: ddelta_pre summed over batch and time (fixed order).
 * Both calls run the tuned bf16 kernels wherever ssm_scan_fwd / ssm_scan_bwd would.
 */
SSM_API ssm_status_t ssm_scan_fwd_fused_dt(const ssm_problem_t* p, const void* x, const void* delta_pre,
                                           const float* delta_bias, const float* A, const void* B, const void* C,
                                           const float* D_skip, const void* z, const float* h0, void* out,
                                           float* h_last, void* saved_states, void* workspace, size_t workspace_bytes,
                                           void* stream /* cudaStream_t */);
SSM_API ssm_status_t ssm_scan_bwd_fused_dt(const ssm_problem_t* p, const void* x, const void* delta_pre,
                                           const float* delta_bias, const float* A, const void* B, const void* C,
                                           const float* D_skip, const void* z, const void* dout,
                                           const void* saved_states, void* dx, void* ddelta_pre, float* ddelta_bias,
                                           float* dA, void* dB, void* dC, float* dD, void* dz, void* workspace,
                                           size_t workspace_bytes, void* stream /* cudaStream_t */);

/* ssm_scan_bwd_fused_dt for a piece of a longer sequence: h0, dh_last and dh0 as in ssm_scan_bwd_state. */
SSM_API ssm_status_t ssm_scan_bwd_fused_dt_state(const ssm_problem_t* p, const void* x, const void* delta_pre,
                                                 const float* delta_bias, const float* A, const void* B,
                                                 const void* C, const float* D_skip, const void* z,
                                                 const void* dout, const float* h0, const float* dh_last,
                                                 const void* saved_states, void* dx, void* ddelta_pre,
                                                 float* ddelta_bias, float* dA, void* dB, void* dC, float* dD,
                                                 void* dz, float* dh0, void* workspace, size_t workspace_bytes,
                                                 void* stream /* cudaStream_t */);

/*
 * One recurrent step (Eq. 2a/2b evaluated for a single t, the mode used for autoregressive inference): p->L must be
 * 1; x, delta, z, out are [batch][D], B, C are [batch][N] (io_dtype), A [D][N], D_skip [D]; the float32 state
 * h [batch][D][N] is read and overwritten with the state after the step (when N >= 4: h and A 16-byte aligned, B and
 * C aligned to four of their elements).  Needs no workspace.
 */
SSM_API ssm_status_t ssm_step(const ssm_problem_t* p, const void* x, const void* delta, const float* A, const void* B,
                              const void* C, const float* D_skip, const void* z, float* h, void* out,
                              void* stream /* cudaStream_t */);

/*
 * Backward: gradients of loss = sum(dout * out) with respect to every input (the adjoint of the four lines at
 * the top; the states are recomputed on chip from checkpoint states, Section 3.3, recomputation).
 *   x, delta, A, B, C, D_skip, z   the forward inputs, same rules as above
 *   dout                  in, io_dtype [batch][L][D], required
 *   saved_states          in, float32, as written by ssm_scan_fwd with SSM_FLAG_SAVE_STATES for the same problem and
 *                         inputs; NULL makes backward rebuild the checkpoints itself (one more forward sweep)
 *   dx, ddelta            out, io_dtype [batch][L][D], required
 *   dA                    out, float32 [D][N], required
 *   dB, dC                out, io_dtype [batch][L][N], required
 *   dD                    out, float32 [D]; may be NULL; written only with SSM_FLAG_HAS_DSKIP
 *   dz                    out, io_dtype [batch][L][D]; may be NULL; written only with SSM_FLAG_HAS_Z
 *   workspace             scratch of at least ssm_scan_bwd_workspace_bytes(p) bytes
 */
SSM_API ssm_status_t ssm_scan_bwd(const ssm_problem_t* p, const void* x, const void* delta, const float* A, const void* B,
                          const void* C, const float* D_skip, const void* z, const void* dout,
                          const void* saved_states, void* dx, void* ddelta, float* dA, void* dB, void* dC, float* dD,
                          void* dz, void* workspace, size_t workspace_bytes, void* stream /* cudaStream_t */);

/*
 * Backward of a piece of a longer sequence (the counterpart of ssm_scan_fwd_state; Appendix D: the scan is continued
 * chunk by chunk through the intermediate states, and the chain rule crosses a cut the same way).  Same as
 * ssm_scan_bwd, plus
 *   h0        in, float32 [batch][D][N]: the state before the first step, as given to ssm_scan_fwd_state (NULL: zero);
 *             only read when saved_states is NULL (saved states already contain its effect)
 *   dh_last   in, float32 [batch][D][N]: gradient of the loss with respect to the state after the last step that
 *             arrives from outside this piece (the dh0 of the following piece); NULL: zero
 *   dh0       out, float32 [batch][D][N]: gradient with respect to h0; NULL: not wanted
 * Walking the pieces of a sequence from last to first, passing each piece's dh0 as the previous piece's dh_last, gives
 * the gradients of the whole sequence (dA and dD of the pieces add up).
 */
SSM_API ssm_status_t ssm_scan_bwd_state(const ssm_problem_t* p, const void* x, const void* delta, const float* A,
                                        const void* B, const void* C, const float* D_skip, const void* z,
                                        const void* dout, const float* h0, const float* dh_last,
                                        const void* saved_states, void* dx, void* ddelta, float* dA, void* dB, void* dC,
                                        float* dD, void* dz, float* dh0, void* workspace, size_t workspace_bytes,
                                        void* stream /* cudaStream_t */);

/*
 * Reads back whether the last ssm_scan_fwd* / ssm_scan_bwd* call on this workspace completed.  The tuned kernels give
 * every resident warp an equal share of the (channel group, time) work; where a share ends inside a channel group, the
 * next warp continues that group and first waits (with a bounded number of polls) for the state or adjoint the warp
 * before it hands over through the workspace.  If such a wait ever gives up, the waiting warps stop and a status word
 * (the first word of every non-empty workspace) is set.  This call synchronises `stream`, copies that word to the host
 * and returns SSM_ERR_TIMEOUT if it is set (the results of that call are then incomplete), SSM_OK otherwise.  `p` and
 * `workspace` must be those of the call.  A library built with -DSSM_DEBUG_BOUNDS (the stand-in for a memory checker:
 * every tile row index and every global row / channel offset of the tuned kernels is range-checked, a bad one is
 * clamped or its access skipped, nothing traps) reports a violation here as SSM_ERR_BOUNDS.
 */
SSM_API ssm_status_t ssm_scan_check_status(const ssm_problem_t* p, const void* workspace, void* stream /* cudaStream_t */);

/*
 * Forward without any caller-provided scratch memory.  (The paper has no counterpart: this entry point exists for
 * the integration of the library, not for the method.)
 *
 * It is for callers that are not allowed to allocate device memory at the point where they call the scan -- for
 * example a layer plug-in that receives only its input and output buffers from a host framework and must not
 * allocate while enqueueing work, because a device allocation synchronises the GPU, or an application whose memory
 * budget is fixed at start-up.  Same arguments and results as ssm_scan_fwd, minus the workspace: the scratch memory
 * of the time-split forward path is a fixed array of SSM_STATIC_SCRATCH_BYTES bytes inside the library's device
 * image, present on every GPU that loads the library until the process exits.
 *   - A problem whose ssm_scan_fwd_workspace_bytes() exceeds SSM_STATIC_SCRATCH_BYTES is refused with
 *     SSM_ERR_WORKSPACE before anything is launched; use ssm_scan_fwd with your own workspace for those.
 *   - The call allocates and frees nothing.  The first call on a device looks up the device address of the array
 *     (with that device current) and keeps it; make that first call outside any stream capture.
 *   - All calls on a device share the one array: two calls that can overlap on the GPU (different streams, no
 *     dependency between them) race on it and must be ordered by the caller.  The array keeps the contents of the last
 *     call; the kernels overwrite every word of it before they read it, so nothing needs clearing in between.
 */
#define SSM_STATIC_SCRATCH_BYTES (4u << 20)
SSM_API ssm_status_t ssm_scan_fwd_static(const ssm_problem_t* p, const void* x, const void* delta, const float* A,
                                         const void* B, const void* C, const float* D_skip, const void* z, void* out,
                                         void* saved_states, void* stream /* cudaStream_t */);

/*
 * Forward + backward of one batch held in HOST memory, copies included (the paper has no counterpart: its kernels
 * start from tensors already in HBM).  Equivalent to copying every input to the device, calling ssm_scan_fwd with
 * SSM_FLAG_SAVE_STATES and ssm_scan_bwd with those states, and copying every result back; the batch is cut into up
 * to 8 pieces whose copies in, computation and copies out overlap on three streams (the batch entries are
 * independent, Section 2 "Structure and Dimensions").
 *   x, delta, z, dout, B, C, A, D_skip      in, HOST pointers, layouts and dtypes as for ssm_scan_fwd / ssm_scan_bwd
 *   out, dx, ddelta, dz, dB, dC, dA, dD     out, HOST pointers, every element overwritten; dz / dD are required iff
 *                                           SSM_FLAG_HAS_Z / SSM_FLAG_HAS_DSKIP
 *   device_arena   DEVICE scratch of at least ssm_scan_host_arena_bytes(p) bytes, 256-byte aligned, caller-owned
 *   stream         the call is ordered after everything already enqueued on it, and work enqueued on it afterwards
 *                  is ordered after every copy of this call; the call itself does not wait for the GPU
 * Host buffers should be page-locked: with pageable memory the results are the same but the copies do not overlap.
 * The host buffers and the arena must stay valid and untouched until the stream has passed the call.  dA and dD are
 * summed over the pieces in ascending order, so they can differ in the last bit from one ssm_scan_bwd call over the
 * whole batch; everything else is identical.  The library keeps two helper streams per device (created on first use)
 * and allocates no device memory.  Flags other than HAS_Z, HAS_DSKIP, GENERAL_A and ZOH_BBAR are ignored.
 * Errors: SSM_ERR_INVALID_ARG / SSM_ERR_UNSUPPORTED as for the device calls, SSM_ERR_WORKSPACE for a short, NULL or
 * misaligned arena (nothing is enqueued), SSM_ERR_CUDA if a runtime call fails (the stream is still ordered after
 * whatever had been enqueued).
 */
SSM_API size_t ssm_scan_host_arena_bytes(const ssm_problem_t* p);
SSM_API ssm_status_t ssm_scan_fwd_bwd_host(const ssm_problem_t* p, const void* x, const void* delta, const float* A,
                                           const void* B, const void* C, const float* D_skip, const void* z,
                                           const void* dout, void* out, void* dx, void* ddelta, float* dA, void* dB,
                                           void* dC, float* dD, void* dz, void* device_arena, size_t arena_bytes,
                                           void* stream /* cudaStream_t */);

/* Human-readable name of a status code (static storage). */
SSM_API const char* ssm_status_string(ssm_status_t s);

/*
 * Describes how the library would run this problem: number of time segments the sequence is split into, steps per
 * segment, channels per thread block and states per thread of the forward kernel.  Any output pointer may be NULL.
 * Returns SSM_OK or the validation error.  Host-only; launches nothing.
 */
SSM_API ssm_status_t ssm_scan_plan(const ssm_problem_t* p, int32_t* n_segments, int32_t* segment_steps,
                           int32_t* channels_per_block, int32_t* states_per_thread);

/*
 * The same for the backward pass, which decides about its time split on its own terms (Appendix D, chunking; the
 * checkpoint states do not depend on the split): number of time segments, steps per segment, and the number of
 * channels whose dB / dC terms are summed before they leave a kernel as a partial sum.  Any output pointer may be NULL.
 * Host-only; launches nothing.
 */
SSM_API ssm_status_t ssm_scan_bwd_plan(const ssm_problem_t* p, int32_t* n_segments, int32_t* segment_steps,
                                       int32_t* channels_per_group);

#ifdef __cplusplus
}
#endif
#endif /* SSM_SCAN_H_ */
