/*
 * osdn.h -- C ABI of the B200 (sm_100a) OSDN layer library.
 *
 * The library computes the chunkwise-parallel, gated, online-scaled delta-rule
 * sequence layer (OSDN / OSGDN with Adaptive Preconditioner Forgetting):
 *
 *   phase 1  (Algorithm 1; Eq. "dt_update_apf"; beta-aware form
 *             Eq. "extension_beta_aware_phase1"), per (sequence, head), t = 1..L:
 *       ktil_t  = d_t (.) k_t                          (write key, pre-update d)
 *       c_t     = eta * b_t * (1 - b_t <d_t, k_t^2>) / max(|k_t|^2, eps),  b_t = beta_t or 1
 *       d_{t+1} = clip(rho_t d_t + c_t k_t^2, d_min, d_max),  rho_t = 1 | exp(g_t) | exp(l_t)
 *   phase 2  (Eq. "recurrent_form" with the gate of the backbone-extension appendix):
 *       S_t = exp(g_t) S_{t-1} + beta_t (v_t - exp(g_t) S_{t-1} k_t) ktil_t^T ,  o_t = scale * S_t q_t
 *
 * evaluated chunk by chunk (chunk = 64 tokens) through the UT / WY transform of the
 * chunkwise-WY appendix and its gated form (decay-ratio Gram, unit-triangular inverse,
 * pseudo keys W and values U, suffix-gated state advance), and the reverse-mode
 * derivative of all of it (Section 3.5: phase 2 yields dL/dktil, the gradient through d
 * is a reverse sweep over the projected affine recurrence).
 *
 * Conventions
 *   - Every data pointer is a DEVICE pointer unless the name ends in _host.  The caller
 *     owns all buffers; the library allocates no device memory and keeps no state
 *     between calls.  Calls only enqueue work on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = default stream) and return without synchronising.
 *   - Token tensors are packed [T_total, H, D] row-major (a dense [B, T, H, D] batch is
 *     the same memory).  q, k, v, out, dout, dq, dk, dv are `io_dtype` (fp32 or bf16);
 *     beta, gate (log-decay g <= 0), log-retention, states, preconditioners and their
 *     gradients are fp32.  States are [S, H, V, K], preconditioners [S, H, K], where
 *     S = B (dense) or nseq (var-len).  All pointers must be 16-byte aligned.
 *   - Sequences: dense (nseq == 0): B sequences of T tokens.  Var-len (nseq > 0): B must
 *     be 1, T is the packed token count and cu_seqlens (device, int32, nseq+1 entries,
 *     non-decreasing, cu[0] = 0, cu[nseq] = T) gives the boundaries; state and
 *     preconditioner restart at every boundary and chunks never straddle sequences.
 *   - Return value: 0 on success, a negative osdn_status otherwise.  Arguments are
 *     validated before anything is launched; on error nothing has been enqueued.
 *     Errors detected on the device (a bounded wait that ran out) are recorded in the
 *     first 4 bytes of the workspace, readable with osdn_read_device_status after the
 *     stream has been synchronised.
 */
#ifndef OSDN_H_
#define OSDN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum osdn_status {
    OSDN_OK = 0,
    OSDN_INVALID_ARG = -1,        /* null required pointer, bad enum, inconsistent sizes   */
    OSDN_UNSUPPORTED_SHAPE = -2,  /* K or V not in {64, 128}, chunk != 64, T <= 0, ...      */
    OSDN_MISALIGNED = -3,         /* a pointer is not 16-byte aligned                      */
    OSDN_WORKSPACE_TOO_SMALL = -4,
    OSDN_CUDA_ERROR = -5,         /* a CUDA runtime call or launch failed                  */
    OSDN_STATIC_SCRATCH_TOO_SMALL = -6 /* osdn_fwd_static: problem larger than the built-in scratch */
} osdn_status;

/* Values found in the device status word (first 4 bytes of a workspace) after a call whose kernels
 * met an error on the device.  101..113, 121, 122, 131: a bounded wait inside a kernel ran out (an
 * mbarrier of the tensor-core kernels, the backward's tile queue, a ready flag of the merged forward
 * launch, a ring barrier of the pipelined preconditioner pass); the kernel then skipped the dependent
 * work and returned, and the outputs of that call are undefined. */
enum {
    OSDN_DEVICE_OK = 0,
    OSDN_DEVICE_BAD_CU_SEQLENS = 120,   /* cu_seqlens broke its contract (cu[0] != 0, a decreasing pair,
                                           cu[nseq] != T); sequences were clamped into [0, T], so no
                                           access left the user tensors, but the results are undefined */
    OSDN_DEVICE_SELFTEST_TIMEOUT = 199  /* written by osdn_selftest_wait_timeout                         */
};

enum { OSDN_FP32 = 0, OSDN_BF16 = 1 };
/* Retention of the preconditioner (Eq. "dt_update_apf"): none, the layer's gate, a separate
 * log-retention per (token, head), or one per coordinate (the vector-retention extension of the
 * update's affine form: diag(r_t) in place of r_t I). */
enum { OSDN_APF_NONE = 0, OSDN_APF_ALIAS_GATE = 1, OSDN_APF_SEPARATE = 2, OSDN_APF_VECTOR = 3 };
enum {
    OSDN_FLAG_SAVE_RESIDUALS = 1,  /* osdn_fwd: keep chunk residuals in the workspace for osdn_bwd */
    OSDN_FLAG_RESIDUALS_VALID = 2, /* osdn_bwd: the workspace holds the residuals of the matching
                                      osdn_fwd call (same params, same inputs); otherwise osdn_bwd
                                      recomputes the forward itself                              */
    OSDN_FLAG_FORCE_SIMT = 4       /* use the fp32 CUDA-core kernels even for bf16 I/O          */
};

typedef struct osdn_params {
    int32_t B, T, H, K, V;      /* dense: [B,T,H,*]; var-len: B = 1, T = packed tokens          */
    int32_t chunk;              /* 64                                                            */
    int32_t io_dtype;           /* OSDN_FP32 | OSDN_BF16                                         */
    float   eta, d_min, d_max;  /* step size and box of the preconditioner (0.003, 0.5, 2.0)     */
    float   eps;                /* floor of |k|^2 (1e-6)                                         */
    float   scale;              /* output scale on q; <= 0 selects K^-1/2                        */
    int32_t beta_aware;         /* 1: b_t = beta_t ; 0: b_t = 1                                  */
    int32_t apf_mode;           /* OSDN_APF_*                                                    */
    int32_t clamp;              /* 1: project onto the box after every token ; 0: never          */
    int32_t nseq;               /* 0 = dense                                                     */
    const int32_t* cu_seqlens;  /* device pointer, nseq+1 entries (var-len only)                 */
    int32_t flags;              /* OSDN_FLAG_*                                                   */
} osdn_params;

/* Bytes of device scratch the calls below need for these params (need_bwd != 0: enough
 * for osdn_fwd with OSDN_FLAG_SAVE_RESIDUALS followed by osdn_bwd).  0 on invalid params. */
size_t osdn_workspace_bytes(const osdn_params* p, int need_bwd);

/*
 * Forward (Algorithm 1 + the gated chunk form).
 *   in : q,k [T,H,K], v [T,H,V] io_dtype; beta, gate [T,H] fp32;
 *        apf_log_ret fp32: [T,H] for apf_mode == SEPARATE, [T,H,K] for VECTOR (required for
 *        these two modes, else may be NULL);
 *        init_state [S,H,V,K] (NULL = zeros); precond_in [S,H,K] (NULL = ones).
 *   out: out [T,H,V] io_dtype; final_state [S,H,V,K] and precond_out [S,H,K] fp32 (either may
 *        be NULL; precond_out may alias precond_in).
 *   workspace: >= osdn_workspace_bytes(p, flags & SAVE_RESIDUALS) bytes, 256-byte aligned.
 */
int osdn_fwd(const osdn_params* p, const void* q, const void* k, const void* v,
             const float* beta, const float* gate, const float* apf_log_ret,
             const float* init_state, const float* precond_in,
             void* out, float* final_state, float* precond_out,
             void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward (Section 3.5): gradients of sum(out*dout) + sum(final_state*dfinal_state) +
 * sum(precond_out*dprecond_out) with respect to every forward input.
 *   in : the forward inputs; dout [T,H,V] io_dtype; dfinal_state, dprecond_out (NULL = zeros).
 *   out: dq, dk [T,H,K], dv [T,H,V] io_dtype; dbeta, dgate [T,H] fp32;
 *        dapf_log_ret, shaped like apf_log_ret (written iff apf_mode is SEPARATE or VECTOR; may be
 *        NULL otherwise);
 *        dinit_state [S,H,V,K], dprecond_in [S,H,K] (either may be NULL).
 *   The projection passes gradient where d_min <= pre-projection value <= d_max;
 *   max(|k|^2, eps) passes gradient where |k|^2 > eps.
 *   workspace: >= osdn_workspace_bytes(p, 1) bytes.
 */
int osdn_bwd(const osdn_params* p, const void* q, const void* k, const void* v,
             const float* beta, const float* gate, const float* apf_log_ret,
             const float* init_state, const float* precond_in,
             const void* dout, const float* dfinal_state, const float* dprecond_out,
             void* dq, void* dk, void* dv, float* dbeta, float* dgate, float* dapf_log_ret,
             float* dinit_state, float* dprecond_in,
             void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Phase 1 alone (Algorithm 1 as its own pass; Section 3.5 "Phase 1"): advances the
 * preconditioner over the given tokens and optionally emits the write keys.
 *   in : k [T,H,K] io_dtype; beta [T,H]; gate_or_log_ret (the log-retention source: the gate
 *        [T,H] for ALIAS_GATE, the separate log-retention [T,H] for SEPARATE or [T,H,K] for VECTOR;
 *        may be NULL for APF_NONE); precond_in [S,H,K] (NULL = ones).
 *   out: k_tilde_out [T,H,K] io_dtype (may be NULL); precond_out [S,H,K] (required; may alias
 *        precond_in).  Needs no workspace for dense batches; var-len reads cu_seqlens directly.
 */
int osdn_precond_update(const osdn_params* p, const void* k, const float* beta,
                        const float* gate_or_log_ret, const float* precond_in,
                        void* k_tilde_out, float* precond_out, void* cuda_stream);

/*
 * Residual ratio of the paper's mechanism diagnostic (Section "Mechanism diagnostic"; Eq. "qt_form" in
 * the proof of the token-local theorem), a by-product of the same sweep: for every token-head
 *     q_t = f_t(S_t) / f_t(S_{t-1}) = (1 - beta_t <d_t, k_t^2>)^2,   f_t(S) = |S k_t - v_t|^2 / 2,
 * the factor by which the write of token t shrinks its own loss (with the gate, S_{t-1} is the gated
 * state the write starts from), where d_t is the preconditioner the write key of token t is formed
 * with; it needs neither the state nor the values.  eta = 0 with precond_in = NULL gives the ratio of
 * the unscaled delta rule.
 *   in : k, beta, gate_or_log_ret, precond_in as for osdn_precond_update.
 *   out: ratio_out [T,H] fp32 (may be NULL); log_ratio_sum [S,H] fp32 = sum over the sequence of
 *        log(max(q_t, FLT_MIN)) (may be NULL; the geometric mean of a chain is exp(sum / length));
 *        at least one of the two; precond_out [S,H,K] (may be NULL; may alias precond_in).
 */
int osdn_residual_ratio(const osdn_params* p, const void* k, const float* beta,
                        const float* gate_or_log_ret, const float* precond_in,
                        float* ratio_out, float* log_ratio_sum, float* precond_out, void* cuda_stream);

/*
 * Recurrent (decode) step (appendix paragraph "Single-token recurrence kernel for OSGDN", stated
 * for q_len <= 64): for the p->T new tokens of each of the p->B sequences, in order,
 *     alpha_t = exp(g_t);  ktil_t = d_t (.) k_t;  d_{t+1} as in osdn_fwd (Algorithm 1 with APF and the
 *     box projection);  S_t = alpha_t S_{t-1} + beta_t (v_t - alpha_t S_{t-1} k_t) ktil_t^T;
 *     o_t = scale S_t q_t,
 * in one launch.  It is the recurrence osdn_fwd evaluates chunk by chunk, so a prefill with osdn_fwd
 * (final_state, precond_out) followed by this call continues the same sequence.
 *   in    : q, k [B,T,H,K], v [B,T,H,V] io_dtype; beta, gate [B,T,H] fp32; apf_log_ret [B,T,H]
 *           (apf_mode == SEPARATE) or [B,T,H,K] (VECTOR), required for these two modes.  Dense batches only (p->nseq == 0).
 *   in/out: state [B,H,V,K] fp32 and precond [B,H,K] fp32, the caller's cache, updated in place.
 *   out   : out [B,T,H,V] io_dtype.
 * All pointers are DEVICE pointers, 16-byte aligned.  No workspace, nothing is allocated.  Any T >= 1
 * is accepted; the call is sequential over T, so long prompts belong to osdn_fwd.  Errors as for
 * osdn_fwd (nothing is launched on an argument error).
 */
int osdn_decode_step(const osdn_params* p, const void* q, const void* k, const void* v,
                     const float* beta, const float* gate, const float* apf_log_ret,
                     float* state, float* precond, void* out, void* cuda_stream);

/*
 * Channel-gate variant of the layer: the OSKDA backbone extension (appendix "Kimi Delta Attention with
 * Online Scaling").  The scalar gate of osdn_fwd becomes one gate per key channel,
 *     Sbar = S_{t-1} Diag(alpha_t),  alpha_t = exp(gate_k[t]) in (0,1]^K,
 *     u = v_t - Sbar k_t,   S_t = Sbar + beta_t u ktil_t^T,   o_t = scale S_t q_t,
 * with ktil_t = d_t (.) k_t and d_{t+1} exactly as in osdn_fwd (the beta-aware phase 1 of that appendix;
 * the preconditioner's retention is its own input and never the channel gate, so OSDN_APF_ALIAS_GATE is
 * rejected with OSDN_INVALID_ARG).  The paper writes the state as K x V with the gate, the read key and
 * the scaled write key acting from the left; that state is the transpose of the [S,H,V,K] state used
 * here and by every other call of this library.
 *   gate_k   [T,H,K] fp32 DEVICE, log of the channel gates (<= 0); every other argument, the layouts,
 *            the flags, the alignment rules, ownership and the error codes are those of osdn_fwd / osdn_bwd.
 *   dgate_k  [T,H,K] fp32, written in full.
 *   workspace: osdn_kda_workspace_bytes(p, need_bwd) bytes (0 is returned for rejected parameters); for
 *            the backward it includes, beside the regions of osdn_workspace_bytes, one row history of 16
 *            tokens and four row checkpoints per state row (S * H * V * 20 * K floats) and an fp32
 *            accumulator for dq.
 * This path runs on CUDA cores in fp32 for both io_dtypes (one warp per state row, sequential over the
 * tokens of a sequence): it is the extension's reference implementation on the device, not a tuned one.
 */
size_t osdn_kda_workspace_bytes(const osdn_params* p, int need_bwd);
int osdn_kda_fwd(const osdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                 const float* gate_k, const float* apf_log_ret, const float* init_state,
                 const float* precond_in, void* out, float* final_state, float* precond_out,
                 void* workspace, size_t workspace_bytes, void* cuda_stream);
int osdn_kda_bwd(const osdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                 const float* gate_k, const float* apf_log_ret, const float* init_state,
                 const float* precond_in, const void* dout, const float* dfinal_state,
                 const float* dprecond_out, void* dq, void* dk, void* dv, float* dbeta, float* dgate_k,
                 float* dapf_log_ret, float* dinit_state, float* dprecond_in, void* workspace,
                 size_t workspace_bytes, void* cuda_stream);

/*
 * Forward pass for callers that cannot provide a workspace.  (The paper has no counterpart to
 * this call; it exists for deployment reasons only.)
 *
 * Some callers are not able to allocate device memory at the point where they need the layer:
 * code running inside a serving loop whose memory pool is fixed at start-up, plugins that are
 * handed input and output buffers by a host framework but no allocator, and code that must not
 * call cudaMalloc because that call synchronises the device.  osdn_fwd_static computes exactly
 * what osdn_fwd computes (same kernels, same results) but takes its scratch space from a fixed
 * array of OSDN_STATIC_SCRATCH_BYTES that is part of the library image: every GPU that loads the
 * library holds that array until the process exits.  The call allocates nothing, neither with
 * cudaMalloc nor through any library.
 *
 *   - Inputs and outputs are passed exactly as for osdn_fwd (flags other than
 *     OSDN_FLAG_FORCE_SIMT are ignored: residuals for a backward pass are not kept).
 *   - Problems whose forward workspace (osdn_workspace_bytes(p, 0)) exceeds
 *     OSDN_STATIC_SCRATCH_BYTES are rejected with OSDN_STATIC_SCRATCH_TOO_SMALL before anything is
 *     launched; use osdn_fwd with a caller-owned workspace for those.
 *   - The first call on each device looks up the device address of the array (with that device
 *     current) and remembers it; make that first call before starting any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the last call left in it;
 *     the call clears the part that has to start at zero itself.  Two calls that overlap on the
 *     GPU (different streams, or different host threads without ordering) race on the array and
 *     give undefined results: serialise them.
 *   - The array is looked up for the device that is current when the call is made: `cuda_stream`
 *     must be a stream of that device.
 *   - The device status word of such a call sits inside the array, where the caller cannot point
 *     osdn_read_device_status at it: osdn_read_static_status reads it (synchronous 4-byte copy from
 *     the array of the current device; call it after synchronising the stream).
 */
#define OSDN_STATIC_SCRATCH_BYTES (32u << 20)
int osdn_fwd_static(const osdn_params* p, const void* q, const void* k, const void* v,
                    const float* beta, const float* gate, const float* apf_log_ret,
                    const float* init_state, const float* precond_in,
                    void* out, float* final_state, float* precond_out, void* cuda_stream);
int osdn_read_static_status(int32_t* status_host);

/*
 * Host-buffer convenience for end-to-end measurements: copies the inputs (HOST pointers,
 * ideally pinned) into `staging` (device scratch of osdn_host_staging_bytes bytes), runs
 * osdn_fwd (and osdn_bwd when dout_host != NULL) and copies out / the gradients back to the
 * host buffers, without synchronising: when the call returns everything is enqueued and ordered
 * before whatever is enqueued on `cuda_stream` next.  Same layouts as above.
 *
 * A dense batch with B > 1 is cut into its B sequences (independent problems): the inputs of
 * sequence b + 1 arrive and the results of sequence b - 1 leave while sequence b is computed.  The
 * copies run on two internal streams that fork from and join `cuda_stream`; the streams and the
 * events between them are created on the first such call on a device and kept.  Packed batches
 * (nseq > 0) and B = 1 run in one piece on `cuda_stream` alone and create nothing.
 */
size_t osdn_host_staging_bytes(const osdn_params* p, int with_bwd);
int osdn_step_host(const osdn_params* p, const void* q_host, const void* k_host, const void* v_host,
                   const float* beta_host, const float* gate_host, const void* dout_host,
                   void* out_host, void* dq_host, void* dk_host, void* dv_host,
                   float* dbeta_host, float* dgate_host,
                   void* staging, size_t staging_bytes, void* cuda_stream);

/*
 * Location of a named region inside a workspace laid out for (p, need_bwd): "p1_skip"
 * ([chunks, H, 2] uint32: bit i of the 64-bit pair = token i of the chunk was skipped by the
 * sequential preconditioner pass, i.e. it was entered on the lower face of the box and its
 * projection mask is all zero) and "p1_mask" ([T, H, 32] uint32, with R = K/32: bit r of word l =
 * the projection passed gradient for coordinate R l + r; valid for tokens that were not skipped).
 * Chunks are numbered sequence by sequence, ceil(len / 64) per sequence.  Filled by osdn_fwd with
 * OSDN_FLAG_SAVE_RESIDUALS.  For inspection and tests; returns 0 or OSDN_INVALID_ARG.
 */
int osdn_workspace_region(const osdn_params* p, int need_bwd, const char* name, size_t* offset, size_t* bytes);

/* Reads the device status word at the head of a workspace (synchronous 4-byte copy).
 * 0 = no device-side error recorded. */
int osdn_read_device_status(const void* workspace, int32_t* status_host);

/*
 * Self-test of the device-side error path (no counterpart in the paper).  Every wait inside the
 * tensor-core kernels is bounded: when it runs out the kernel records a code in the device status
 * word and returns instead of spinning.  This call exercises exactly that mechanism by itself: it
 * clears the status word of `workspace` (device memory, >= 256 bytes, 256-byte aligned) and launches
 * one warp that waits, for at most about `limit_us` microseconds (1..100000), on a barrier nothing
 * ever arrives on.  The kernel returns by itself; after synchronising the stream
 * osdn_read_device_status yields OSDN_DEVICE_SELFTEST_TIMEOUT.
 */
int osdn_selftest_wait_timeout(void* workspace, uint32_t limit_us, void* cuda_stream);

const char* osdn_status_string(int status);

/* Number of kernel launches the most recent osdn_fwd / osdn_bwd / osdn_precond_update call of
 * this thread enqueued (for launch accounting in benchmarks). */
int osdn_last_launch_count(void);

/*
 * Optional per-kernel timing for benchmarks (not part of the method).  While enabled, the library
 * records a CUDA event on the launching stream before each of its kernels (at most 2048 marks
 * since the last enable; later launches go unrecorded).  After synchronising the stream,
 * osdn_stage_timing_read(i, &name, &ms) yields the name and duration of the i-th recorded kernel
 * (name == NULL for separators between calls) and returns the number of marks.  Process-wide, not
 * thread safe; enable(0) switches it off again.
 */
void osdn_stage_timing_enable(int on);
int osdn_stage_timing_read(int index, const char** name, float* ms);

#ifdef __cplusplus
}
#endif
#endif /* OSDN_H_ */
