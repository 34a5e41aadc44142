/*
 * e2ttt.h - C ABI of the E2-TTT chunk-parallel fast-weight update for NVIDIA B200 (sm_100a).
 *
 * What is computed (paper: "Rethinking Expressivity and Efficiency in Test-Time Training").
 * For each of the B*H independent sequences, the L tokens are cut into chunks of C tokens.  A
 * chunk starts from the fast-weight state W_0 and momentum state M_0 left by the previous chunk
 * (Section 3, "Primal Formulation") and
 *   - emits the outputs o_t = f_{W_0}(q_t) from the chunk-start weights (Eq. "chunkwise_output",
 *     Algorithm 1 line 1);
 *   - takes the per-token negative gradients G_t = -grad_W 1/2 ||f_{W_0}(k_t) - v_t||^2 at the
 *     chunk-start weights with one inner forward/backward over the whole chunk (Algorithm 1
 *     lines 1 and 3, Appendix "Single Backward Pass for Both Aggregates");
 *   - forms the scalar kernels K^W_t, K^M_t and the three carries from the per-token gates with
 *     suffix scans (Eq. "scalar_aux", Algorithm 1 line 2);
 *   - jumps to the chunk-end states with Proposition 1 (Eq. "Mc_closed", "Wc_closed"; Algorithm 1
 *     lines 4-7):
 *         M_C = bt_0 M_0 + sum_t K^M_t G_t
 *         W_C = gt_0 W_0 + bt_0 R_1 M_0 + sum_t K^W_t G_t
 *     which equal the result of the token-wise recurrence  M_t = beta_t M_{t-1} + eta_t G_t,
 *     W_t = gamma_t W_{t-1} + M_t  (Eq. "tokenwise_ttt_decay_momentum").
 * Fast-weight networks (Section 4, "Fast-weight Network"):
 *     E2TTT_MLP_GELU : f_W(x) = x + LN(W2 GELU(W1 x)),               W1 [h,d], W2 [d,h]
 *     E2TTT_SWIGLU   : f_W(x) = x + LN(W3 (SiLU(W1 x) * (W2 x))),    W1 [h,d], W2 [h,d], W3 [d,h]
 * LN is a layer norm over the d outputs without affine parameters (biased variance, ln_eps inside
 * the square root); GELU is the exact erf form.  All matrices of the collection share the same
 * per-token scalars (Section 2: for a multi-layer learner W_t stands for all of its matrices).
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers unless the comment says "host".  Pointer tables
 *     (W_init and friends) are HOST arrays of e2ttt_num_matrices(kind) device pointers.
 *   - Tensors are dense and row-major: there are no stride fields, a caller with another layout
 *     makes a dense copy first.  q, k, v, o and their gradients: [B, H, L, d] in io_dtype.  Gates and gate gradients: [B, H, L] fp32.  Fast-weight / momentum matrices and
 *     their gradients: [B, H, rows, cols] fp32.
 *   - The caller owns every buffer.  The library allocates nothing and keeps no state between
 *     calls other than cached kernel attributes (one exception, stated there:
 *     e2ttt_chunk_fwd_noalloc uses a scratch array of its own).  Work is enqueued on `stream` (a cudaStream_t
 *     passed as void*, NULL = the default stream); no entry point synchronises with the host.
 *   - Return value: E2TTT_OK (0) or a negative e2ttt_status.  Arguments are validated before
 *     anything is launched, so a failing call leaves every output untouched.  Nothing throws,
 *     aborts or prints.
 *   - Final-state buffers may alias the initial-state buffers (in-place state update).  No other
 *     output may overlap an input or another output.
 */
#ifndef E2TTT_H
#define E2TTT_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define E2TTT_API __attribute__((visibility("default")))
#else
#define E2TTT_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { E2TTT_MLP_GELU = 0, E2TTT_SWIGLU = 1 } e2ttt_kind;
typedef enum { E2TTT_F32 = 0, E2TTT_BF16 = 1 } e2ttt_dtype;

/* Which kernel family serves the call.
 *   AUTO    : TCGEN05 where it serves (kind, io_dtype, d, h, C); else TILED for bf16 I/O and SIMT for
 *             fp32 I/O.  The backward has no fused kernel: AUTO and TCGEN05 mean TILED there.
 *             TCGEN05 serves today: GELU-MLP, bf16 I/O, C in {16, 32, 64}, any L (a shorter last chunk), d in {64, 128},
 *             h in {128, 256, 384, 512} (shapes below 128 x 512 and chunks below 64 tokens run zero-padded in
 *             the same tiles); and the SwiGLU forward at d = 128, h = 384, C in {16, 32, 64}, bf16 I/O, without
 *             post-chunk normalisation.  Asked for with TCGEN05 (not chosen by AUTO), both kernels also
 *             run chunks of 128, 256 and 512 tokens (the paper's chunk size) as 2, 4, 8 blocks of 64 at the
 *             chunk-start weights; the GELU-MLP kernel's plain bf16 operands then leave the W1 momentum outside the 2e-2
 *             bound when the gradients of a long chunk cancel (3-4e-2 measured at C = 512)
 *             (its gate / up projection reads the fast weights as two bf16 terms: a plain bf16 copy leaves
 *             some chunks outside the 2e-2 parity bound, the product z1 z2 multiplies the rounding up).
 *   SIMT    : plain CUDA-core kernels for any shape.  With fp32 I/O they compute in fp64
 *             internally; with bf16 I/O in fp32.
 *   TCGEN05 : the fused kernel: bf16 operands on the 5th-generation tensor cores, fp32 accumulation
 *             and the fp32 state in tensor memory for the whole sequence; E2TTT_ERR_SHAPE if it
 *             does not serve the shape.
 *   TILED   : the any-shape kernels of SIMT with every matrix product on the 5th-generation tensor
 *             cores (operands rounded to bf16, fp32 accumulation); intermediates and state stay
 *             fp32 in the workspace.  bf16 I/O only (E2TTT_ERR_SHAPE otherwise). */
typedef enum { E2TTT_IMPL_AUTO = 0, E2TTT_IMPL_SIMT = 1, E2TTT_IMPL_TCGEN05 = 2, E2TTT_IMPL_TILED = 3 } e2ttt_impl;

typedef enum {
    E2TTT_OK = 0,
    E2TTT_ERR_NULL = -1,      /* a required pointer is NULL */
    E2TTT_ERR_SHAPE = -2,     /* non-positive dimension, C > 512, d or h beyond the compiled limits,
                                 L not a multiple of C on a path that needs it, unknown kind */
    E2TTT_ERR_DTYPE = -3,     /* unknown io_dtype / impl */
    E2TTT_ERR_ALIGN = -4,     /* q, k, v, o (and gradients) must be 16-byte aligned */
    E2TTT_ERR_WORKSPACE = -5, /* workspace NULL or smaller than e2ttt_workspace_bytes() */
    E2TTT_ERR_ARCH = -6,      /* current device is not compute capability 10.x */
    E2TTT_ERR_CUDA = -7,      /* the CUDA runtime refused a launch or attribute (no sync is done) */
    E2TTT_ERR_TIMEOUT = -8    /* a bounded device-side wait gave up */
} e2ttt_status;

typedef struct {
    int32_t B, H;     /* batch and heads: B*H independent sequences */
    int32_t L;        /* tokens per sequence */
    int32_t d;        /* head dimension (input and output width of the fast-weight network) */
    int32_t h;        /* hidden width of the fast-weight network */
    int32_t C;        /* chunk size, 1..512 (the paper trains with 512); the fused kernels serve C = 16, 32, 64
                         (and 128, 256, 512 on request).
                         Every path accepts a shorter last chunk (L need not be a multiple of C). */
    int32_t kind;     /* e2ttt_kind */
    int32_t io_dtype; /* e2ttt_dtype of q, k, v, o, d_o, dq, dk, dv */
    float ln_eps;     /* layer-norm epsilon (the paper gives none; 1e-5 is the usual default) */
    int32_t impl;     /* e2ttt_impl */
    int32_t ckpt_every; /* which chunk-start states a forward with save_states keeps for the backward
                         (Section 3.2 leaves the training-time memory plan to the implementation):
                         0 or 1: the state of every chunk (2 * matrices * d * h values per chunk and sequence);
                         n >= 2: only the states of chunks 0, n, 2n, ..; the backward then recomputes the states
                         of n chunks at a time from the nearest checkpoint (one more any-shape forward over the
                         sequence in exchange for ceil(L/C/n) + n + 2 stored states instead of L/C + 1).
                         The forward and the backward of one training step must be given the same value.
                         Not with the *_normed calls (E2TTT_ERR_SHAPE for n >= 2 there). */
} e2ttt_params;

/* Number of fast-weight matrices of a network kind (2 or 3); 0 for an unknown kind. */
E2TTT_API int e2ttt_num_matrices(int kind);

/* Rows and columns of matrix i (0-based) of the collection, Section 4 "Fast-weight Network".
 * Returns E2TTT_ERR_SHAPE for a bad kind or index. */
E2TTT_API int e2ttt_matrix_shape(int kind, int d, int h, int i, int* rows, int* cols);

/* Bytes of caller-provided device workspace a call with these parameters needs.
 * save_states != 0: the size for a forward that also records the chunk-start states (every chunk's, or
 * the checkpoints p->ckpt_every selects plus room for one recomputed segment), and for the backward
 * that consumes them.  `bytes` is a host pointer. */
E2TTT_API int e2ttt_workspace_bytes(const e2ttt_params* p, int save_states, size_t* bytes);

/* Forward over all chunks of all sequences (Algorithm 1 applied chunk after chunk, Section 3.2).
 *   q, k, v          in   [B,H,L,d] io_dtype
 *   eta, beta, gamma in   [B,H,L] fp32: learning rate, momentum factor and decay factor of
 *                         Eq. "tokenwise_ttt_decay_momentum" (the parameterisation that produces
 *                         them, Section 4 "Input-Dependent Dynamics", is the caller's)
 *   W_init           in   host table of device pointers, matrix i [B,H,rows_i,cols_i] fp32
 *   M_init           in   same layout, or NULL for a zero initial momentum
 *   o                out  [B,H,L,d] io_dtype
 *   W_final, M_final out  host tables, same layout as W_init; may alias W_init / M_init
 *   workspace        device scratch of at least e2ttt_workspace_bytes(p, save_states) bytes,
 *                    256-byte aligned; with save_states != 0 it holds, after the call, the
 *                    (W, M) at the start of every chunk for e2ttt_chunk_bwd
 */
E2TTT_API int e2ttt_chunk_fwd(const e2ttt_params* p,
                    const void* q, const void* k, const void* v,
                    const float* eta, const float* beta, const float* gamma,
                    const float* const* W_init, const float* const* M_init,
                    void* o, float* const* W_final, float* const* M_final,
                    void* workspace, size_t workspace_bytes, int save_states, void* stream);

/* Reverse pass of e2ttt_chunk_fwd: the adjoint of the same program (the outer-loop gradient, which
 * the paper's own implementation leaves to automatic differentiation, Appendix "Training Details").
 *   q .. M_init            in   as in the forward
 *   d_o                    in   [B,H,L,d] io_dtype, gradient of the loss w.r.t. o
 *   dW_final, dM_final     in   host tables (fp32, state layout) or NULL for zeros
 *   dq, dk, dv             out  [B,H,L,d] io_dtype
 *   d_eta, d_beta, d_gamma out  [B,H,L] fp32, gradients w.r.t. the three gates as independent inputs
 *   dW_init, dM_init       out  host tables, state layout, fp32; may alias dW_final / dM_final
 *   workspace              sized by e2ttt_workspace_bytes(p, 1)
 *   states_saved           != 0: the workspace still holds the chunk-start states written by
 *                          e2ttt_chunk_fwd(save_states=1) for the same inputs (same p->ckpt_every); 0: they
 *                          are recomputed first, by the fused forward where it serves the shape
 * Both network kinds are supported.  The reverse pass runs on the any-shape kernels (SIMT, or TILED with
 * tensor-core products for bf16 I/O); there is no fused reverse kernel.  With p->ckpt_every >= 2 the call is a
 * sequence of launches on `stream` (per segment: one forward that recomputes its states, one reverse sweep).
 */
E2TTT_API int e2ttt_chunk_bwd(const e2ttt_params* p,
                    const void* q, const void* k, const void* v,
                    const float* eta, const float* beta, const float* gamma,
                    const float* const* W_init, const float* const* M_init,
                    const void* d_o, const float* const* dW_final, const float* const* dM_final,
                    void* dq, void* dk, void* dv, float* d_eta, float* d_beta, float* d_gamma,
                    float* const* dW_init, float* const* dM_init,
                    void* workspace, size_t workspace_bytes, int states_saved, void* stream);

/* The same two calls with post-chunk normalisation of the fast weights (Appendix "Implementation details":
 * L2 normalisation of the fast-weight matrices at each chunk boundary, as a stabiliser).  The paper gives neither
 * the axis nor the target; the reading taken here: after the state transition of every chunk, each row w of each
 * W_i (the weights of one output unit; the momentum is left alone) becomes  n w / (||w||_2 + norm_eps), where n
 * is that row's target norm.  The next chunk starts from, and W_final is, the normalised state, so calls chain.
 *   row_norm    in  (host array of nmat device pointers)  [B,H,rows_i] fp32 targets (rows_i as in
 *                                                          e2ttt_matrix_shape); a model passes the row norms
 *                                                          of its learned initial fast weights
 *   norm_eps    in                                         >= 0
 *   d_row_norm  out (host array of nmat device pointers, or NULL)  adjoints of the targets, [B,H,rows_i] fp32
 * Everything else as in e2ttt_chunk_fwd / e2ttt_chunk_bwd.  The forward runs on the fused tensor-core kernel
 * where that serves the shape (AUTO, TCGEN05), the backward on the any-shape kernels (TCGEN05 means TILED
 * there).  e2ttt_workspace_bytes_normed sizes the workspace for either (the backward always needs the
 * save_states = 1 size).  A backward with states_saved = 1 needs the states of
 * e2ttt_chunk_fwd_normed(save_states = 1) with the same targets. */
E2TTT_API int e2ttt_workspace_bytes_normed(const e2ttt_params* p, int save_states, size_t* bytes);
E2TTT_API int e2ttt_chunk_fwd_normed(const e2ttt_params* p, const void* q, const void* k, const void* v,
                                     const float* eta, const float* beta, const float* gamma,
                                     const float* const* W_init, const float* const* M_init,
                                     const float* const* row_norm, float norm_eps,
                                     void* o, float* const* W_final, float* const* M_final,
                                     void* workspace, size_t workspace_bytes, int save_states, void* stream);
E2TTT_API int e2ttt_chunk_bwd_normed(const e2ttt_params* p, const void* q, const void* k, const void* v,
                                     const float* eta, const float* beta, const float* gamma,
                                     const float* const* W_init, const float* const* M_init,
                                     const float* const* row_norm, float norm_eps,
                                     const void* d_o, const float* const* dW_final, const float* const* dM_final,
                                     void* dq, void* dk, void* dv, float* d_eta, float* d_beta, float* d_gamma,
                                     float* const* dW_init, float* const* dM_init, float* const* d_row_norm,
                                     void* workspace, size_t workspace_bytes, int states_saved, void* stream);

/* Outputs of fixed fast weights, no update: o[b,h,t,:] = f_W(q[b,h,t,:]) for t < p->L  (Algorithm 1 line 1
 * with the weights held fixed; the streaming / decode use of the method).  Between two chunk boundaries every
 * token is answered from the chunk-start weights W_0, and the state changes only when a whole chunk of keys,
 * values and gates has accumulated: that step is e2ttt_chunk_fwd over those C tokens (its `o` equals what this
 * call returned for the same tokens).  So a decoder calls e2ttt_apply per incoming token (p->L = 1) and
 * e2ttt_chunk_fwd once every C tokens.
 *   p        in  (host)    B, H, d, h, kind, io_dtype, ln_eps as above; L = tokens per sequence in this call;
 *                          C and impl are not used but must hold valid values (every field is validated)
 *   q        in  (device)  [B,H,L,d] io_dtype, 16-byte aligned
 *   W        in  (host array of device pointers)  the nmat fast-weight matrices, fp32, shapes as above
 *   o        out (device)  [B,H,L,d] io_dtype, 16-byte aligned
 * Needs no workspace; the work is enqueued on `stream`; nothing is allocated and the host is not synchronised.
 * Arithmetic: fp32 throughout (weights are read as fp32, never rounded).  For a few tokens the call is bound
 * by reading W once: 4 * nmat * d * h bytes per (b, h).
 * Returns E2TTT_OK or E2TTT_ERR_NULL / _SHAPE / _DTYPE / _ALIGN / _ARCH / _CUDA. */
E2TTT_API int e2ttt_apply(const e2ttt_params* p, const void* q, const float* const* W, void* o, void* stream);

/* Token preparation, the step of the model right before the chunk update (Section 4, "Overall Architecture",
 * Eqs. "eta_parameterization", "beta_parameterization", "decay_derivation"):
 *   q = silu(q_raw) / max(||silu(q_raw)||_2, norm_eps)  per token and head, k likewise from k_raw;
 *   eta = eta_base sigmoid(a_eta),  beta = sigmoid(a_beta)^(1/tau),
 *   gamma = 1 - eta * alpha_base sigmoid(a_alpha).
 * The logits a_* are the outputs of the model's small linear heads, which stay with the caller.  (The paper does
 * not say how a zero vector is normalised: the max(., norm_eps) of the common library routine is a reading.)
 *   p        in  (host)    B, H, L, d, io_dtype; the other fields are not used but must hold valid values
 *                          (every field is validated)
 *   g        in  (host)    eta_base > 0, tau > 0, alpha_base >= 0, norm_eps >= 0
 *   q_raw, k_raw      in  (device)  [B,H,L,d] io_dtype
 *   a_eta, a_beta, a_alpha  in (device)  [B,H,L] fp32
 *   q, k     out (device)  [B,H,L,d] io_dtype (may alias q_raw, k_raw)
 *   eta, beta, gamma  out (device)  [B,H,L] fp32: what e2ttt_chunk_fwd takes
 * e2ttt_prepare_bwd gives the adjoints of q_raw, k_raw and the three logits from those of q, k, eta, beta,
 * gamma (what e2ttt_chunk_bwd returns); it re-reads the forward's inputs and needs none of its outputs.
 * Arithmetic in fp32; no workspace; enqueued on `stream`; HBM-bound (every byte read once, written once).
 * These two kernels take no workspace and therefore have no device status word: their bounded waits guard bulk
 * loads, which cannot fail short of a device fault (and that the next runtime call reports).
 * Returns E2TTT_OK or E2TTT_ERR_NULL / _SHAPE / _DTYPE / _ARCH / _CUDA. */
typedef struct {
    float eta_base, tau, alpha_base, norm_eps;
} e2ttt_gate_params;
E2TTT_API int e2ttt_prepare_fwd(const e2ttt_params* p, const e2ttt_gate_params* g, const void* q_raw,
                                const void* k_raw, const float* a_eta, const float* a_beta, const float* a_alpha,
                                void* q, void* k, float* eta, float* beta, float* gamma, void* stream);
E2TTT_API int e2ttt_prepare_bwd(const e2ttt_params* p, const e2ttt_gate_params* g, const void* q_raw,
                                const void* k_raw, const float* a_eta, const float* a_beta, const float* a_alpha,
                                const void* dq, const void* dk, const float* d_eta, const float* d_beta,
                                const float* d_gamma, void* dq_raw, void* dk_raw, float* da_eta, float* da_beta,
                                float* da_alpha, void* stream);

/* Reads back the device status word of the last launch that used `workspace` (the first word of every
 * workspace).  workspace == NULL reads the word of the scratch array e2ttt_chunk_fwd_noalloc uses on the
 * current device (0 if that entry point has not run there yet).  This is the one entry point that
 * synchronises: it waits for `stream`.
 *   status  out (host)  0 after a clean run; otherwise the code of the first bounded device-side wait
 *                       that gave up (the tensor-core kernels never spin without a limit)
 * Returns E2TTT_OK, E2TTT_ERR_TIMEOUT when the word is non-zero, or E2TTT_ERR_NULL / E2TTT_ERR_CUDA.
 * (No counterpart in the paper: an operational guard of this implementation.) */
E2TTT_API int e2ttt_device_status(const void* workspace, void* stream, int* status);

/* Forward without any caller-provided scratch.  (The paper has no counterpart: this exists for the
 * library's users, not for the method.)
 *
 * Who needs it: code that runs where asking the CUDA runtime for device memory is off the table -
 * a plugin handed only its input and output buffers by a host application that owns the memory
 * pool, a real-time loop that must not touch the allocator after start-up, a process whose memory
 * budget was fixed and spent before this call.  Such callers cannot size and allocate the workspace
 * e2ttt_chunk_fwd asks for.
 *
 * Same arguments and results as e2ttt_chunk_fwd(save_states = 0), minus the workspace.  The scratch
 * is a fixed array of E2TTT_NOALLOC_SCRATCH_BYTES inside the library's device image, so every GPU
 * that loads the library gives up that much memory until the process exits.  A call whose
 * e2ttt_workspace_bytes(p, 0) exceeds it returns E2TTT_ERR_WORKSPACE and launches nothing (with fp32
 * I/O the benchmark's tiny configuration, B*H = 1, d = 64, h = 256, C = 16, needs about 0.8 MiB;
 * bf16 I/O needs half as much per sequence).  The call itself allocates and frees nothing.
 *
 * The first call on each device looks up the array's device address (one runtime query, with that
 * device current) and remembers it; make that first call outside any stream capture.
 * All calls on a device share the one array.  It keeps whatever the previous call left there, which
 * is harmless: the kernel writes every scratch word before reading it, nothing has to start at
 * zero.  But two calls that run on the GPU at the same time (different streams, or different host
 * threads) would overwrite each other's intermediates: serialise them.
 */
#define E2TTT_NOALLOC_SCRATCH_BYTES (8u << 20)
E2TTT_API int e2ttt_chunk_fwd_noalloc(const e2ttt_params* p,
                    const void* q, const void* k, const void* v,
                    const float* eta, const float* beta, const float* gamma,
                    const float* const* W_init, const float* const* M_init,
                    void* o, float* const* W_final, float* const* M_final, void* stream);

/* Self-test of the device-side failure path, in a form that fails nothing: one CTA waits, for at most
 * `limit_cycles` SM cycles (1 .. 2e9), on a barrier that nobody signals.  The bounded wait runs out, the kernel
 * records its code in the status word of `workspace` (at least 256 bytes, 256-byte aligned, device) and
 * returns; e2ttt_device_status(workspace, ...) then reports E2TTT_ERR_TIMEOUT with a non-zero word, exactly as
 * it would after a real stall.  Nothing traps or hangs and the context stays usable.
 * (No counterpart in the paper: an operational guard of this implementation.)
 * Returns E2TTT_OK (the kernel was enqueued) or E2TTT_ERR_NULL / _WORKSPACE / _ALIGN / _SHAPE / _ARCH / _CUDA. */
E2TTT_API int e2ttt_selftest_wait_timeout(void* workspace, size_t workspace_bytes, long long limit_cycles, void* stream);

/* Static description of a status code (never NULL). */
E2TTT_API const char* e2ttt_status_string(int status);

/* Library version, major*10000 + minor*100 + patch. */
E2TTT_API int e2ttt_version(void);

#ifdef __cplusplus
}
#endif
#endif /* E2TTT_H */
