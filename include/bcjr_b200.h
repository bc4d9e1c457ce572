/*
 * bcjr_b200 -- C ABI of the B200 (sm_100a) BCJR soft-quantisation library.
 *
 * One weight block w[0..n) is encoded by a path through a bitshift trellis with S = 2^Lb
 * states: from state s the k input bits b lead to s' = ((s << k) | b) mod S, and state s
 * emits the scalar codebook[s]  (paper Section 3.1).  All calls treat `num_blocks`
 * independent blocks stored back to back (block i = W[i*n .. i*n+n), i.e. a row-major
 * matrix whose rows are cut into consecutive blocks of n).
 *
 * Conventions shared by every entry point
 *   - "device" pointers are CUDA device memory of the context's device, caller-owned; the
 *     library never frees or reallocates them.  "host" pointers are ordinary host memory.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*, NULL = the
 *     default stream) unless stated otherwise.  The context owns its scratch memory; it
 *     grows on demand (cudaMalloc on the calling thread) and is reused by later calls, so
 *     two calls on one context must not overlap on the GPU.
 *   - Every call returns a bcjr_status; nothing throws, aborts or traps.
 *   - The first state is free and the last state is free (no tail biting); the
 *     log-potential of state s at step t is  -(w_t - codebook[s])^2 / (2 T)  (Eq. 4).
 */
#ifndef BCJR_B200_H
#define BCJR_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bcjr_ctx bcjr_ctx;

typedef enum {
    BCJR_OK = 0,
    BCJR_EINVAL = -1,        /* bad argument (NULL pointer, dims out of range, T <= 0, ...) */
    BCJR_ENOMEM = -2,        /* scratch allocation failed */
    BCJR_ECUDA = -3,         /* a CUDA runtime call failed; see bcjr_last_cuda_error */
    BCJR_ESTATE = -4,        /* bcjr_backward without a preceding bcjr_soft_quantize */
    BCJR_EUNSUPPORTED = -5,  /* (Lb, k) combination the kernels do not cover */
    BCJR_ETIMEOUT = -6,      /* a bounded device-side wait gave up (reported by bcjr_sync_status) */
    BCJR_ENUMERIC = -7,      /* non-finite values met on the device */
    BCJR_ETOOLARGE = -8      /* problem does not fit the fixed scratch of bcjr_soft_quantize_static */
} bcjr_status;

/* Diagnostics gathered on the device since the last bcjr_sync_status. */
typedef struct {
    int32_t device_status;        /* BCJR_OK or the first device-side error */
    float max_posterior_defect;   /* max over blocks and steps of |sum_s gamma_t(s) - 1| (Eq. 6) */
    float max_logz_mismatch;      /* max |log Z (alpha side) - log Z (beta side)|, natural log */
    int32_t kernel_launches;      /* kernels launched by this context since creation */
    int32_t last_path;            /* kernels used by the last call: 0 = generic, 1 = large-trellis (Lb = 16), 2 = one warp per block (Lb = 11..13, k = 2) */
} bcjr_diag;

/* Limits: 1 <= k <= 4, k <= Lb <= 16, Lb - k <= 14, n >= 1, T > 0 and finite.
 *
 * Which kernel serves a shape (all give the same results within float32 tolerance; speed differs):
 *   Lb = 16, k = 2 or 3:  tensor-memory kernels.  Forward and Viterbi for n <= 2048 / 4096; backward
 *                         for n <= 1024.  Longer blocks step down: backward 1024 < n <= 2048 runs the
 *                         four-CTA register kernel (about 1.7x slower per weight), and anything longer
 *                         the generic one-CTA kernels (more than 10x slower per weight at Lb = 16).
 *   Lb = 11..13, k = 2:   one warp per block, sixteen (forward) or eight (backward) blocks per SM at Lb = 12, table in
 *                         tensor memory; any n.  The backward call with grad_codebook at Lb = 12, 13 gives a block to
 *                         two warps ("bwd_variant" = 1: one warp).
 *   V = 2, Lb = 16, k = 2: forward on clusters of two CTAs (n <= 2048), backward on clusters of four (table and
 *                         gradient accumulators are 1 MB of tensor memory; n <= 1024); longer blocks and every
 *                         other V = 2 shape run the one-CTA vector kernels.
 *   everything else:      generic kernels, one CTA per block (also "path" = 1).
 * Block lengths of a few hundred weights (the paper uses 256) are the intended range. */

/* Creates a context bound to CUDA device `device_ordinal`.  *out is owned by the caller
 * and released with bcjr_destroy.  Synchronous. */
bcjr_status bcjr_create(bcjr_ctx **out, int device_ordinal);

/* Frees the context and its scratch memory (synchronises the device first). */
bcjr_status bcjr_destroy(bcjr_ctx *ctx);

/* Tuning / test hooks.
 *   "path"        0 auto, 1 force the generic kernels, 2 force the large-trellis kernels
 *                 (BCJR_EUNSUPPORTED at call time when they do not cover the shape)
 *   "fwd_variant" large-trellis forward kernel: 0 = one CTA per block with the codebook in tensor
 *                 memory (Lb = 16, k = 2 or 3), 1 = two-CTA cluster kernel with the codebook in registers.
 *                 Vector emissions (V = 2, Lb = 16, k = 2): 0 = clusters of two CTAs (the table whole in two
 *                 tensor memories, all SMs), 1 = clusters of four (the backward kernel's shape)
 *   "bwd_variant" large-trellis backward call (Lb = 16, k = 2 or 3).  0 (default): with grad_codebook, two
 *                 kernels per chunk of as many blocks as the GPU has SMs -- the alpha sweeps on one CTA per
 *                 block, then the beta sweeps on two-CTA clusters with codebook and gradient accumulators in
 *                 tensor memory; without grad_codebook at k = 2, one kernel with both sweeps on one CTA per
 *                 block.  1 = four-CTA clusters, registers.  2 = one two-CTA tensor-memory kernel for both
 *                 sweeps, one cluster barrier per step.  3 = the same with the butterflies ordered so that a
 *                 step starts before the whole cluster has finished the previous one (k = 2; k = 3 as 2).
 *                 4 = as 0, but the two-kernel call also without grad_codebook.
 *   "history_every_m"  1 (default): the large-trellis forward kernel stores the forward messages of every step
 *                 for its beta sweep; m = 2..16: it keeps them for every m-th step only and recomputes the
 *                 m - 1 steps in between inside the beta sweep (1/m of the history traffic to HBM for
 *                 (m-1)/m of an alpha sweep more arithmetic; same results within float32 rounding; Lb = 16, k = 2,
 *                 n <= 512, otherwise the option has no effect)
 *   "max_ctas"    cap on resident thread blocks (0 = fill the GPU)
 *   "record_block_defect"  1: every scalar forward call also records, per block, max over steps of
 *                 |sum_s gamma_t(s) - 1| (read back with bcjr_block_defects); 0 (default): only the
 *                 maximum over the call is kept (bcjr_diag)
 *   "wait_limit_ms"  wall-time budget of one device-side wait (default 2000).  A wait that outlasts it
 *                 gives up: the kernel still runs to its end, the outputs of the call are
 *                 meaningless and bcjr_sync_status returns BCJR_ETIMEOUT; the context stays usable.
 *   "debug_drop_history_load"  test hook for that path: while non-zero, one warp of thread block 0
 *                 withholds one arrival in a large-trellis backward call, so the waits of its cluster
 *                 must run out.
 * The last two synchronise the device before they take effect. */
bcjr_status bcjr_set_option(bcjr_ctx *ctx, const char *name, int64_t value);

/*
 * Soft codeword (Eq. 3 / Eq. 7): soft[t] = sum_s codebook[s] * p_T(s_t = s | w), with the
 * marginals from the temperature-T forward-backward recursions of Eq. 5-6 carried in the
 * log domain.
 *   W         device in   [num_blocks * n] float32
 *   codebook  device in   [2^Lb] float32, or NULL for the computed Gaussian emission of Section 3.1,
 *                         codebook[s] = Phi^-1((s + 1/2) / 2^Lb) (what bcjr_gaussian_codebook writes out): at
 *                         Lb = 16, k = 2 or 3 the kernels then evaluate the entries themselves while filling
 *                         their tensor-memory slices and no table is read; other shapes use a table the
 *                         context keeps.  viterbi_hard and bcjr_ste_forward take NULL the same way.
 *   soft      device out  [num_blocks * n] float32
 *   logZ      device out  [num_blocks] float32, natural log of Z_T per block (sum over legal
 *                         paths of exp(-E/T), no prior constant); may be NULL
 * Saves, for bcjr_backward: the W and codebook POINTERS (borrowed: keep them valid and
 * unchanged until the matching bcjr_backward has been enqueued), the dims, T, and a private
 * copy of `soft`.
 */
bcjr_status bcjr_soft_quantize(bcjr_ctx *ctx, const float *W, const float *codebook,
                               int Lb, int k, int n, int64_t num_blocks, float T,
                               float *soft, float *logZ, void *cuda_stream);

/*
 * Backward pass of the autograd node of Section 3.5 for l = sum(grad_soft * soft), T held
 * constant: the exact derivative of Eq. 7 through both recursions.
 *   grad_soft      device in   [num_blocks * n]
 *   grad_W         device out  [num_blocks * n]
 *   grad_codebook  device out  [2^Lb], OVERWRITTEN with the sum over all blocks (direct term
 *                  through the emitted value plus the term through the energies); may be NULL: the table is
 *                  then treated as fixed, as in the paper's experiments, and the 2^16-state kernel runs
 *                  without its accumulator half.  Must be NULL after a forward call with a NULL codebook
 *                  (BCJR_EINVAL otherwise: a computed emission has no table to differentiate).
 * Uses the state saved by the last bcjr_soft_quantize on this context; BCJR_ESTATE if none.
 */
bcjr_status bcjr_backward(bcjr_ctx *ctx, const float *grad_soft,
                          float *grad_W, float *grad_codebook, void *cuda_stream);

/*
 * Viterbi hard code (Section 3.2): the legal path minimising sum_t (w_t - codebook[s_t])^2.
 * Path metrics are accumulated in IEEE double, d = (double)w - (double)c, m += d*d, without
 * fused multiply-add; ties go to the lowest predecessor and the lowest final state.
 *   path_bits  device out  [num_blocks * path_stride_bytes]; per block Lb + k(n-1) bits, most
 *              significant first: s_1 in Lb bits, then the k input bits of every later step;
 *              bit i is stored in byte i>>3 at bit position 7-(i&7); padding bits are zero.
 *              path_stride_bytes >= ceil((Lb + k(n-1)) / 8).  May be NULL.
 *   states     device out  [num_blocks * n] uint16 state sequence; may be NULL
 *   hard       device out  [num_blocks * n] float32, exact copies of codebook entries; may be NULL
 */
bcjr_status viterbi_hard(bcjr_ctx *ctx, const float *W, const float *codebook,
                         int Lb, int k, int n, int64_t num_blocks,
                         uint8_t *path_bits, int64_t path_stride_bytes,
                         uint16_t *states, float *hard, void *cuda_stream);

/*
 * Vector emissions (the paper's "L=16, k=2, V=2" configuration, Section 3.1 and Section 4
 * "Quantization configuration"; its kernel section's 128-step, 16-predecessor recursion): every
 * state emits V numbers, a trellis step consumes V weights and k*V input bits,
 *     s' = ((s << kV) | b) mod 2^Lb,   e_t(s) = -(1/(2T)) sum_v (w[V t + v] - codebook[s*V + v])^2,
 *     soft[V t + v] = sum_s codebook[s*V + v] gamma_t(s).
 * The paper writes only the scalar emission; this vector form is the reading taken here.
 *   codebook   device in  [2^Lb * V], row s = the V numbers state s emits
 *   n          weights per block, a multiple of V (n / V trellis steps)
 *   k, V       V = 1 forwards to the scalar call; V = 2 with k = 1 or 2 is supported, anything else
 *              returns BCJR_EUNSUPPORTED.  With V = 2 every array must be 8-byte aligned (BCJR_EINVAL).
 * A following bcjr_backward then expects/returns grad_codebook as [2^Lb * V].
 * viterbi_hard_vec: states [num_blocks * n/V] uint16, hard [num_blocks * n] (the emitted numbers),
 * path bits Lb + kV (n/V - 1) per block in the layout of viterbi_hard; squared error summed over
 * the V components in IEEE double, components added in order, no fused multiply-add.
 * Otherwise as bcjr_soft_quantize / viterbi_hard.
 */
bcjr_status bcjr_soft_quantize_vec(bcjr_ctx *ctx, const float *W, const float *codebook,
                                   int Lb, int k, int V, int n, int64_t num_blocks, float T,
                                   float *soft, float *logZ, void *cuda_stream);
bcjr_status viterbi_hard_vec(bcjr_ctx *ctx, const float *W, const float *codebook,
                             int Lb, int k, int V, int n, int64_t num_blocks,
                             uint8_t *path_bits, int64_t path_stride_bytes,
                             uint16_t *states, float *hard, void *cuda_stream);

/*
 * The steps on either side of the trellis pass in the per-layer QAT loop (Algorithm 1).
 *
 * bcjr_temperature: the annealing schedule of Section 3.6, T_t = T_0 (T_end / T_0)^(t / N_steps)
 *   (host arithmetic; t = 0 gives T_0, t = N_steps gives T_end; 0.0 on invalid arguments).
 * bcjr_gaussian_codebook: the computed Gaussian emission of Section 3.1 written out as a table,
 *   codebook[s] = Phi^-1((s + 1/2) / 2^Lb), s = 0 .. 2^Lb - 1 (device out).  The paper's "incoherent
 *   permutation" of this table is not specified and is not applied.
 * bcjr_adam_update: one Adam step (the update Algorithm 1 applies to the continuous pre-image) on a
 *   device array, in place: m, v are the moment buffers (device, same size, zero before step 1),
 *   t >= 1 the step number; bias-corrected.  All four arrays 16-byte aligned (BCJR_EINVAL otherwise).
 * bcjr_backward_adam: bcjr_backward into context-owned gradient buffers followed by the Adam step
 *   on W_latent (which must be the W given to the last forward call on this context) and, when
 *   `codebook` is not NULL (then it must be that call's codebook), on the table with step size lr_c.
 *   The saved forward state is consumed: the next bcjr_backward needs a new forward call.
 * The paper has the loss of Algorithm 1 (layer output against the teacher's) outside these calls:
 * the caller turns the soft codeword into grad_soft.
 */
double bcjr_temperature(double T0, double T_end, int t, int n_steps);
bcjr_status bcjr_gaussian_codebook(bcjr_ctx *ctx, int Lb, float *codebook, void *cuda_stream);
bcjr_status bcjr_adam_update(bcjr_ctx *ctx, float *param, const float *grad, float *m, float *v,
                             int64_t numel, int t, float lr, float beta1, float beta2, float eps,
                             void *cuda_stream);
bcjr_status bcjr_backward_adam(bcjr_ctx *ctx, const float *grad_soft, float *W_latent, float *m_W, float *v_W,
                               float *codebook, float *m_c, float *v_c, int t, float lr_W, float lr_c,
                               float beta1, float beta2, float eps, void *cuda_stream);

/*
 * Incoherence processing before / after the trellis pass (Section 3.1: "a random-sign Hadamard
 * rotation on both sides"; Section 4, "Quantization configuration": scales over groups of 16).
 * The paper gives no formulas; these calls use
 *     forward:  out = H_m diag(sign_rows) W diag(sign_cols) H_n / sqrt(m n)
 *     inverse:  out = diag(sign_rows) H_m W H_n diag(sign_cols) / sqrt(m n)
 * with Sylvester-ordered Walsh-Hadamard matrices (H H = size * I), so inverse(forward(W)) = W, and
 *     scales[g] = sqrt(mean of the squares of elements 16g .. 16g+15),  W_scaled = W / scales[g]
 *     (a group of zeros gets scale 0 and stays zero).
 *   W, out      device [m * n] row-major; out may be W (in place); 16-byte aligned
 *   m, n        powers of two, >= 8; n <= 8192 (BCJR_EUNSUPPORTED above)
 *   sign_rows   device [m], sign_cols device [n]: +1.0f / -1.0f (sign_cols 16-byte aligned)
 *   numel       multiple of 16; scales has numel / 16 entries
 */
bcjr_status bcjr_rht(bcjr_ctx *ctx, const float *W, float *out, int m, int n,
                     const float *sign_rows, const float *sign_cols, int inverse, void *cuda_stream);
bcjr_status bcjr_group_scale(bcjr_ctx *ctx, const float *W, float *scales, float *W_scaled,
                             int64_t numel, void *cuda_stream);
bcjr_status bcjr_group_unscale(bcjr_ctx *ctx, const float *W_scaled, const float *scales, float *W,
                               int64_t numel, void *cuda_stream);

/*
 * BCJR-STE forward (Section 3.8, "BCJR-STE variant"): the value that goes forward is the hard
 * Viterbi codeword, while the state saved on the context is that of the temperature-T relaxation,
 * so that a following bcjr_backward returns the gradient of the finite-temperature soft codeword
 * (the straight-through gradient replaced by the true gradient of the relaxation).  Equivalent
 * to bcjr_soft_quantize followed by viterbi_hard on the same inputs.
 *   hard    device out  [num_blocks * n] exact copies of codebook entries (required)
 *   states  device out  [num_blocks * n] uint16, may be NULL
 *   soft    device out  [num_blocks * n] soft codeword at T, may be NULL (kept internally only)
 * Same argument checks, borrowing rules and error behaviour as the two calls it is made of.
 */
bcjr_status bcjr_ste_forward(bcjr_ctx *ctx, const float *W, const float *codebook,
                             int Lb, int k, int n, int64_t num_blocks, float T,
                             float *hard, uint16_t *states, float *soft, void *cuda_stream);

/*
 * One training-style step with HOST buffers (pinned or pageable): copies W, codebook and
 * grad_soft to the device, runs bcjr_soft_quantize and bcjr_backward, and copies soft,
 * grad_W and grad_codebook back, all on `cuda_stream`; returns after the stream has been
 * synchronised.  Any of soft / grad_W / grad_codebook may be NULL (not copied back).
 */
bcjr_status bcjr_step_host(bcjr_ctx *ctx, const float *W_host, const float *codebook_host,
                           const float *grad_soft_host, int Lb, int k, int n, int64_t num_blocks,
                           float T, float *soft_host, float *grad_W_host, float *grad_codebook_host,
                           void *cuda_stream);

/* Synchronises `cuda_stream`, then reports and clears the device-side status and
 * diagnostics.  Returns the device status (BCJR_OK when clean). */
bcjr_status bcjr_sync_status(bcjr_ctx *ctx, void *cuda_stream, bcjr_diag *out);

/* Per-block posterior defect of the last bcjr_soft_quantize made while "record_block_defect" was 1
 * (Eq. 6: the marginals of a step sum to one; the deviation measures the float32 rounding a block's
 * messages have accumulated).  Synchronises `cuda_stream`, then copies the first `count` values
 * (count <= that call's num_blocks, else BCJR_ESTATE) to host_out (host, float32).  A block the
 * kernel in use does not instrument reads NaN (the register-table cluster variant, vector emissions). */
bcjr_status bcjr_block_defects(bcjr_ctx *ctx, float *host_out, int64_t count, void *cuda_stream);

/* Scratch bytes currently held by the context. */
int64_t bcjr_workspace_bytes(const bcjr_ctx *ctx);

/* Text of the last CUDA error seen by this context ("" if none). Owned by the context. */
const char *bcjr_last_cuda_error(const bcjr_ctx *ctx);

const char *bcjr_status_string(bcjr_status status);

/*
 * bcjr_soft_quantize_static -- the forward call for callers that cannot allocate.
 * (The paper has no counterpart: this is a packaging of bcjr_soft_quantize, not a step of the
 * method.)
 *
 * Some callers may not call cudaMalloc or cudaFree at all: a latency-critical host loop that
 * cannot afford the device-wide synchronisation those calls imply, a process whose device
 * memory was handed to another allocator up front, a plug-in that may only launch work on the
 * buffers it is given.  This entry point computes what bcjr_soft_quantize computes (the same
 * soft codeword and log Z within float32 tolerance; it always runs the one-CTA-per-block
 * generic kernel, also for the shapes where bcjr_soft_quantize picks a tensor-memory kernel,
 * so the two are not bit-identical there) but needs no context and never allocates or frees:
 * its scratch is a fixed array of BCJR_STATIC_SCRATCH_BYTES that is part of the library image
 * on every GPU that loads the library, for the life of the process.
 *
 *   W, codebook, soft, logZ, cuda_stream: as for bcjr_soft_quantize (device pointers of the
 *   CURRENT device; logZ may be NULL).  Nothing is saved for a backward pass.
 *
 * Limits: the messages must fit shared memory (Lb - k <= 14) and one block's history must fit
 * the scratch: n * 2^(Lb-k) * 4 + (n+2) * 4 bytes (rounded up to 256) <= BCJR_STATIC_SCRATCH_BYTES
 * - 256.  Larger problems are refused with BCJR_ETOOLARGE before anything is launched.  The
 * number of blocks is unlimited; the scratch caps how many thread blocks run at once: at
 * Lb = 16, k = 2, n = 256 one block's history is 16 MiB, so a single thread block works through
 * all blocks in turn (one SM of the GPU); at Lb = 12 the same scratch feeds 127 thread blocks.
 * Throughput-critical callers that can allocate should use bcjr_soft_quantize.
 *
 * Not reported: there is no context to query, so device-side diagnostics (a non-finite input
 * that bcjr_sync_status would report as BCJR_ENUMERIC, the posterior defect) are not available
 * from this call; a block with non-finite input yields non-finite output for that block only.
 *
 * Set-up: the first call on each device looks up the device address of the scratch array
 * (once, under a lock; that device must be current, as it is for the call itself).  Make that
 * first call outside any stream capture.
 *
 * Sharing: all calls on a device use the same scratch, and it keeps the previous call's
 * contents (the part that must start from zero is cleared on the stream at each call).  Calls
 * whose kernels could overlap on the GPU -- different streams, or different host threads
 * without ordering -- race on it: order them on one stream or with events.
 */
#define BCJR_STATIC_SCRATCH_BYTES (32u << 20)
bcjr_status bcjr_soft_quantize_static(const float *W, const float *codebook, int Lb, int k, int n,
                                      int64_t num_blocks, float T, float *soft, float *logZ,
                                      void *cuda_stream);

/* Size in bytes of the fixed scratch array behind bcjr_soft_quantize_static. */
int64_t bcjr_static_scratch_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* BCJR_B200_H */
