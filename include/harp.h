/* harp.h -- C ABI of the B200 (sm_100a) HARP apply library.
 *
 * A HARP processor is the orthogonal map (row-vector convention, y = x Q)
 *
 *     Q = D_s . Pi . T,      T = M_0 . M_1 ... M_{m-1}
 *
 * D_s : Rademacher sign diagonal (paper, Section "HARP processors": sign flips as in
 *       RHT preprocessing; Assumption 1(d): applied as diagonal matrices).
 * Pi  : a fixed permutation, applied as a gather v_i = u_{perm[i]} (the "fixed
 *       permutation convention" of Theorem 1).
 * M_t : stride stage t of Eq. 7 with the Mixed-Radix schedule of Eq. 6:
 *       s_t = prod_{j<t} b_j, g = d/(b_t s_t); for every (alpha < g, beta < s_t) the b_t
 *       coordinates {alpha b_t s_t + r s_t + beta : r < b_t} (Lemma 1) are multiplied on
 *       the right by block kernel K_t[c], c = alpha s_t + beta:
 *           out[base + j s_t] = sum_i in[base + i s_t] * K_t[c][i][j].
 *       Stage 0 (stride 1) is applied first (Algorithm 1, Eq. 8).
 *
 * All functions return a status, never throw and never abort; nothing is launched on
 * invalid input.  Pointers are marked HOST or DEVICE.  Device buffers are caller-owned and
 * contiguous row-major; results overwrite the input.  A buffer must be aligned to its
 * element size (else HARP_ERR_BAD_DIM); the fast kernels additionally need a 16-byte
 * aligned base, and a call that lacks it runs on the generic kernel.
 * The library never falls back to a CPU path: unsupported shapes return
 * HARP_ERR_UNSUPPORTED.
 */
#ifndef HARP_H_
#define HARP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct harp_plan harp_plan_t; /* opaque; immutable after create */

typedef enum {
    HARP_OK = 0,
    HARP_ERR_NULL = 1,          /* a required pointer is NULL                         */
    HARP_ERR_BAD_DIM = 2,       /* d < 2, n_rows < 0, or d too large                  */
    HARP_ERR_BAD_SCHEDULE = 3,  /* n_stages < 1, a radix < 2, or prod(radices) != d   */
    HARP_ERR_BAD_PERM = 4,      /* perm is not a bijection of 0..d-1                  */
    HARP_ERR_BAD_SIGNS = 5,     /* a sign is not +1 or -1                             */
    HARP_ERR_BAD_DTYPE = 6,
    HARP_ERR_DIM_MISMATCH = 7,
    HARP_ERR_UNSUPPORTED = 8,   /* valid input this build has no kernel for           */
    HARP_ERR_ALLOC = 9,         /* host or device allocation failed                   */
    HARP_ERR_CUDA = 10,         /* a CUDA runtime call or launch failed               */
    HARP_ERR_TOO_LARGE = 11     /* exceeds a documented fixed capacity                */
} harp_status_t;

typedef enum { HARP_F32 = 0, HARP_BF16 = 1 } harp_dtype_t;

/* Kernel families; HARP_KERNEL_AUTO lets the library choose. */
typedef enum {
    HARP_KERNEL_AUTO = 0,
    HARP_KERNEL_GENERIC = 1,   /* CUDA cores, any plan                                   */
    HARP_KERNEL_FAST = 2,      /* tensor cores, whole rows per CTA                       */
    HARP_KERNEL_SPLIT = 3,     /* tensor cores, two passes over column groups (wide rows) */
    HARP_KERNEL_TMEM = 4       /* tcgen05.mma, 128 rows per tile, operands in tensor memory */
} harp_kernel_t;

/* Build a processor (Eq. 6-9 of the paper; Algorithm 1 lines 2 and 7-8 for the stride
 * and block-kernel layout).
 *   out      HOST  receives the plan; untouched on error
 *   d        transformed dimension, 2 <= d <= 2^20 (plans are built for any such d; whether a kernel
 *            exists for it is decided per call: fp32 or permuted rows beyond d = 32768 and bf16 rows
 *            no tensor-core path takes return HARP_ERR_UNSUPPORTED from harp_apply)
 *   n_stages m >= 1;  radices HOST int32[m], each >= 2, product == d
 *   perm     HOST int32[d] bijection, forward gathers v[i] = u[perm[i]]; NULL = identity
 *   signs    HOST int8[d] with entries +1/-1;  NULL = all +1
 *   blocks   HOST array of m pointers; blocks[t] = float[d/b_t][b_t][b_t] row-major
 * Every host array is copied; the plan owns its device copies on the current CUDA
 * device.  Orthogonality of the blocks is not checked: the library applies what it is
 * given.  Validation happens before the first CUDA call. */
harp_status_t harp_plan_create(harp_plan_t **out, int64_t d, int32_t n_stages,
                               const int32_t *radices, const int32_t *perm,
                               const int8_t *signs, const float *const *blocks);

/* Greedy Mixed-Radix schedule (Algorithm 2, appendix "Stage schedules and Mixed-Radix
 * construction"): peel the preferred radix b_base while it divides d, then the largest factors
 * <= b_max down to 2, then the leftover factor as one last stage.
 *   radices  HOST int32[max_stages], receives the schedule
 * Returns the number of stages, or -1 (d < 2, a radix bound < 2, NULL, or max_stages too small). */
int32_t harp_greedy_schedule(int64_t d, int32_t b_base, int32_t b_max, int32_t *radices,
                             int32_t max_stages);

/* Parameters per block of radix b: 1 (Givens angle) for b = 2, b(b-1)/2 (strict upper triangle of
 * the skew-symmetric matrix A, row-major, i < j) otherwise (Eq. 10, 11, 13). */
int32_t harp_theta_params_per_block(int32_t b);

/* Block kernels of one stage from stored parameters, B_c = Q(theta_c) G_b (Eq. 9): Q is the Givens
 * rotation [[cos,-sin],[sin,cos]] for b = 2 (Eq. 10) and the Cayley map (I+A)^{-1}(I-A) for b > 2
 * (Eq. 11).  All pointers HOST; no CUDA call is made.
 *   theta     float[n_blocks][n_par] or NULL
 *   theta_q   int8[n_blocks][n_par] with scales float[n_blocks] (int8 storage of the appendix:
 *             a = scale * q), used when theta is NULL
 *   mixer     float[b][b] orthogonal base mixer G_b, or NULL for the normalised Sylvester Hadamard
 *             matrix (b a power of two; otherwise HARP_ERR_NULL)
 *   out_blocks float[n_blocks][b][b], the layout harp_plan_create expects
 * Arithmetic in fp64, one rounding to fp32. */
harp_status_t harp_blocks_from_theta(int32_t b, int64_t n_blocks, const float *theta,
                                     const int8_t *theta_q, const float *scales,
                                     const float *mixer, float *out_blocks);

/* The same reconstruction on the GPU (Section "Parameter quantization for deployment", appendix "Int8
 * storage of HARP parameters": the orthogonal block is rebuilt from the stored angles / upper triangle
 * at runtime).  Every pointer is DEVICE memory on the current device, with the layouts of
 * harp_blocks_from_theta; one thread block per matrix block solves (I + A) Q = I - A in fp64 (Gauss-
 * Jordan with partial pivoting in shared memory) and multiplies by the mixer, one rounding to fp32.
 * b <= harp_theta_device_max_radix() (54), else HARP_ERR_UNSUPPORTED.  Asynchronous on stream;
 * allocates nothing. */
harp_status_t harp_blocks_from_theta_device(int32_t b, int64_t n_blocks, const float *theta,
                                            const int8_t *theta_q, const float *scales,
                                            const float *mixer, float *out_blocks, void *stream);
int32_t harp_theta_device_max_radix(void);

/* Gradient with respect to the stored parameters of one stage, given the gradient with respect to
 * its block kernels (harp_grad_blocks, copied to the host): the chain rule through B_c = Q(theta_c) G_b
 * (Eq. 9-11), i.e. what the parameter update of Algorithm 3 needs.  All pointers HOST; no CUDA call.
 *   theta       float[n_blocks][n_par], the point at which the blocks were built
 *   mixer       as in harp_blocks_from_theta
 *   grad_blocks float[n_blocks][b][b] = dL/dB_c
 *   grad_theta  float[n_blocks][n_par] = dL/dtheta_c (overwritten)
 * Arithmetic in fp64, one rounding to fp32.  HARP_ERR_BAD_SCHEDULE if I + A is singular. */
harp_status_t harp_grad_theta(int32_t b, int64_t n_blocks, const float *theta, const float *mixer,
                              const float *grad_blocks, float *grad_theta);

/* harp_plan_create with every stage's blocks rebuilt from the stored parameters: by the device
 * kernels of harp_blocks_from_theta_device for radices they take, by harp_blocks_from_theta otherwise.  theta, theta_q,
 * scales, mixers are HOST arrays of n_stages pointers (theta or theta_q may be NULL as a whole;
 * mixers may be NULL if every radix is a power of two). */
harp_status_t harp_plan_create_from_theta(harp_plan_t **out, int64_t d, int32_t n_stages,
                                          const int32_t *radices, const int32_t *perm,
                                          const int8_t *signs, const float *const *theta,
                                          const int8_t *const *theta_q,
                                          const float *const *scales,
                                          const float *const *mixers);

/* Kronecker fallback (Eq. 12): the plan of dimension d = K * n2 equal to
 * (H~_K / sqrt K) (x) T_{n2}: the stages of the n2-plan act on each of the K contiguous runs of n2
 * coordinates, then one radix-K stage of stride n2 mixes the runs with the fixed table.
 *   radices, blocks_n2  HOST description of T_{n2} as for harp_plan_create
 *   hk       HOST float[K][K] with entries +1/-1 and H H^T = K I (else HARP_ERR_BAD_SIGNS /
 *            HARP_ERR_BAD_SCHEDULE); used as out[k'] = sum_k in[k] H[k][k'] / sqrt K
 *   perm, signs  over d, as for harp_plan_create */
harp_status_t harp_plan_create_kronecker(harp_plan_t **out, int64_t n2, int32_t n_stages,
                                         const int32_t *radices, const float *const *blocks_n2,
                                         int32_t K, const float *hk, const int32_t *perm,
                                         const int8_t *signs);

/* Release the plan and its device memory.  NULL is allowed. */
void harp_plan_destroy(harp_plan_t *plan);

/* d of the plan, or -1 for NULL. */
int64_t harp_plan_dim(const harp_plan_t *plan);

/* Apply the processor to a batch of rows, in place (Algorithm 1: y = x T(Theta), with
 * the sign diagonal and permutation in front; transpose != 0 applies Q^T, the map used
 * on the output side of a layer, W^ = U W~^ V^T).
 *   x        DEVICE n_rows x d, dtype fp32 or bf16, overwritten with the result
 *   stream   a cudaStream_t passed as void* (NULL = default stream)
 * Asynchronous on stream; does not synchronise.  n_rows == 0 returns HARP_OK without
 * a launch.  A plan may be applied from several streams at once.  Stream order holds as for
 * any kernel; some kernels are launched so that their set-up (plan data only) may begin while
 * earlier work in the stream is still running -- they read and write x only after that work
 * has completed.
 * Arithmetic.  fp32 rows: fp32 block kernels, fp32 accumulate, the result is the fp32 sum (one
 * rounding per stage).  bf16 rows on the tensor-core kernels (what HARP_KERNEL_AUTO picks for
 * bf16 whenever a plan has one): neighbouring stages are fused at plan time into dense blocks of
 * width 8 to 64 (fp64 product, rounded once to bf16), every block product accumulates in fp32,
 * and the rows are rounded to bf16, to nearest even, after every fused group of stages -- two to
 * five roundings per coordinate instead of one, measured 2e-4 to 7e-4 of the row norm against a
 * tolerance of 8e-3.  bf16 rows on HARP_KERNEL_GENERIC: fp32 throughout, one rounding at the
 * store. */
harp_status_t harp_apply(const harp_plan_t *plan, void *x, int64_t n_rows, harp_dtype_t dtype,
                         int transpose, void *stream);

/* Same as harp_apply with an explicit kernel family (tests and benchmarks).
 * Returns HARP_ERR_UNSUPPORTED if that family has no kernel for this plan/dtype. */
harp_status_t harp_apply_ex(const harp_plan_t *plan, void *x, int64_t n_rows,
                            harp_dtype_t dtype, int transpose, harp_kernel_t kernel,
                            void *stream);

/* Several passes (Section "HARP processors": independent copies of a schedule may be composed;
 * one pass is the paper's default).  Forward computes x <- x Q_0 Q_1 ... Q_{n-1} with
 * Q_k = the processor of plans[k], one harp_apply per pass in that order; transpose != 0 computes
 * x <- x Q_{n-1}^T ... Q_0^T, the inverse for orthogonal blocks.
 *   plans     HOST array of n_passes plan handles of the same dimension (each may have its own
 *             schedule, permutation and signs; a pass after the first usually has neither)
 *   x         DEVICE n_rows x d, overwritten
 * Errors: HARP_ERR_NULL, HARP_ERR_BAD_SCHEDULE (n_passes < 1), HARP_ERR_DIM_MISMATCH, and those
 * of harp_apply (a failing pass leaves x partly transformed).  Asynchronous on stream. */
harp_status_t harp_apply_passes(const harp_plan_t *const *plans, int32_t n_passes, void *x,
                                int64_t n_rows, harp_dtype_t dtype, int transpose, void *stream);

/* Two-sided processing of a weight matrix, W <- Q_out^T W Q_in (paper, Section
 * "Incoherence processing": W~ = U^T W V with U = Q_out, V = Q_in; Algorithm 3 line 3).
 *   W        DEVICE d_out x d_in row-major, d_out = dim(plan_out), d_in = dim(plan_in)
 *   scratch  DEVICE buffer of harp_two_sided_scratch_bytes(...) bytes, 256-byte aligned,
 *            or NULL to let the call allocate and free it on the stream
 *            (cudaMallocAsync/cudaFreeAsync).  It is used only when the column side has to go
 *            through a transposed copy of W (plan_out with a permutation, fp32, or d_in not a
 *            multiple of 8); otherwise the columns are processed in place and it is ignored.
 * Both plans must live on the current device (else HARP_ERR_DIM_MISMATCH).
 * Asynchronous on stream. */
harp_status_t harp_apply_two_sided(void *W, harp_dtype_t dtype, const harp_plan_t *plan_out,
                                   const harp_plan_t *plan_in, void *scratch, void *stream);

/* Bytes of scratch harp_apply_two_sided needs for these plans and dtype (0 on bad input). */
int64_t harp_two_sided_scratch_bytes(const harp_plan_t *plan_out, const harp_plan_t *plan_in,
                                     harp_dtype_t dtype);

/* Two-sided processing without any allocation (the paper has no counterpart: this entry
 * point exists for deployment, not for the method).  It is meant for callers that cannot
 * allocate device memory at call time -- a serving process whose memory pool was sized
 * once at start-up, a host framework that owns the whole device budget, or any context in
 * which an allocation would synchronise or fail.  It computes the same map as
 * harp_apply_two_sided, always by the transpose route (rows through Q_in, transpose, rows
 * through Q_out, transpose back; bf16 results can differ from the other entry point's in the
 * last rounding, and it costs two more passes over W than the in-place column kernels), and
 * keeps the transposed copy of W in a fixed array that is compiled into the library; the array
 * becomes resident when the library's module is loaded on a device (at the latest by the first
 * call) and stays (harp_two_sided_static_capacity_bytes() = 32 MiB) until the process exits.
 *   W        DEVICE d_out x d_in row-major, overwritten; d_out*d_in*sizeof(dtype) must not
 *            exceed the capacity, otherwise HARP_ERR_TOO_LARGE and nothing is launched
 *   plans    must live on the current device (else HARP_ERR_DIM_MISMATCH)
 * No cudaMalloc/cudaFree or other allocating call is made.  The first call on a device
 * looks up the array's device address; make that first call outside any stream capture.
 * All calls share the one array, which keeps whatever the last call left in it (nothing
 * needs to start at zero: every byte is written before it is read).  Two calls that
 * overlap on the GPU -- different streams, or different host threads -- race on it; run
 * them one after the other.  Asynchronous on stream. */
harp_status_t harp_apply_two_sided_static(void *W, harp_dtype_t dtype,
                                          const harp_plan_t *plan_out,
                                          const harp_plan_t *plan_in, void *stream);

/* Capacity in bytes of the fixed scratch array used by harp_apply_two_sided_static. */
int64_t harp_two_sided_static_capacity_bytes(void);

/* ---- Gradient with respect to the block kernels (what Algorithm 3 needs from the apply; the
 * gradient with respect to the rows is harp_apply with transpose = 1 on dL/dy) ----------------
 * For y = x Q (harp_apply, transpose = 0) and a scalar loss L with G = dL/dy:
 *   dL/dK_t[c][i][j] = sum over rows of v_t[base_c + i s_t] * g_{t+1}[base_c + j s_t],
 * v_t the input of stage t in the forward pass and g_{t+1} = dL/d(output of stage t)
 * (g_m = G, g_t = g_{t+1} M_t^T) -- the chain rule through Algorithm 1.
 *   x, gy      DEVICE n_rows x d of dtype, read only
 *   grad       DEVICE float[harp_plan_n_params(plan)], laid out like the blocks given to
 *              harp_plan_create (stage after stage, [D_t][b_t][b_t]); overwritten, or added to
 *              if accumulate != 0
 * Any schedule is accepted.  Sums over rows are taken in fp64 by one thread per entry (no
 * atomics: the result does not depend on scheduling).  The call allocates and frees scratch
 * on the stream (at most ~256 MB, from a memory pool of the library's own that keeps what it has
 * been given until the process ends); HARP_ERR_ALLOC if that fails.  Asynchronous on stream. */
harp_status_t harp_grad_blocks(const harp_plan_t *plan, const void *x, const void *gy, int64_t n_rows,
                               harp_dtype_t dtype, float *grad, int accumulate, void *stream);

/* Number of block-kernel entries of the plan: sum over stages of d * b_t (-1 for NULL). */
int64_t harp_plan_n_params(const harp_plan_t *plan);

/* ---- Diagnostics of a processed layer (appendix "Incoherence diagnostics") ----------------
 * One pass over a row-major DEVICE matrix each; asynchronous on stream; nothing is allocated.
 * out is a DEVICE array of four doubles, 8-byte aligned, owned by the caller: out[0] receives
 * the result, out[1..3] the accumulators named below (the call zeroes all four first).
 * Matrices are contiguous (leading dimension = number of columns) and aligned to their
 * element size; 16-byte alignment with a column count that is a multiple of 16 bytes takes
 * the vectorised path.  Errors: HARP_ERR_NULL, HARP_ERR_BAD_DIM (non-positive or > 2^31
 * extents, misaligned pointers, block outside [1, n]), HARP_ERR_BAD_DTYPE, HARP_ERR_CUDA. */

/* Weight incoherence, Eq. 4: mu_W(A) = sqrt(m n) * max|A_ij| / ||A||_F for A (m x n).
 * out[1] = max|A_ij|, out[2] = ||A||_F^2; mu_W = 0 for the zero matrix. */
harp_status_t harp_weight_incoherence(const void *A, int64_t m, int64_t n, harp_dtype_t dtype,
                                      double *out, void *stream);

/* Off-block energy of the rotated curvature proxy, Eq. 15:
 * R_bd = (1/n^2) * sum over block pairs p != q of ||H_pq||_F^2, the blocks being the
 * quantizer's contiguous partition of the n coordinates into runs of `block` (the last run
 * may be shorter).  H is n x n (for instance the result of harp_apply_two_sided(H, V, V)).
 * out[2] = ||H||_F^2, out[3] = sum of squared entries inside the diagonal blocks. */
harp_status_t harp_offblock_energy(const void *H, int64_t n, int64_t block, harp_dtype_t dtype,
                                   double *out, void *stream);

/* Diagonal Hessian-weighted reconstruction proxy, Eq. 14:
 * L_diag = 1/(d_out d_in) * sum_ij (Wt_ij - Wq_ij)^2 * wbar_j,  w_j = |H_jj|, wbar = w / mean(w).
 *   Wt, Wq  DEVICE d_out x d_in, the rotated weight and its quantised copy (the quantizer is
 *           the caller's; the paper treats Q(Wt) as a constant of the step)
 *   H       DEVICE d_in x d_in of h_dtype, only its diagonal is read
 * out[1] = sum_ij (Wt_ij - Wq_ij)^2 w_j, out[2] = sum_j w_j; L_diag = 0 if every w_j is 0. */
harp_status_t harp_diag_weighted_error(const void *Wt, const void *Wq, int64_t d_out, int64_t d_in,
                                       harp_dtype_t dtype, const void *H, harp_dtype_t h_dtype,
                                       double *out, void *stream);

/* Apply to rows that live in HOST memory (pinned memory gives full copy speed).  Unlike
 * harp_apply this call changes the plan (its staging buffers and streams): one call at a time
 * per plan, from one host thread.  It
 * copies chunks of 16 MiB host->device, applies, copies back, on four internal streams so
 * that copies in both directions overlap each other and the kernels; returns after the last
 * copy has completed.  The device staging buffers (four) belong to the plan and are created at
 * the first call.
 *   x_host   HOST n_rows x d, overwritten with the result */
harp_status_t harp_apply_host(harp_plan_t *plan, void *x_host, int64_t n_rows,
                              harp_dtype_t dtype, int transpose);

/* Device-side wait status of the plan's HARP_KERNEL_TMEM kernels.  Every wait inside those kernels
 * (on a bulk copy, on the tensor core, on another warp) has an iteration limit; a wait that runs out
 * sets a device word, the kernel releases its tensor memory and returns, and the rows it was working
 * on are left undefined.  Returns 0 if no wait has given up since the plan was built, a positive
 * code naming the wait otherwise, -1 for NULL or a failed copy.  Synchronises with the device. */
int32_t harp_plan_error_word(const harp_plan_t *plan);

/* Per-section cycle counters of the tensor-memory kernels and of the whole-row kernel, for profiling
 * notes.  They count only in a library built with HARP_TM_TIMING=1 / HARP_FAST_TIMING=1 in the
 * environment of the build step (clock reads at section boundaries, summed over CTAs; slot 0 = tiles);
 * otherwise the sixteen slots read zero.  out HOST int64[16]; reset != 0 clears them.  0 on success. */
int32_t harp_debug_tm_timing(int64_t *out, int32_t reset);
int32_t harp_debug_fast_timing(int64_t *out, int32_t reset);

/* Number of kernels this library has launched in the calling process (all plans). */
int64_t harp_launch_count(void);

/* Static, human-readable text for a status. */
const char *harp_status_string(harp_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* HARP_H_ */
