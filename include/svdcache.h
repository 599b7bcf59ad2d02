/*
 * svdcache.h — C ABI of the B200-native SVD-Cache hot path (sm_100a).
 *
 * SVD-Cache ("Forecast the Principal, Stabilize the Residual") splits the hidden
 * feature F (N tokens x D) of a DiT block into a rank-k principal part in a fixed,
 * pre-computed right-singular basis V_k and an orthogonal residual, forecasts the
 * principal part with an exponential moving average and reuses the residual:
 *
 *   one-off        V_k  = top-k right singular vectors of a stack of features  (Eq. 4-7)
 *   full step      C    = F V_k                                                (Eq. 8-9)
 *                  R    = F - C V_k^T                                          (Eq. 10)
 *                  Chat = C  on the first full step, else beta Chat + (1-beta) C (Eq. 11)
 *   cached step    Fhat = Chat V_k^T + R                                       (Sec. 3.5)
 *
 * Conventions
 *   - Every function returns an int status: SVDCACHE_OK or a negative SVDCACHE_ERR_*.
 *     Nothing throws.  svdcache_status_string() gives text.
 *   - "device" pointers are CUDA device addresses owned by the caller; "host" pointers
 *     are ordinary host addresses.  The library allocates no device memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  The step
 *     and basis calls only enqueue work on it and return; they never synchronise.
 *     Calls that must hand a number back to the host say so.
 *   - Matrices are row-major.  `ld` is the row pitch in ELEMENTS (>= the row width).
 *   - dtype is the storage type of F, R and Fhat: SVDCACHE_F32 or SVDCACHE_BF16.
 *     Coefficients (C, Chat) are always fp32.  For SVDCACHE_BF16 the kernels read a
 *     bf16 copy of V_k (made by svdcache_basis_prepare) and accumulate in fp32; for
 *     SVDCACHE_F32 they read V_k in fp32 and accumulate in fp64.
 *   - Shape limits: 1 <= N, 8 <= D <= 16384, D % 8 == 0, 8 <= k <= 256, k % 8 == 0,
 *     k <= D.  F, R, Fhat, V_k and all library-defined buffers must be 16-byte aligned,
 *     and (ld * element size) % 16 == 0.  Violations return SVDCACHE_ERR_BAD_SHAPE /
 *     SVDCACHE_ERR_BAD_ALIGN before anything is launched.
 *   - NaN / Inf in the inputs propagate per IEEE-754 and are not errors.
 */
#ifndef SVDCACHE_H_
#define SVDCACHE_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define SVDCACHE_API __attribute__((visibility("default")))
#else
#define SVDCACHE_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define SVDCACHE_OK                0
#define SVDCACHE_ERR_INVALID_ARG  (-1) /* NULL pointer, unknown dtype, bad scalar      */
#define SVDCACHE_ERR_BAD_SHAPE    (-2) /* N, D, k, ld outside the limits above          */
#define SVDCACHE_ERR_BAD_ALIGN    (-3) /* a pointer or pitch is not 16-byte aligned     */
#define SVDCACHE_ERR_STATE        (-4) /* cached step on a state that saw no full step  */
#define SVDCACHE_ERR_WORKSPACE    (-5) /* workspace / buffer smaller than required      */
#define SVDCACHE_ERR_TIMEOUT      (-6) /* a bounded in-kernel wait ran out              */
#define SVDCACHE_ERR_CUDA         (-7) /* a CUDA runtime / driver call failed           */
#define SVDCACHE_ERR_NOT_CONVERGED (-8) /* eigen-solver hit its iteration limit         */
#define SVDCACHE_ERR_SCRATCH_LIMIT (-9) /* problem needs more than the built-in scratch    */

#define SVDCACHE_F32   0
#define SVDCACHE_BF16  1

/* Predictors of the principal coefficients on cached steps (Sec. 3.4; Sec. 5.3, Fig. 4(b)). */
#define SVDCACHE_PREDICT_EMA     0  /* the method's own: the EMA state of Eq. 11                          */
#define SVDCACHE_PREDICT_TAYLOR  1  /* Taylor expansion in the step offset, backward-difference derivatives */
#define SVDCACHE_PREDICT_NEWTON  2  /* polynomial through the last order+1 full steps (Newton backward form) */

/* Text for a status code (static storage, never NULL). */
SVDCACHE_API const char *svdcache_status_string(int status);

/* Text of the last CUDA error seen by the calling thread inside this library. */
SVDCACHE_API const char *svdcache_last_cuda_error(void);

/* ---------------------------------------------------------------------------------
 * Calibration: the "one-time SVD" of Sec. 3.3 (Eq. 4, Eq. 5, Eq. 7).
 *
 * The right singular vectors of a row-stack Fstack (M x D) are the eigenvectors of the
 * Gram matrix G = Fstack^T Fstack, and sigma_i^2 its eigenvalues.  The stack may be fed
 * in pieces: begin, accumulate (any number of times, any row counts), finish.
 *
 *   workspace  device, caller-owned scratch of at least
 *              svdcache_calibrate_workspace_bytes(D, k) bytes, 256-byte aligned; it
 *              carries G between the three calls and must not be touched in between.
 *   F          device, M x D rows of dtype `dtype` with pitch ld; only read.
 *   Vk         device, out: D x k fp32, orthonormal columns ordered by descending
 *              eigenvalue; in each column the entry of largest magnitude is positive.
 *   lambda     device, out, k doubles (eigenvalues of G = sigma_i^2), or NULL.
 *   trace      device, out, 1 double: trace(G) = |Fstack|_F^2 = sum of ALL sigma_i^2
 *              (the denominator of the energy criterion, Eq. 6), or NULL.
 *   info       host, out, 4 doubles or NULL: {multiplications by G done, largest
 *              relative eigen-residual |G v - lambda v| / lambda_1 over the k pairs,
 *              Ritz block width, Jacobi sweeps of the last Rayleigh-Ritz step}.
 *
 * begin and accumulate only enqueue work.  finish synchronises `stream` several times
 * (it reads convergence numbers back) and returns SVDCACHE_ERR_NOT_CONVERGED if the
 * residual target was not met within the iteration limit (outputs are still written).
 * G is accumulated in a fixed order: results are bit-reproducible run to run.  fp32 stacks,
 * narrow or short bf16 stacks are summed in fp64 throughout (eigenvalues good to ~1e-10
 * relative).  bf16 stacks of at least 2048 rows per accumulate call whose width is a
 * multiple of 128 go through the tensor cores: exact bf16 products, fp32 sums over chunks of
 * 2048 rows, fp64 across chunks.  The tensor cores truncate the fp32 running sum, so G comes
 * out smaller by a few 1e-6, almost uniformly: eigenvalues (and the trace) carry that
 * relative error, the eigenvectors are affected far below the 1e-4 principal-angle bound.
 * Chunks start at the first row of each accumulate call, so feeding the same stack in
 * different pieces changes the last bits on that path.
 * ------------------------------------------------------------------------------- */
SVDCACHE_API int svdcache_calibrate_workspace_bytes(int D, int k, size_t *bytes /* host, out */);
SVDCACHE_API int svdcache_calibrate_begin(int D, int k, void *workspace, size_t workspace_bytes, void *stream);
SVDCACHE_API int svdcache_calibrate_accumulate(const void *F, int64_t M, int D, int64_t ld, int dtype,
                                  void *workspace, size_t workspace_bytes, void *stream);
SVDCACHE_API int svdcache_calibrate_finish(int D, int k, float *Vk, double *lambda, double *trace,
                              double *info, void *workspace, size_t workspace_bytes,
                              void *stream);
/* One-shot form: begin + accumulate(Fstack) + finish. */
SVDCACHE_API int svdcache_calibrate(const void *Fstack, int64_t M, int D, int64_t ld, int dtype, int k,
                       float *Vk, double *lambda, double *trace, double *info,
                       void *workspace, size_t workspace_bytes, void *stream);

/* Where the Gram matrix sits in a calibration workspace (Eq. 4): D x D doubles, row-major, `offset`
 * bytes from the start, complete between the last accumulate and the finish.  Row-sharded
 * calibration over several GPUs: every rank begins and accumulates its own rows, the ranks sum
 * this region (one all-reduce of D x D doubles), every rank finishes on the sum. */
SVDCACHE_API int svdcache_calibrate_gram_region(int D, size_t *offset, size_t *bytes /* host, out */);

/* Stability of the decomposition across "prompts" (Fig. 1(b)): similarity = cosine similarity x
 * magnitude similarity (min / max of the two norms).  For the singular values sigma = sqrt(lambda)
 * of two calibrations A and B: out[0] = cos(sigma_A, sigma_B) * min(|sigma_A|, |sigma_B|) / max(..).
 * For the right singular vectors (unit columns, sign-free): column_cos[j] = |<v_j^A, v_j^B>|,
 * out[1] = their mean.  VkA, VkB device D x k fp32, lambda device k doubles, column_cos device k
 * doubles (out), out host 2 doubles.  Synchronises `stream`. */
SVDCACHE_API int svdcache_basis_similarity(const float *VkA, const double *lambdaA, const float *VkB,
                              const double *lambdaB, int D, int k, double *column_cos,
                              double *out, void *stream);

/* ---------------------------------------------------------------------------------
 * Calibration for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this entry point exists for how the library gets embedded, not for the
 * method.)
 *
 * svdcache_calibrate wants a workspace, and a host program normally gets one from
 * cudaMalloc.  Some hosts may not call it where calibration has to run: a plugin inside
 * an inference server whose memory pool was sized and handed out at start-up, code that
 * runs between the launches of a latency-critical loop where an allocation would
 * synchronise the device, or a process whose allocator is simply owned by someone else.
 * For them the library carries SVDCACHE_BUILTIN_SCRATCH_BYTES of scratch inside its own
 * device image (every GPU that loads the library holds that much until the process exits)
 * and this call uses it in place of the workspace.  Same arguments, results and status
 * codes as svdcache_calibrate otherwise; inputs and outputs are still the caller's.
 *
 *   - Size limit: svdcache_calibrate_workspace_bytes(D, k) must not exceed
 *     SVDCACHE_BUILTIN_SCRATCH_BYTES (e.g. D = 512 with k = 64 fits, D = 1152 does not);
 *     beyond it the call returns SVDCACHE_ERR_SCRATCH_LIMIT and launches nothing.
 *   - It calls no cudaMalloc / cudaFree and no routine that allocates.
 *   - The first call on a device looks up the scratch's device address
 *     (cudaGetSymbolAddress, with that device current) and keeps it; make that first call
 *     before starting any stream capture.
 *   - There is ONE scratch array per device and every call uses it.  It still holds the
 *     previous call's contents when a call starts; the call clears what it accumulates into
 *     before use.  Two calls whose GPU work overlaps (different streams, different threads)
 *     would trample each other: keep them ordered, e.g. on one stream.
 *   - Like svdcache_calibrate it synchronises `stream` while it iterates.
 * ------------------------------------------------------------------------------- */
#define SVDCACHE_BUILTIN_SCRATCH_BYTES (4u << 20)
SVDCACHE_API int svdcache_calibrate_noalloc(const void *Fstack, int64_t M, int D, int64_t ld, int dtype, int k,
                               float *Vk, double *lambda, double *trace, double *info, void *stream);

/* Rank selection by energy threshold (Eq. 6): the smallest k' <= n with
 * sum_{i<=k'} lambda_i / trace >= tau; n if the n listed eigenvalues fall short.
 * lambda: HOST array of n descending eigenvalues.  Pure host arithmetic. */
SVDCACHE_API int svdcache_rank_for_energy(const double *lambda, int n, double trace, double tau,
                             int *k_out /* host, out */);

/* ---------------------------------------------------------------------------------
 * Basis buffer: the cached reference basis of Eq. 7 in the layouts the step kernels
 * read.  Layout (all sections 256-byte aligned, offsets from svdcache_basis_layout):
 *   header (256 B) | V fp32 [D x k] | V^T fp32 [k x D] | V bf16 [D x k] | V^T bf16 [k x D]
 * The two bf16 sections exist only for dtype = SVDCACHE_BF16; they hold V_k rounded to
 * nearest-even, and are the values the bf16 kernels multiply with.
 * ------------------------------------------------------------------------------- */
SVDCACHE_API int svdcache_basis_bytes(int D, int k, int dtype, size_t *bytes /* host, out */);
SVDCACHE_API int svdcache_basis_layout(int D, int k, int dtype,
                          size_t *v_f32_offset, size_t *vt_f32_offset,
                          size_t *v_bf16_offset, size_t *vt_bf16_offset /* host, out; may be NULL */);
/* Vk: device D x k fp32 (only read).  basis: device, out, >= svdcache_basis_bytes. */
SVDCACHE_API int svdcache_basis_prepare(const float *Vk, int D, int k, int dtype, void *basis,
                           size_t basis_bytes, void *stream);

/* ---------------------------------------------------------------------------------
 * Per-block cache state, a caller-owned flat device buffer (checkpoint = memcpy):
 *   header (256 B) | Chat fp32 [N x k] | Chat operand copy | R dtype [N x D]   (dense, no pitch)
 * The operand copy exists only for dtype = SVDCACHE_BF16: Chat as two bf16 arrays [N x k],
 * hi = bf16(Chat) and lo = bf16(Chat - hi), which every full step rewrites together with
 * Chat and the cached step feeds to the tensor cores as they are (hi + lo carries ~16
 * mantissa bits).  Offsets of Chat and R come from svdcache_state_layout.
 * The header counts the full steps the state has seen and carries a sticky device
 * status word.  svdcache_state_reset must be called once before first use (and again to
 * start a new sampling run): it clears the counter, so the next full step initialises
 * the EMA with Chat = C.
 * ------------------------------------------------------------------------------- */
SVDCACHE_API int svdcache_state_bytes(int64_t N, int D, int k, int dtype, size_t *bytes /* host, out */);
SVDCACHE_API int svdcache_state_layout(int64_t N, int D, int k, int dtype,
                          size_t *chat_offset, size_t *r_offset /* host, out */);
SVDCACHE_API int svdcache_state_reset(void *state, int64_t N, int D, int k, int dtype, void *stream);
/* Synchronises `stream`, then reads the header: full steps seen, device status word
 * (SVDCACHE_OK, SVDCACHE_ERR_STATE or SVDCACHE_ERR_TIMEOUT).  Outputs are host. */
SVDCACHE_API int svdcache_state_query(const void *state, void *stream, int64_t *full_steps, int *status);

/* ---------------------------------------------------------------------------------
 * Full step (Eq. 8 - Eq. 11), one fused pass: C = F V_k, R = F - C V_k^T stored into
 * the state, Chat updated in the state (Chat = C if the state has seen no full step
 * yet).  F passes through untouched: the sampler keeps using the true feature.
 *   F      device, N x D, pitch ld, only read
 *   basis  device, from svdcache_basis_prepare for the same D, k, dtype
 *   state  device, in/out
 *   C_out  device, out, N x k fp32 (this step's coefficients), or NULL
 *   beta   EMA weight in [0, 1] (the paper uses 0.9)
 * ------------------------------------------------------------------------------- */
SVDCACHE_API int svdcache_full_step(const void *F, int64_t ld, const void *basis, void *state,
                       float *C_out, int64_t N, int D, int k, int dtype, float beta,
                       void *stream);

/* ---------------------------------------------------------------------------------
 * Cached step (Sec. 3.5): Fhat = Chat V_k^T + R.  The EMA state changes only at full
 * steps, so every cached step until the next full step returns the same Fhat;
 * `steps_since_full` is ignored by the EMA (the predictors that use it are the
 * svdcache_cached_step_forecast calls below).  If the state has seen no full step the kernel writes nothing and records
 * SVDCACHE_ERR_STATE in the state header (read it with svdcache_state_query).
 *   Fhat   device, out, N x D, pitch ld
 * ------------------------------------------------------------------------------- */
SVDCACHE_API int svdcache_cached_step(const void *state, const void *basis, void *Fhat, int64_t ld,
                         int64_t N, int D, int k, int dtype, int steps_since_full,
                         void *stream);

/* ---------------------------------------------------------------------------------
 * Batched forms: the same operation on `nblocks` independent DiT blocks in ONE launch
 * (Eq. 8 - Eq. 11 / Sec. 3.5 per block).  Block b uses F + b*F_stride, basis +
 * b*basis_stride, state + b*state_stride, out + b*out_stride; all strides are in BYTES
 * and multiples of 256.  Shapes, dtype and beta are shared.
 * ------------------------------------------------------------------------------- */
SVDCACHE_API int svdcache_full_step_batched(int nblocks, const void *F, int64_t ld, size_t F_stride,
                               const void *basis, size_t basis_stride, void *state,
                               size_t state_stride, float *C_out, size_t C_stride,
                               int64_t N, int D, int k, int dtype, float beta, void *stream);
SVDCACHE_API int svdcache_cached_step_batched(int nblocks, const void *state, size_t state_stride,
                                 const void *basis, size_t basis_stride, void *Fhat,
                                 int64_t ld, size_t Fhat_stride, int64_t N, int D, int k,
                                 int dtype, int steps_since_full, void *stream);

/* ---------------------------------------------------------------------------------
 * Blocks of different rank in one call (Eq. 6: the rank follows each block's spectrum, see
 * svdcache_rank_for_energy).  k_per_block is a HOST array of nblocks ranks; block b's basis and
 * state buffers are laid out for k_per_block[b] and sit b * stride bytes from the first (the
 * strides must cover the largest of them; C_out rows are k_per_block[b] wide).  Consecutive
 * blocks of equal rank go out as one batched launch; everything else is as in the batched
 * forms above.
 * ------------------------------------------------------------------------------- */
SVDCACHE_API int svdcache_full_step_ranked_batched(int nblocks, const void *F, int64_t ld, size_t F_stride,
                                      const void *basis, size_t basis_stride, void *state,
                                      size_t state_stride, float *C_out, size_t C_stride, int64_t N,
                                      int D, const int *k_per_block, int dtype, float beta,
                                      void *stream);
SVDCACHE_API int svdcache_cached_step_ranked_batched(int nblocks, const void *state, size_t state_stride,
                                        const void *basis, size_t basis_stride, void *Fhat,
                                        int64_t ld, size_t Fhat_stride, int64_t N, int D,
                                        const int *k_per_block, int dtype, int steps_since_full,
                                        void *stream);

/* ---------------------------------------------------------------------------------
 * Other predictors on the principal coefficients (Sec. 5.3, Fig. 4(b)): the decomposition
 * paired with a predictor that extrapolates inside the interval.  The caller keeps the
 * coefficients C of the last order+1 full steps (the C_out of svdcache_full_step) and hands
 * them over newest first; the residual is still the stored R (Sec. 3.5):
 *     Fhat = (sum_j w_j C_{n-j}) V_k^T + R,      u = steps_since_full / interval,
 *     backward differences D^i of the history, and
 *     SVDCACHE_PREDICT_TAYLOR   sum_i u^i / i! D^i
 *     SVDCACHE_PREDICT_NEWTON   sum_i u (u+1) ... (u+i-1) / i! D^i   (exact for polynomials of degree <= order)
 *     SVDCACHE_PREDICT_EMA      ignores the history: the plain cached step.
 * order 0 of either is plain reuse of the newest coefficients (Eq. 3).  order <= 7.
 *   svdcache_forecast_weights  host: the order+1 weights w_j (newest first) into w
 *   svdcache_forecast_bytes    host: size of the forecast buffer for N x k coefficients
 *   C_hist     HOST array of order+1 DEVICE pointers, each N x k fp32 (block b at + b*C_stride bytes)
 *   forecast   device scratch, 256-byte aligned, >= svdcache_forecast_bytes (block b at
 *              + b*forecast_stride): receives the forecast (fp32, then its split-bf16 pair)
 * Two launches: the forecast (N k work), then the cached-step kernel reading it.  The state is
 * only read.  Errors as svdcache_cached_step.
 * ------------------------------------------------------------------------------- */
SVDCACHE_API int svdcache_forecast_weights(int predictor, int order, int steps_since_full, int interval,
                              double *w /* host, out, order+1 */);
SVDCACHE_API int svdcache_forecast_bytes(int64_t N, int k, size_t *bytes /* host, out */);
SVDCACHE_API int svdcache_cached_step_forecast_batched(int nblocks, const void *state, size_t state_stride,
                                          const void *basis, size_t basis_stride, void *Fhat,
                                          int64_t ld, size_t Fhat_stride, int64_t N, int D, int k,
                                          int dtype, const float *const *C_hist, size_t C_stride,
                                          int predictor, int order, int steps_since_full,
                                          int interval, void *forecast, size_t forecast_stride,
                                          void *stream);

/* ---------------------------------------------------------------------------------
 * Ablation of Sec. 4.5 (Fig. 4(c)): the stored residual as an EMA of the residuals,
 *     R <- F - C V_k^T on the first full step, else beta_r R + (1 - beta_r)(F - C V_k^T).
 * beta_r = 0 is svdcache_full_step itself (the method: the residual is reused as it is);
 * beta = beta_r = 0 is "reuse on both" (Eq. 3); beta, beta_r > 0 is "EMA on both".  With
 * beta_r > 0 the step reads the old R as well (N D more elements than the method's step): the
 * epilogue of the fused kernel loads it and blends before the one rounding to the I/O dtype.
 * Arguments as svdcache_full_step_batched.
 * ------------------------------------------------------------------------------- */
SVDCACHE_API int svdcache_full_step_residual_ema_batched(int nblocks, const void *F, int64_t ld,
                                            size_t F_stride, const void *basis, size_t basis_stride,
                                            void *state, size_t state_stride, float *C_out,
                                            size_t C_stride, int64_t N, int D, int k, int dtype,
                                            float beta, float beta_r, void *stream);

/* ---------------------------------------------------------------------------------
 * The cached singular values and the left factors of Eq. 7 - Eq. 8.
 *   svdcache_singular_values  sigma_i = sqrt(lambda_i) of the calibration spectrum (device arrays of k)
 *   svdcache_left_factors     U = C diag(sigma)^-1 (Eq. 8), C and U device N x k fp32; a column whose
 *                             sigma is 0 is set to 0.  (The step kernels never form U: sigma cancels
 *                             between Eq. 8 and Eq. 9.)
 * ------------------------------------------------------------------------------- */
SVDCACHE_API int svdcache_singular_values(const double *lambda, int k, double *sigma, void *stream);
SVDCACHE_API int svdcache_left_factors(const float *C, const double *sigma, int64_t N, int k, float *U,
                          void *stream);

/* ---------------------------------------------------------------------------------
 * Introspection for benchmarks and tests (host only).
 *   svdcache_kernel_launches: kernels this library has launched in this process.
 *   svdcache_set_path: a process-wide switch for tests and benchmarks (every later step call
 *                      of every thread sees it; not meant for production code).
 *                      0 = pick automatically, 1 = force the CUDA-core kernels,
 *                      2 = force the tcgen05 kernels (error if the shape is outside what
 *                      they support).  Returns the previous setting.
 *   svdcache_last_path: which kernel family the last step call used (1 or 2).
 * ------------------------------------------------------------------------------- */
SVDCACHE_API uint64_t svdcache_kernel_launches(void);
SVDCACHE_API int svdcache_set_path(int path);
SVDCACHE_API int svdcache_last_path(void);

/* Self-test of the time-out path (no counterpart in the paper).  Every wait inside the
 * tcgen05 kernels is bounded (~2 s): when one runs out the kernel stops, stores
 * SVDCACHE_ERR_TIMEOUT in the state header of block 0 together with which wait it was, and
 * returns, so the context stays usable.  This call launches one small CTA that waits, with the
 * same code, for an event that never comes, for `limit_cycles` SM cycles (1 .. 2e8): afterwards
 * svdcache_state_query on `state` (a reset state buffer, device, 256-byte aligned) must report
 * SVDCACHE_ERR_TIMEOUT, the word at byte 36 of the header reads 99 << 16 (wait site 99, CTA 0),
 * and svdcache_state_reset clears both.  Asynchronous on `stream`.  Nothing is faulted or hung. */
SVDCACHE_API int svdcache_selftest_wait_timeout(void *state, int64_t limit_cycles, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* SVDCACHE_H_ */
