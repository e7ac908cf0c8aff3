/*
 * sds.h - C ABI of libsds: speculative sampling for diffusion chains on one GPU.
 *
 * The library runs, for B independent chains, the draft-then-verify window of
 * "Accelerated Diffusion Models via Speculative Sampling" (arxiv 2501.05370):
 *   - target chain: Gaussian transitions N(m^q_k(y), sigma_k^2 I)                  (Eq. 3)
 *   - frozen-target drafter: same transition with the denoiser output frozen       (Eq. 6 and the
 *     "Efficient frozen draft strategy" paragraph of Appendix B)
 *   - window loop: draft L steps, one batched target pass, sequential accept       (Algorithms 1, 4)
 *   - accept test and adjusted law: reflection maximal coupling                    (Algorithm 3)
 *   - Langevin variant: same loop with m = x - gamma grad E, sigma = sqrt(2 gamma) (Algorithm 5)
 *
 * Every transition mean is affine in (state, denoiser output): m_k(y, D) = a_k*y + c_k*D.
 * The caller supplies a_k, c_k, sigma_k (k = 0..K-1 is the transition Y_k -> Y_{k+1}) and a denoiser.
 *
 * Conventions
 *   - "dev" pointers are device pointers on the current CUDA device, "host" pointers are host
 *     pointers. All are owned by the caller; the library neither frees nor allocates device memory.
 *     Its only device storage is the workspace the caller binds (size from sds_workspace_bytes).
 *   - Host arrays of sds_schedule are copied at sds_create. Device arrays named in sds_denoiser
 *     must stay valid until sds_destroy.
 *   - All work is enqueued on the stream given to sds_bind. Calls return after enqueueing except
 *     sds_bind, sds_advance with a non-NULL n_active, sds_sample_all(_host), and sds_get with a host
 *     destination, which wait for the stream.
 *   - Every call returns SDS_OK (0) or a negative code; nothing throws across the boundary.
 *     sds_last_cuda_error gives the CUDA error behind SDS_ECUDA.
 *   - A context is used by one host thread at a time. Contexts are independent.
 *   - Random numbers: Philox-4x32-10, counter (q, k, b_lo, stream + 256*b_hi), key = seed, where
 *     q = element index / 4, k = transition index, b = global chain id (chain_id_offset + local
 *     index). Stream 0 = draft noise, 1 = accept uniform, 2 = initial state. Results of a chain
 *     therefore do not depend on which other chains share the context.
 */
#ifndef SDS_H_
#define SDS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ---- */
#define SDS_OK            0
#define SDS_EINVAL       (-1)   /* NULL pointer, B<=0, d<=0, L not in [1,32], non-finite schedule, sigma_k<=0 */
#define SDS_ESTATE       (-2)   /* call order other than bind -> reset -> (draft -> verify_window -> advance)* */
#define SDS_ENOMEM       (-3)   /* workspace too small or misaligned */
#define SDS_EUNSUPPORTED (-4)   /* unknown denoiser kind / dtype / drafter mode, shape the kernels cannot take */
#define SDS_ECUDA        (-5)   /* a CUDA call failed; see sds_last_cuda_error */
#define SDS_ETIMEOUT     (-6)   /* a bounded device-side wait gave up */
#define SDS_ENONFINITE   (-7)   /* some chain produced a non-finite log-ratio and was frozen; others valid */
#define SDS_ECALLBACK    (-8)   /* the user denoiser callback returned non-zero */

/* ---- denoiser kinds, dtypes, drafter modes, sds_get selectors ---- */
#define SDS_DEN_GMM       1     /* closed-form Gaussian-mixture posterior mean / energy gradient */
#define SDS_DEN_MLP       2     /* bf16 MLP with per-step embedding rows */
#define SDS_DEN_CALLBACK  3     /* user function on device buffers */
#define SDS_DEN_PHI4      4     /* energy gradient of the phi^4 lattice model (Langevin chains, Appendix K) */

#define SDS_F32           0
#define SDS_BF16          1

#define SDS_FROZEN_PREV   0     /* drafter reuses the newest target output on the accepted path (no extra call;
                                   the fallback the "efficient frozen draft strategy" paragraph offers, used always) */
#define SDS_FROZEN_EXACT  1     /* main-text frozen drafter (Eq. 6): sds_draft first evaluates the target at
                                   (Y_n, t_n) for every active chain; that output is also row 1 of the batch,
                                   so position 1 always accepts. Two sequential target calls per window. */

#define SDS_INDEPENDENT   2     /* a second, cheaper model proposes every draft step (Eq. 5); needs
                                   sds_create_with_drafter */

#define SDS_PICARD        3     /* draft means from Picard iterations of the deterministic sampler (Appendix C,
                                   parallel sampling as drafting); needs sds_create_picard */

#define SDS_GET_X         1     /* float  [nrows, d]  drafted states fed to the target (row r = rowoff[s]+j-1) */
#define SDS_GET_TAIL      2     /* float  [B, d]      last drafted state of each chain's window */
#define SDS_GET_DQ        3     /* float  [nrows, d]  target denoiser outputs, same rows as X */
#define SDS_GET_DC        4     /* float  [B, d]      carried (frozen) denoiser output */
#define SDS_GET_Y         5     /* float  [B, d]      current state Y_n */
#define SDS_GET_N         6     /* int32  [B]         current index n_b */
#define SDS_GET_ACT       7     /* int32  [B]         active chain ids, first n_active entries valid */
#define SDS_GET_ROWOFF    8     /* int32  [B+1]       first row of each active slot; [n_active] = nrows */
#define SDS_GET_S1        9     /* double [B, L]      |Delta|^2 per (chain, position) of the last verify */
#define SDS_GET_S2        10    /* double [B, L]      Delta . Z */
#define SDS_GET_ELL       11    /* float  [B, L]      log acceptance ratio */
#define SDS_GET_LOGU      12    /* float  [B, L]      log of the accept uniform */
#define SDS_GET_ACCMASK   13    /* uint32 [B]         bit j-1 set = position j accepted */
#define SDS_GET_JSTAR     14    /* int32  [B]         first rejected position, Lt+1 if none */
#define SDS_GET_NFE_CALLS 15    /* int32  [B]         sequential batched target calls the chain took part in */
#define SDS_GET_NFE_ROWS  16    /* int32  [B]         target rows evaluated for the chain */
#define SDS_GET_CTL       17    /* int32  [16]        n_active, nrows, windows done, error word, frozen chains, ...;
                                   [7]: chain-stages in which every position was accepted (SDS_OPT_STAGED_WINDOWS);
                                   [8], [9]: mixing-GEMM tiles of the split-precision mixture run with all six
                                   products / with the three of the first plane since sds_reset;
                                   [10]: mixing-GEMM tiles skipped since sds_reset (SDS_OPT_ONEHOT_ROWS);
                                   [11]: how the last sds_sample_all ran its windows (bit 0: SDS_OPT_REGEN_DRAFTS in effect,
                                   bit 2: rows of skipped one-hot blocks read from the means table, see SDS_OPT_ONEHOT_ROWS);
                                   [12]: window positions whose accept test was evaluated since sds_reset
                                   (the window kernels; with SDS_OPT_VERIFY_EARLY_EXIT fewer than the rows drafted);
                                   [13]: those of them evaluated with the drafted states made again (SDS_OPT_REGEN_DRAFTS);
                                   [14]: drafted rows stored as floats since sds_reset (the others only as bf16 copies) */
#define SDS_GET_ROWK      18    /* int32  [nrows]     transition index of each row */
#define SDS_GET_DP        19    /* float  [nrows, d]  independent drafter: the draft model's output per drafted row */

typedef struct sds_ctx sds_ctx;   /* opaque, owned by the library */

/* Transition schedule, caller-owned host arrays copied at create.
 * mean_k(y, D) = a[k]*y + c[k]*D, std sigma[k] > 0 shared by target and drafter (the method needs
 * equal covariances: Section 3.3 and the appendix on unequal variances).
 * tcond: [K, tcond_dim] per-step scalars handed to the denoiser (GMM: 4 per step, see below), in
 * double: the mixture logits are differences of large terms, so their coefficients keep full precision. */
typedef struct {
  int32_t K;
  const float* a;
  const float* c;
  const float* sigma;
  const double* tcond;
  int32_t tcond_dim;
} sds_schedule;

/* User denoiser: rows of x_dev [rows, d] (float, dense) at transition indices k_dev [rows] ->
 * out_dev [rows, d]. Must enqueue on `stream` (a cudaStream_t) and return 0. */
typedef int (*sds_denoise_fn)(void* user, const float* x_dev, const int32_t* k_dev, int64_t rows,
                              int32_t d, float* out_dev, void* stream);

/* Exactly one kind is used.
 * GMM (mixture of ncomp isotropic Gaussians sharing one std): with tcond[k] = (A, Bq, C, E)
 *     r = softmax_c( logw[c] + A * <x, mu_c> + Bq * |mu_c|^2 ),   D(x, k) = C * sum_c r_c mu_c + E * x.
 *   Posterior mean E[x0 | x_t] of a variance-preserving forward process and the energy gradient of
 *   the mixture both have this form (binding helpers compute the four scalars).
 *   means_dev: [ncomp, d] float (SDS_F32) or bf16 (SDS_BF16; then <x,mu> and the mixing sum run on
 *   tensor cores with x and r rounded to bf16). logw_dev: [ncomp] float. Float mixtures take at most 7264
 *   components (one logit per component and warp in shared memory); more is SDS_EUNSUPPORTED.
 * MLP: nlayer linear layers dims[0]=d -> ... -> dims[nlayer]=d.
 *   h_l = SiLU(W_l h_{l-1} + bias_l + temb_l[k]) for l < nlayer, output = W_nlayer h + bias (float).
 *   W_dev[l]: [dims[l+1], dims[l]] bf16 row-major; bias_dev[l]: [dims[l+1]] float;
 *   temb_dev[l]: [K, dims[l+1]] bf16 (NULL for the last layer). Every dims[] a multiple of 128.
 * PHI4: D(x) = grad E(x), E(x) = coupling/2 sum_{|i-j|=1} (x_i - x_j)^2 + sum_i (x_i^2 - 1)^2 on a
 *   grid_side x grid_side lattice (d = grid_side^2), every neighbouring pair once, free boundaries
 *   unless periodic != 0. Used with the Langevin schedule a = 1, c = -gamma, sigma = sqrt(2 gamma). */
typedef struct {
  int32_t kind;
  int32_t ncomp;
  const void* means_dev;
  const float* logw_dev;
  int32_t means_dtype;
  int32_t nlayer;
  const void* const* W_dev;
  const float* const* bias_dev;
  const void* const* temb_dev;
  const int32_t* dims;
  sds_denoise_fn fn;
  void* user;
  int32_t grid_side;
  float coupling;
  int32_t periodic;
} sds_denoiser;

/* Bytes of device workspace sds_bind needs for this problem (256-byte aligned base required). */
int sds_workspace_bytes(const sds_schedule* sch, const sds_denoiser* den, int64_t B, int32_t d,
                        int32_t L, size_t* bytes);

/* Create a context for B chains of dimension d with window L (Algorithm 4's inputs L, K, p, q).
 * Validates and copies the schedule. No device work. */
int sds_create(const sds_schedule* sch, const sds_denoiser* den, int64_t B, int32_t d, int32_t L,
               sds_ctx** out);

/* Same with a second, cheaper denoiser as independent draft model (Eq. 5): the draft mean at
 * every position is a_k y + c_k D^p(y, k) with D^p = `drafter` (any kind but the callback), evaluated
 * sequentially, one position of all chains per call. drafter_tcond: [K, 4] host doubles (the
 * mixture coefficients of the draft model; NULL unless the drafter is a mixture). Bind with
 * SDS_INDEPENDENT. One batched target call per window. sds_sample_all uses the window kernels, or the
 * whole-chain kernel when target and draft model are both small float mixtures (<= 32 components, d <= 256). */
int sds_workspace_bytes_with_drafter(const sds_schedule* sch, const sds_denoiser* den, const sds_denoiser* drafter,
                                     const double* drafter_tcond, int64_t B, int32_t d, int32_t L, size_t* bytes);
int sds_create_with_drafter(const sds_schedule* sch, const sds_denoiser* den, const sds_denoiser* drafter,
                            const double* drafter_tcond, int64_t B, int32_t d, int32_t L, sds_ctx** out);

/* Picard drafter (Appendix C, "parallel sampling and speculative correction"): per window,
 * calls >= 1 batched target calls build the draft. Points F_0..F_{Lt-1} of the deterministic
 * sampler F_{j+1} = a_det[k] F_j + c_det[k] D(F_j, k), k = n+j, F_0 = Y_n, start as the rollout
 * with the carried target output frozen and are refined by calls-1 Picard iterations (each one
 * target call on all points of the previous iterate); the last call evaluates the target at the
 * points and the draft mean of position j is the stochastic step from F_{j-1}:
 * m^p_j = a_k F_{j-1} + c_k D(F_{j-1}, k), independent of the earlier drafted states. Position 1
 * is thereby drafted from the target itself and always accepts. a_det, c_det: host arrays [K]
 * (copied), finite. Bind with SDS_PICARD. Target calls per window: calls + 1 (calls for a window
 * of one position). SDS_GET_DP returns the draft means per drafted row. The carried output follows
 * the SDS_FROZEN_PREV rule. sds_sample_all uses the window kernels. */
int sds_workspace_bytes_picard(const sds_schedule* sch, const sds_denoiser* den, int64_t B, int32_t d, int32_t L,
                               size_t* bytes);
int sds_create_picard(const sds_schedule* sch, const sds_denoiser* den, int32_t calls, const float* a_det,
                      const float* c_det, int64_t B, int32_t d, int32_t L, sds_ctx** out);

/* Attach workspace, stream (cudaStream_t, may be NULL for the default stream), seed, drafter mode
 * and the global id of local chain 0. Uploads the schedule into the workspace and waits for it. */
int sds_bind(sds_ctx* ctx, void* workspace_dev, size_t bytes, void* cuda_stream, uint64_t seed,
             int32_t drafter_mode, int64_t chain_id_offset);

/* Start all chains: Y_0 ~ N(0, I) from stream 2, n = 0, carried output D(Y_0, 0) (the one initial
 * target call of the efficient frozen drafter), counters cleared, all chains active. */
int sds_reset(sds_ctx* ctx);

/* Draft: for every active chain, X[r0] = Y_n and, for j = 1..Lt (Lt = min(L, K-n)),
 * W_j = a_k W_{j-1} + c_k D_c + sigma_k xi_{b,k}, k = n+j-1 (Algorithm 4, draft loop; Eq. 6). */
int sds_draft(sds_ctx* ctx);

/* Batched target pass on the drafted rows, then per position Delta = (m^p - m^q)/sigma,
 * Z = (W_j - m^p)/sigma, log ratio = -|Delta|^2/2 - Delta.Z, accept iff log U <= log ratio,
 * first rejection per chain, and the reflected state m^q + sigma (Z - 2 (Delta.Z/|Delta|^2) Delta)
 * written over the rejected draft (Algorithm 4, verification loop; Algorithm 3). */
int sds_verify_window(sds_ctx* ctx);

/* n <- n + adv with adv = min(first rejection, Lt); Y <- W_adv; carried output <- target output of
 * row adv; counters; rebuild the dense list of chains with n < K (Algorithm 4, "Set n <- k").
 * n_active (host, may be NULL): if given, waits for the stream and stores the number of active chains. */
int sds_advance(sds_ctx* ctx, int64_t* n_active);

/* reset, then windows until no chain is active; copies Y_K to out_dev [B, d] and the counters to
 * nfe_calls_dev / nfe_rows_dev [B] (either may be NULL). Waits for the stream.
 * Small float mixtures and the lattice model run as one persistent kernel, one warp per chain, same results. */
int sds_sample_all(sds_ctx* ctx, float* out_dev, int32_t* nfe_calls_dev, int32_t* nfe_rows_dev);

/* Options. SDS_OPT_WHOLE_CHAIN_KERNEL (default 1): let sds_sample_all run small float mixtures
 * (d <= 256, <= 32 components; SDS_FROZEN_PREV, SDS_FROZEN_EXACT, or SDS_INDEPENDENT with a draft model of
 * the same kind) and the lattice model
 * (d <= 256, SDS_FROZEN_EXACT) as one persistent kernel; 0 forces the window-by-window kernels.
 * After the whole-chain kernel only Y, N, DC and the NFE counters are meaningful for sds_get. */
#define SDS_OPT_WHOLE_CHAIN_KERNEL 1
/* SDS_OPT_TENSOR_SPLIT (default 1): float mixtures with more than 32 components whose shapes tile
 * for the tensor cores (ncomp % 128 == 0, d % 128 == 0) run both contractions as bf16 tensor-core
 * GEMMs on a three-way split of every float operand (six partial products, float accumulation);
 * 0 forces the float ALU kernel. */
#define SDS_OPT_TENSOR_SPLIT 2
/* SDS_OPT_GEMM_PAIR (default 1): tensor-core GEMMs whose N is a multiple of 256 run on clusters of
 * two CTAs that share one 256 x 256 tile (each CTA stages half of the B tile); 0 keeps one CTA
 * per 128 x 256 tile. Same products, same accumulation order per output element: both give the
 * same bits. Falls back to one CTA per tile where no cluster can be resident. */
#define SDS_OPT_GEMM_PAIR 3
/* SDS_OPT_VERIFY_EARLY_EXIT (default 1): Algorithm 4 stops at the first rejection, so nothing after
 * it is needed. For d % 4 == 0, 256 < d <= 16384 (one CTA per chain) with the full-space test and a
 * frozen or independent drafter, verify takes the positions in blocks of two (d >= 2048: the first position alone,
 * then pairs) or four (d < 2048), decides a block's
 * accept tests before reading the next and skips every block after the one that holds the first
 * rejection. Decisions, first-reject indices, reflected states and counters are unchanged; the
 * diagnostic arrays (SDS_GET_S1, _S2, _ELL, _LOGU, bits of _ACCMASK) hold zeros for the skipped
 * positions. 0 evaluates every position of every window. */
#define SDS_OPT_VERIFY_EARLY_EXIT 4
/* SDS_OPT_FUSE_ADVANCE (default 1): inside sds_sample_all, for d % 4 == 0 with d <= 256 or
 * 2048 < d <= 16384, the verify kernel also performs the advance step of its chain, and the CTA that finishes
 * last rebuilds the active list, so a window is draft, denoiser, verify: one launch less. Same
 * results. The step-wise calls sds_verify_window / sds_advance are not affected. */
#define SDS_OPT_FUSE_ADVANCE 5
/* SDS_OPT_RAW_ROWS (default 1): inside sds_sample_all, for mixture denoisers on the tensor cores with a
 * frozen drafter, the mixing GEMM stores its accumulators and the verify and advance kernels, which
 * hold the rows' inputs anyway, apply the affine map C acc + E x with the same operations: the GEMM's
 * epilogue no longer reads the rows. Same results, bit for bit. */
#define SDS_OPT_RAW_ROWS 6
/* SDS_OPT_REGEN_DRAFTS (default 1; needs SDS_OPT_FUSE_ADVANCE): inside sds_sample_all, for SDS_FROZEN_PREV with
 * d % 4 == 0, 256 < d <= 16384, the full-space test and a target that reads only the bf16 copy of its
 * input rows (the MLP; the bf16 mixture with SDS_OPT_RAW_ROWS), the draft kernel stores only that copy and
 * the verify kernel does not read drafted states at all. A drafted state (Algorithm 4, draft step) is a
 * function of Y_n, the frozen target output and the chain's noise, which is a function of (seed, chain,
 * step): verify runs the draft recurrence again in registers with the draft kernel's own operations,
 * reads only the target outputs, and advances its chains. Same results, bit for bit. SDS_GET_X and
 * SDS_GET_TAIL are then stale after sds_sample_all. With value 1 the choice is made window by window: while
 * most drafts pass, a window is verified over many positions and reading the drafted rows back is cheaper
 * than drawing their noise a second time, so the rows are stored and read as without the option; once the
 * latest finished window needed at most L/4 + 1 positions per chain (known one window late), the rows are
 * made again. Value 2 makes them again in every window. */
#define SDS_OPT_REGEN_DRAFTS 7
/* SDS_OPT_ONEHOT_ROWS (default 1): mixtures on the tensor cores. The softmax pass stores weights below 2^-40 of
 * their row as exact zeros (either way). A row left with a single weight is one-hot: its weight is 1 and its
 * mixing sum is that component's mean. With this option the mixing GEMM skips every block of 256 rows whose
 * rows are all one-hot, and a copy kernel writes mean rows there instead (sharply peaked posteriors: late
 * diffusion steps, well separated Langevin modes). The product with an exact one-hot row is the mean itself,
 * so the results are the same bit for bit; 0 sends every block through the GEMM. Inside sds_sample_all with
 * SDS_OPT_RAW_ROWS in effect the copy is not made either: the verify and advance kernels read the skipped
 * blocks' rows from the mixture's means table by component index (SDS_GET_DQ is then stale for those rows). */
#define SDS_OPT_ONEHOT_ROWS 8
/* SDS_OPT_STAGED_WINDOWS (default 0 = off): inside sds_sample_all, for SDS_FROZEN_PREV without a projection, every
 * launch drafts, evaluates and verifies at most `stage` positions of each chain's window. A chain whose stage
 * accepted all its positions continues with the REST OF THE SAME WINDOW in the next launch: its carried output
 * stays frozen, the draws are keyed by chain and step as always, and the accept tests run in the same order, so
 * the samples (and every accept decision) are those of whole windows of L positions, bit for bit. What changes
 * is the work: rows after a rejection are never drafted nor given to the target, at the price of one more
 * sequential target call for each stage a chain passes. The paper evaluates the target on all L drafted states
 * in one batched pass (Algorithm 4); this is that window evaluated lazily, for batches in which the rows of a
 * pass are not free. nfe_calls counts the launches a chain took part in, nfe_rows the rows evaluated for it,
 * both as they really were. Values: 1..32 a fixed stage length; SDS_STAGED_ADAPTIVE: the length starts at L,
 * doubles when more than half of the chain-stages of the latest finished launch passed, halves (down to 1)
 * when fewer than an eighth did. Control word [7] counts the chain-stages that passed since reset. */
#define SDS_OPT_STAGED_WINDOWS 9
#define SDS_STAGED_ADAPTIVE 255
int sds_set_option(sds_ctx* ctx, int32_t option, int64_t value);

/* Temperature of the accept test (Appendix D, temperature rejection): a draft is accepted iff
 * log U <= (log ratio) / tau; the reflection is unchanged. tau = 1 (default) is the exact method;
 * tau > 1 accepts more and moves the output toward the draft model, tau < 1 the other way: the
 * samples then no longer follow the target law exactly. SDS_GET_ELL returns the tempered value. */
int sds_set_temperature(sds_ctx* ctx, double tau);

/* Accept test decided in the image of a matrix A (Appendix F, reflection coupling with a full
 * matrix, written in the original space): with P = A^+ A the log ratio is -(Delta + 2Z)^T P Delta / 2
 * and a rejected draft becomes m^q + sigma (Z - 2 (Z^T P Delta)/(Delta^T P Delta) Delta).
 * Q_dev: device array [r, d] of floats, ORTHONORMAL rows spanning the row space of A (so that
 * P = Q^T Q; the caller orthonormalises, the library does not check), caller-owned and alive for
 * as long as it is set; r in [1, d], d <= 16384 (else SDS_EUNSUPPORTED). NULL with r = 0 restores
 * the full-space test (the exact method). With r < d the samples no longer follow the target law;
 * the images A Y~ and A Y are maximally coupled. SDS_GET_S1 / SDS_GET_S2 then return
 * Delta^T P Delta and Z^T P Delta. The whole-chain kernel is not used while a projection is set. */
int sds_set_projection(sds_ctx* ctx, const float* Q_dev, int32_t r);

/* Same with host buffers: copies the mixture parameters means_host [ncomp, d] (float or bf16, the
 * dtype named at create) and logw_host [ncomp] (float) to the device arrays named at create
 * (NULL = keep what is on the device), runs sds_sample_all, copies the results to host memory.
 * All copies are on the bound stream. */
int sds_sample_all_host(sds_ctx* ctx, const void* means_host, const float* logw_host,
                        float* out_host, int32_t* nfe_calls_host, int32_t* nfe_rows_host);

/* Copy an internal array (selector above) to dst; dst_is_host != 0 waits for the stream. */
int sds_get(sds_ctx* ctx, int32_t what, void* dst, size_t bytes, int32_t dst_is_host);

/* Teacher forcing / resume: overwrite state Y [B,d], indices n [B], carried output Dc [B,d]
 * (device pointers; any may be NULL = keep) and rebuild the active list. */
int sds_set_state(sds_ctx* ctx, const float* Y_dev, const int32_t* n_dev, const float* Dc_dev);

/* Stand-alone target pass (kernel-level parity and timing): the context's denoiser on
 * x_dev [rows, d] at steps k_dev [rows] -> out_dev [rows, d]; rows <= B*L. */
int sds_denoise(sds_ctx* ctx, const float* x_dev, const int32_t* k_dev, int64_t rows, float* out_dev);

/* Philox normals / uniforms exactly as the path draws them (parity of the generator):
 * out_dev [nb, d] = normals(seed, stream, chain b0+i, step k); u_dev [nb] = uniform(seed, b0+i, k). */
int sds_rng_normals(uint64_t seed, int32_t stream_id, int64_t b0, int64_t nb, int32_t k, int32_t d,
                    float* out_dev, void* cuda_stream);
int sds_rng_uniforms(uint64_t seed, int64_t b0, int64_t nb, int32_t k, float* u_dev, void* cuda_stream);

/* Self-test of the device-side bounded wait used by the tensor-core kernels (their mbarrier waits
 * give up after a fixed number of polls and report SDS_ETIMEOUT instead of spinning): launches one
 * thread that waits `polls` times on a barrier nobody arrives on and stores 1 in *status_dev when
 * the wait ran out (0 would mean the barrier completed). The kernel always terminates. */
int sds_selftest_bounded_wait(int32_t polls, int32_t* status_dev, void* cuda_stream);

/* Number of kernels this context has launched since create (for launch accounting). */
int64_t sds_launch_count(const sds_ctx* ctx);

/* Per-kernel timing (measurement aid; the paper's only cost unit is the target call, Section 7).
 * sds_profile(ctx, 1) makes every later kernel launch of the context bracketed by a pair of CUDA
 * events on the bound stream; sds_profile_read waits for the stream and returns, per kernel kind,
 * the summed device time in milliseconds (ms[SDS_PROF_KINDS], host) and the number of launches
 * (launches[SDS_PROF_KINDS], host); reset != 0 clears the sums. Off by default. */
#define SDS_PROF_INIT     0
#define SDS_PROF_DENOISE  1     /* target denoiser: GEMMs of the tensor-core denoisers, or the float kernel */
#define SDS_PROF_DRAFT    2
#define SDS_PROF_VERIFY   3
#define SDS_PROF_ADVANCE  4
#define SDS_PROF_FUSED    5     /* whole-chain persistent kernel */
#define SDS_PROF_AUX      6     /* |mu|^2, list rebuild, copies of the initial call */
#define SDS_PROF_SOFTMAX  7     /* passes around the two GEMMs of a tensor-core mixture (softmax, row conversions, copies of one-hot rows) */
#define SDS_PROF_DRAFT_MODEL 8  /* every kernel of the independent draft model (SDS_INDEPENDENT) */
#define SDS_PROF_MIX      9     /* mixing GEMM of a tensor-core mixture (SDS_PROF_DENOISE then holds its logits GEMM) */
#define SDS_PROF_KINDS    10
int sds_profile(sds_ctx* ctx, int32_t enable);
int sds_profile_read(sds_ctx* ctx, double* ms, int64_t* launches, int32_t reset);

/* Mixture denoiser pass that allocates nothing and needs no context or workspace.
 * (The paper has no counterpart: this call exists for the way the library is deployed.)
 * For callers that cannot obtain device memory when they need a target pass: code running inside
 * a host application that owns the GPU memory pool, code that must not hit the implicit
 * device synchronisation of an allocation, or a process whose memory budget is fixed at start-up.
 * Computes out_dev[r] = D(x_dev[r], k_dev[r]) exactly as sds_denoise does for a float mixture:
 *   x_dev [rows, d] float, k_dev [rows] int32 in [0, K), means_dev [ncomp, d] float,
 *   logw_dev [ncomp] float, tcond_dev [K, 4] double (A, Bq, C, E per step, device), out_dev [rows, d].
 * All pointers are device pointers owned by the caller; work is enqueued on cuda_stream
 * (cudaStream_t, NULL = default stream) of the current device and the call does not wait for it.
 * The |mu_c|^2 table the kernel needs lives in a fixed array inside the library (32 KiB on every
 * GPU that loads it, until the process exits), so ncomp <= SDS_STATIC_MAX_NCOMP; larger mixtures
 * return SDS_EUNSUPPORTED and do nothing. The call never calls cudaMalloc/cudaFree or any
 * allocating routine.
 * The first call on each device looks up the array's device address; make that first call
 * outside any stream capture.
 * Every call on a device shares the one array and overwrites the entries it uses (nothing needs
 * clearing between calls); two calls whose kernels can overlap on the GPU (different streams, no
 * ordering between them) race on it - order them on one stream or with events. */
#define SDS_STATIC_MAX_NCOMP 4096
int sds_gmm_denoise_static(const float* x_dev, const int32_t* k_dev, int64_t rows, int32_t d, int32_t ncomp,
                           const float* means_dev, const float* logw_dev, const double* tcond_dev, int32_t K,
                           float* out_dev, void* cuda_stream);

const char* sds_strerror(int code);
int sds_last_cuda_error(const sds_ctx* ctx);
void sds_destroy(sds_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* SDS_H_ */
