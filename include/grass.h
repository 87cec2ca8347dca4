/*
 * grass.h -- C ABI of the GRASS per-layer structured-sparse gradient step for
 * NVIDIA B200 (sm_100a).
 *
 * GRASS (arXiv 2406.17660) trains a linear layer W (m x n) through a sparse
 * projection P = (rho B)^T that keeps r of the m gradient rows.  With dY (T x m)
 * the gradient w.r.t. the layer's outputs and X (T x n) its inputs, one
 * iteration of the paper's Algorithm 1 is: every K iterations pick the rows
 * (compute_P, Section 3.2); then G_C = P^T (dY^T X) without forming the m x n
 * gradient (Section 3.1), Adam on the r x n state (Appendix A), and
 * W <- W + alpha P Delta on the r picked rows only (Section 3.1).
 *
 * Conventions shared by every call
 *   - Every pointer is a DEVICE pointer unless it is marked "host".  The caller
 *     owns all buffers; the library allocates no device memory and keeps no
 *     state between calls except one small per-device status word (see
 *     grass_device_status).
 *   - Matrices are row-major; a leading dimension `ld*` is the row pitch in
 *     ELEMENTS and must be >= the row length.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls only enqueue work and return; nothing synchronises except
 *     grass_device_status.
 *   - The return value is a grass_status_t.  Argument errors are detected on
 *     the host, nothing is launched and no output is touched.  Conditions only
 *     the device can see (degenerate norms, a row index outside [0, m), a wait
 *     that ran out) are recorded in the status word and the affected outputs
 *     are left unwritten where that is possible; no kernel traps or aborts.
 *   - Rows are 0-based.  sigma (the paper's sigma_j) is int32 `idx[r]`, the
 *     diagonal of rho is fp32 `rho[r]`: the "2r numbers" storage of P
 *     (Section 3.1, "Efficient Storage of P").
 */
#ifndef GRASS_B200_H_
#define GRASS_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GRASS_OK = 0,
  GRASS_ERR_INVALID_ARG = 1, /* NULL pointer, bad size, r > m, ld < row length, idx out of range */
  GRASS_ERR_ALIGNMENT = 2,   /* a pointer or pitch misses the alignment a path needs */
  GRASS_ERR_UNSUPPORTED = 3, /* dtype or method this build does not implement */
  GRASS_ERR_DEGENERATE = 4,  /* norms negative / non-finite, or all zero for a sampling method */
  GRASS_ERR_WORKSPACE = 5,   /* workspace NULL, misaligned or smaller than *_workspace_bytes */
  GRASS_ERR_CUDA = 6,        /* a CUDA runtime or driver call failed (see stderr) */
  GRASS_ERR_TIMEOUT = 7      /* a bounded device-side wait ran out */
} grass_status_t;

typedef enum { GRASS_F32 = 0, GRASS_BF16 = 1 } grass_dtype_t;

typedef enum {
  GRASS_SEL_TOPR = 0,                 /* Section 3.2 B */
  GRASS_SEL_MULTINOMIAL_NORM = 1,     /* Section 3.2 A, Theorem 1: q ~ norm, with replacement */
  GRASS_SEL_MULTINOMIAL_NORM2 = 2,    /* q ~ norm^2 (subspace preservation), with replacement */
  GRASS_SEL_UNIFORM = 3,              /* q = 1/m, with replacement */
  GRASS_SEL_MULTINOMIAL_NORM_NR = 4,  /* the three distributions without replacement ("-NR") */
  GRASS_SEL_MULTINOMIAL_NORM2_NR = 5,
  GRASS_SEL_UNIFORM_NR = 6
} grass_sel_t;

/*
 * Row norms lambda_k = ||G[k, :]||_2 of a formed gradient (Section 3.2; the
 * "mn" term of compute_P in the paper's summary table).
 *   G      m x n, dtype `dt`, row pitch ldg; read only.
 *   norms  [m] fp32, written.
 * Accumulates in fp32.  Any alignment is accepted (128-bit loads are used when
 * G and ldg allow them).
 */
int grass_row_norms(const void* G, int dt, int64_t m, int64_t n, int64_t ldg,
                    float* norms, void* stream);

/*
 * compute_P (Section 3.2): choose sigma and rho from the row norms.
 *   GRASS_SEL_TOPR: rho = 1, sigma = the r largest norms; equal norms go to
 *     the lower row index.
 *   With replacement (GRASS_SEL_MULTINOMIAL_NORM, _NORM2, GRASS_SEL_UNIFORM):
 *     sigma_j i.i.d. ~ Multinomial(1, q), q_k = w_k / sum(w) with w = lambda,
 *     lambda^2 or 1, rho_j = 1 / sqrt(r q_{sigma_j}).  Draw j inverts
 *     the fp64 running sum of the weights at u_j * sum, u_j = w_j * 2^-32, where
 *     w_j is word (j mod 4) of Philox4x32-10 with key (seed low, seed high) and
 *     counter (j div 4, layer_id, epoch, 0x47524153): sigma_j = min{k : c_k >
 *     u_j * sum}.  The result is a pure function of (norms, seed, layer_id,
 *     epoch); no generator state is kept.
 *   Without replacement (the _NR methods): r distinct rows, rho = 1.  The paper
 *     does not say how the draws are made; here row k scores w_k / (-log u_k),
 *     u_k = (word_k + 1/2) * 2^-32 with word_k = Philox word (k mod 4) of counter
 *     (k div 4, layer_id, epoch, 0x47524153), the score is rounded to fp32, and
 *     the r largest scores win (equal scores: lower row).  This exponential race
 *     has exactly the distribution of r successive draws, each from q restricted
 *     to the rows not yet drawn.  Fewer than r rows of positive weight:
 *     GRASS_ERR_DEGENERATE.
 *   norms  [m] fp32, read only.     idx [r] int32 and rho [r] fp32, written,
 *   ascending by row (repeated rows are adjacent).
 *   ws     scratch of at least grass_select_workspace_bytes(m, r, method)
 *          bytes, 256-byte aligned; contents need not survive the call.
 * 1 <= r <= m < 2^31.  If a norm is negative, NaN or infinite, or all are zero
 * under a sampling method, idx and rho are left unwritten and the status word
 * is set to GRASS_ERR_DEGENERATE.
 */
size_t grass_select_workspace_bytes(int64_t m, int32_t r, int method);
int grass_select(const float* norms, int64_t m, int32_t r, int method, uint64_t seed,
                 uint32_t layer_id, uint32_t epoch, int32_t* idx, float* rho, void* ws,
                 size_t ws_bytes, void* stream);

/*
 * grass_select without a workspace argument, for callers that cannot obtain
 * device memory at the point of the call (the paper has no counterpart; it is
 * a packaging variant of the call above and computes exactly the same idx and
 * rho).  Typical callers: an optimizer hook running inside a framework whose
 * pooling allocator already owns the whole device, so that a raw cudaMalloc
 * would fail; a plugin that is handed tensors but no allocator; a step on a
 * latency-critical path where the device-wide synchronisation an allocation
 * implies is not acceptable.  The scratch (room for the fp64 running sum and
 * the per-row hit counters) lives in a fixed array inside the library image:
 * GRASS_SELECT_STATIC_MAX_M rows, 12 bytes each (192 KiB), held by every GPU
 * that loads the library until the process exits.  How much of it a call
 * touches: the kernel stages the hit counters in shared memory for every m this
 * call accepts, and the running sum too while m <= 12800, so only the
 * running-sum part of the array is ever used, and only by the sampling methods
 * with replacement at 12800 < m <= 16384 (the 13824-row LLaMA-13B projections);
 * all other calls leave the array alone.
 *   - m > GRASS_SELECT_STATIC_MAX_M returns GRASS_ERR_WORKSPACE (and says so on
 *     stderr); nothing is launched.  All other arguments and errors are as for
 *     grass_select.
 *   - The call allocates nothing, on the host or the device.  The first call
 *     on each device looks up the array's device address (with that device
 *     current) and caches it; make that first call during start-up, outside
 *     any stream capture.
 *   - All calls on a device share the one array, which still holds what the
 *     previous call left there.  The kernel overwrites or zeroes every entry
 *     before reading it, so calls that follow one another on a stream are
 *     independent; two calls that may run at the same time on one GPU (two
 *     streams, two host threads) race on the array and must be serialised by
 *     the caller.
 */
#define GRASS_SELECT_STATIC_MAX_M 16384
int grass_select_static(const float* norms, int64_t m, int32_t r, int method, uint64_t seed,
                        uint32_t layer_id, uint32_t epoch, int32_t* idx, float* rho,
                        void* stream);

/*
 * Projected gradient (Section 3.1, "Efficient Gradient Projection"):
 *   Gc[j, c] = rho_j * sum_t dY[t, idx_j] * X[t, c],   j < r, c < n,
 * i.e. rho ((B dY^T) X); the m x n gradient is never formed.
 *   dY   T x m, pitch lddy;  X  T x n, pitch ldx;  both dtype `dt`, read only.
 *   idx  [r] int32 rows in [0, m); may repeat.  NULL means the identity
 *        (requires r == m): the call then returns the dense gradient dY^T X,
 *        which is what a refresh iteration feeds to grass_row_norms.
 *   rho  [r] fp32 or NULL (all ones).
 *   Gc   r x n fp32, pitch ldgc, written.
 *   ws   scratch of at least grass_project_workspace_bytes(T, m, n, r, dt)
 *        bytes, 256-byte aligned.
 * GRASS_BF16 runs on the tensor cores (bf16 products, fp32 accumulation) and
 * needs X 16-byte aligned with ldx a multiple of 8 (and the same of dY / lddy
 * when idx is NULL), else GRASS_ERR_ALIGNMENT.  GRASS_F32 uses fp32 FMA and
 * accepts any alignment.  The sum over tokens is split into a fixed number of
 * slices added in a fixed order: results are bit-reproducible run to run.
 * A row index outside [0, m) contributes zeros and sets the status word.
 * GRASS_BF16: T <= 2 097 120 tokens (GRASS_ERR_UNSUPPORTED beyond: token slices are
 * kept in a 16-bit table of 32- to 128-token units).
 */
size_t grass_project_workspace_bytes(int64_t T, int64_t m, int64_t n, int32_t r, int dt);
int grass_project_grad(const void* dY, int64_t lddy, const void* X, int64_t ldx, int dt,
                       int64_t T, int64_t m, int64_t n, const int32_t* idx, const float* rho,
                       int32_t r, float* Gc, int64_t ldgc, void* ws, size_t ws_bytes,
                       void* stream);

/*
 * Row norms of the weight gradient without forming it (Section 3.1 "Memory
 * savings" applied to compute_P of Section 3.2):
 *   norms[k] = || (dY^T X)[k, :] ||_2,   k < m.
 * The paper's refresh iteration computes the full gradient once to take its row
 * norms; here the dense GEMM's epilogue reduces the squares of each output tile
 * and the m x n matrix is never written.  Arguments as for grass_project_grad
 * with idx = NULL; norms [m] fp32 is written; ws needs
 * grass_grad_row_norms_workspace_bytes(T, m, n, dt) bytes (GRASS_BF16: m * n / 8
 * bytes of per-column-group partial sums, added in a fixed order; a gradient too
 * small to occupy the GPU unsplit is instead summed over token slices in fp32
 * scratch and reduced from there; GRASS_F32: the fp32 path forms the small
 * gradient in ws and calls grass_row_norms).  Every square is taken of a complete
 * dot product.
 */
size_t grass_grad_row_norms_workspace_bytes(int64_t T, int64_t m, int64_t n, int dt);
int grass_grad_row_norms(const void* dY, int64_t lddy, const void* X, int64_t ldx, int dt,
                         int64_t T, int64_t m, int64_t n, float* norms, void* ws, size_t ws_bytes,
                         void* stream);

/*
 * adam.update on the subspace state (Appendix A):
 *   M <- beta1 M + (1 - beta1) Gc;  V <- beta2 V + (1 - beta2) Gc^2;
 *   U = -lr * (M / (1 - beta1^step)) / (sqrt(V / (1 - beta2^step)) + eps).
 *   Gc r x n fp32 (pitch ldgc), read only.  M, V updated in place and U
 *   written, all r x n fp32 with pitch ldstate.  U may alias Gc.
 *   step >= 1 counts the updates since M and V were last zeroed (the paper's
 *   update_state reset is a memset by the caller plus step = 1).
 * Hyper-parameters are doubles so that 1 - beta is formed without first
 * rounding beta to fp32; the element arithmetic is fp32.
 */
int grass_subspace_adam(const float* Gc, int64_t ldgc, float* M, float* V, float* U,
                        int64_t ldstate, int32_t r, int64_t n, double lr, double beta1,
                        double beta2, double eps, int32_t step, void* stream);

/*
 * Row-sparse apply (Algorithm 1 "Apply update"; Section 3.1 "Efficient Weight
 * Update"):  W <- W + alpha P U, i.e. W[idx_j, :] += alpha * rho_j * U[j, :].
 *   W    m x n, dtype wdt, pitch ldw, updated in place; rows not in idx are
 *        not read or written.
 *   U    r x n fp32, pitch ldu.   rho NULL = ones.
 *   idx  [r] ascending (as grass_select writes it); repeated rows must be
 *        adjacent: their terms are summed in fp32 in order of j and the row is
 *        written once (bf16: one round-to-nearest-even at the end).
 * A row index outside [0, m) is skipped and sets the status word.  r <= 65535
 * (one grid row per selected row).
 */
int grass_scatter_update(void* W, int wdt, int64_t m, int64_t n, int64_t ldw, const float* U,
                         int64_t ldu, const int32_t* idx, const float* rho, int32_t r,
                         double alpha, void* stream);

/*
 * grass_subspace_adam followed by grass_scatter_update in one kernel (the two
 * steps of Algorithm 1 after the projection; both are local to a selected row).
 * Arguments as for the two calls; M and V are updated in place, W's selected rows
 * are updated in place, and U is written only if it is not NULL (the update then
 * never touches HBM: 24 bytes per element instead of 36).  Results are
 * bit-identical to calling the two functions in turn.  idx ascending, repeats
 * adjacent (every repeat keeps its own state row; the W row is written once).
 */
int grass_adam_scatter(const float* Gc, int64_t ldgc, float* M, float* V, float* U,
                       int64_t ldstate, void* W, int wdt, int64_t m, int64_t n, int64_t ldw,
                       const int32_t* idx, const float* rho, int32_t r, double lr, double beta1,
                       double beta2, double eps, int32_t step, double alpha, void* stream);

/*
 * The two per-step calls for up to 8 layers of one shape in a single set of
 * launches (the paper applies the same step to every linear layer; the q, k, v, o
 * projections of a block share a shape, as do gate and up).  Small layers are
 * bound by per-launch costs and by split-K partial traffic; one launch over
 * `count` layers has `count` times the tiles, so it needs a `count` times smaller
 * token split.  Every array argument is a HOST array of `count` device pointers;
 * layer g uses dY[g], X[g], idx[g] (required), rho[g] (the array or an entry may be
 * NULL), Gc[g], and M[g], V[g], U[g] (array or entries may be NULL), W[g].  All
 * layers share T, m, n, r, the pitches, the dtype (GRASS_BF16 for the projection)
 * and the hyper-parameters.  Results are bit-identical to `count` separate
 * bit-reproducible calls only where the token split is the same; in general they
 * agree to fp32 summation order.  ws needs
 * grass_project_batched_workspace_bytes(count, T, m, n, r) bytes.
 */
size_t grass_project_batched_workspace_bytes(int32_t count, int64_t T, int64_t m, int64_t n,
                                             int32_t r);
int grass_project_grad_batched(int32_t count, const void* const* dY, int64_t lddy,
                               const void* const* X, int64_t ldx, int64_t T, int64_t m, int64_t n,
                               const int32_t* const* idx, const float* const* rho, int32_t r,
                               float* const* Gc, int64_t ldgc, void* ws, size_t ws_bytes,
                               void* stream);
int grass_adam_scatter_batched(int32_t count, const float* const* Gc, int64_t ldgc,
                               float* const* M, float* const* V, float* const* U, int64_t ldstate,
                               void* const* W, int wdt, int64_t m, int64_t n, int64_t ldw,
                               const int32_t* const* idx, const float* const* rho, int32_t r,
                               double lr, double beta1, double beta2, double eps, int32_t step,
                               double alpha, void* stream);

/*
 * grass_project_grad_batched with the tiling decisions exposed (the paper has no
 * counterpart: it leaves the product rho ((B dY^T) X) of Section 3.1 to a library
 * matmul).  By default the library chooses, from (T, m, n, r, count) alone, the
 * output tile of a CTA, whether two CTAs share each MMA, into how many token slices
 * the sum over T is split, and how the selected columns of dY reach the tensor
 * cores.  A grass_project_opts_t (host pointer; NULL = all defaults) overrides any
 * of these; 0 in a field keeps the default.  Every choice computes the same sums;
 * results differ only in fp32 summation order (the token slices), and are
 * bit-reproducible for fixed options.
 *   gather            GRASS_GATHER_PREPASS: a separate kernel first copies the r
 *                       selected columns into a token-major T x r matrix in ws
 *                       (T <= 2 097 120 tokens, GRASS_ERR_UNSUPPORTED beyond).
 *                     GRASS_GATHER_IN_CTA: every CTA of the GEMM picks the columns
 *                       of its own tile straight into shared memory (tiles of at
 *                       most 128 selected rows; otherwise the default is used).
 *                     GRASS_GATHER_COOPERATIVE: all CTAs of the GEMM share one pass
 *                       over dY while the MMAs run; the picked columns travel
 *                       through the T x r matrix in ws, chunk by chunk.
 *   n_blocks_per_cta  1, 2 or 4 blocks of 128 columns of n per CTA (ignored if the
 *                     accumulators would not fit).
 *   cta_pair          GRASS_PAIR_NEVER / GRASS_PAIR_ALWAYS (where r allows it).
 *   token_slices      number of slices of T (clamped to what T allows).
 *   gather_warps      GRASS_GATHER_COOPERATIVE only: how many of a CTA's eight gather
 *                     warps take part (1..8).
 * grass_project_plan reports what a call with these arguments would do, and the
 * workspace it needs, without touching the GPU (plan: host pointer, written).
 * grass_project_grad_ex takes the arguments of grass_project_grad_batched plus
 * opts; ws needs plan->workspace_bytes bytes for the same arguments.
 */
enum { GRASS_GATHER_AUTO = 0, GRASS_GATHER_PREPASS = 1, GRASS_GATHER_IN_CTA = 2,
       GRASS_GATHER_COOPERATIVE = 3 };
enum { GRASS_PAIR_AUTO = 0, GRASS_PAIR_NEVER = 1, GRASS_PAIR_ALWAYS = 2 };
typedef struct {
  int32_t gather;
  int32_t n_blocks_per_cta;
  int32_t cta_pair;
  int32_t token_slices;
  int32_t gather_warps;
} grass_project_opts_t;
typedef struct {
  int32_t gather;            /* GRASS_GATHER_* actually used */
  int32_t rows_per_tile;     /* selected rows per CTA tile (a multiple of 64) */
  int32_t row_blocks;        /* tiles along r */
  int32_t n_blocks_per_cta;
  int32_t ctas_per_slice;    /* CTAs that share one token slice, over all `count` layers */
  int32_t cta_pair;          /* 1: two CTAs per MMA */
  int32_t token_slices;      /* slices of T, each summed into its own fp32 partial */
  int32_t short_slices;      /* how many of them are the short slices that fill the last wave */
  int32_t long_slice_tokens; /* tokens in the first slice */
  int32_t tokens_per_stage;  /* tokens per pipeline stage (32 or 64) */
  int32_t stages;
  size_t workspace_bytes;
} grass_project_plan_t;
int grass_project_plan(int32_t count, int64_t T, int64_t m, int64_t n, int32_t r,
                       const grass_project_opts_t* opts, grass_project_plan_t* plan);
int grass_project_grad_ex(int32_t count, const void* const* dY, int64_t lddy,
                          const void* const* X, int64_t ldx, int64_t T, int64_t m, int64_t n,
                          const int32_t* const* idx, const float* const* rho, int32_t r,
                          float* const* Gc, int64_t ldgc, void* ws, size_t ws_bytes,
                          const grass_project_opts_t* opts, void* stream);

/*
 * Column form of the apply step, for layers projected on their input dimension
 * (Section 4.1: P acts on the smaller dimension of the gradient, so for m > n
 * the selection picks r of the n columns, G_C = G_W P, and W <- W + alpha U^T P^T):
 *   W[c, idx_j] += alpha * rho_j * U[j, c],   c < m.
 * U is r x m fp32 (the transpose of the m x r projected update, which is what
 * grass_project_grad returns when it is called with dY and X exchanged: select
 * columns of X, contract with dY).  idx ascending in [0, n), repeats adjacent and
 * summed in fp32 in order of j, each element of W rounded once.
 */
int grass_scatter_update_cols(void* W, int wdt, int64_t m, int64_t n, int64_t ldw, const float* U,
                              int64_t ldu, const int32_t* idx, const float* rho, int32_t r,
                              double alpha, void* stream);

/*
 * Read and clear the current device's status word.  Synchronises `stream`.
 * Returns GRASS_OK or the first error a kernel recorded since the last call;
 * if detail (host pointer, may be NULL) is given it receives a kernel-specific
 * value (the offending row index, or the stage a wait gave up in).
 */
int grass_device_status(void* stream, int32_t* detail);

const char* grass_status_string(int status);

/*
 * Self-test of the bounded device-side wait (the paper has no counterpart).  Every
 * mbarrier wait in the projection kernel gives up after a fixed number of SM clocks,
 * records GRASS_ERR_TIMEOUT and lets the kernel return instead of spinning forever.
 * This call launches one thread that waits on a barrier nothing completes, for at
 * most limit_cycles (1 .. 2e9) clocks; afterwards grass_device_status reports
 * GRASS_ERR_TIMEOUT with detail 900 and the context stays usable.
 */
int grass_selftest_bounded_wait(int64_t limit_cycles, void* stream);

/*
 * Per-launch timing of the library's own kernels (a measurement aid; the paper
 * has no counterpart).  Between grass_profile_begin and grass_profile_end every
 * kernel the library launches on the calling thread's behalf is bracketed by a
 * pair of CUDA events recorded on the launch stream, up to max_launches
 * launches (later ones are counted but not timed).  grass_profile_end
 * synchronises the device, writes for launch i its kernel id (grass_kernel_t)
 * and duration in milliseconds to the HOST arrays kernel_id[i] and ms[i]
 * (each of capacity max_launches; either may be NULL), returns the number of
 * launches seen in *n_launches (host) and releases the events.  Not
 * thread-safe; one profile at a time per process.
 */
typedef enum {
  GRASS_K_ROW_NORMS = 0,
  GRASS_K_SELECT = 1,
  GRASS_K_GATHER = 2,        /* copy of the selected dY columns */
  GRASS_K_PROJECT_TC = 3,    /* tcgen05 projection GEMM on the r selected rows */
  GRASS_K_SPLITK_REDUCE = 4,
  GRASS_K_PROJECT_FP32 = 5,
  GRASS_K_ADAM = 6,
  GRASS_K_SCATTER = 7,
  GRASS_K_ADAM_SCATTER = 8,  /* fused Adam + apply */
  GRASS_K_PROJECT_TC_DENSE = 9  /* the same GEMM kernel on all m rows (idx = NULL): dense gradient
                                   or its row norms, i.e. the launches of a refresh iteration */
} grass_kernel_t;
int grass_profile_begin(int32_t max_launches);
int grass_profile_end(int32_t* kernel_id, float* ms, int32_t* n_launches);
/* The same, plus start_ms[i] (host, may be NULL): when launch i began, in milliseconds after
 * the first recorded launch began -- across streams, so overlap between streams is visible. */
int grass_profile_end_timeline(int32_t* kernel_id, float* ms, float* start_ms,
                               int32_t* n_launches);

#ifdef __cplusplus
}
#endif
#endif /* GRASS_B200_H_ */
