/*
 * psgd.h -- C ABI of the B200 (sm_100a) PowerSGD+ gradient-compression library.
 *
 * One handle compresses `count` independent, equally shaped matrix variables
 * X in R^{m x n} (m >= n), each seen by N data-parallel nodes that are simulated
 * as a batch dimension on ONE GPU (problem statement: Sec. 1, Eq. (1); state of
 * the method: Algorithm 2, "Initialize").  All-Reduce Mean of Algorithm 1 is an
 * in-device mean over the node index; there is no inter-GPU communication.
 *
 * Memory layout (row-major, innermost index last), all float32 unless stated:
 *   G      [count][N][m][n]   stochastic gradients g_t^(i)            (input, read-only)
 *   E      [count][N][m][n]   residuals e_t^(i); persistent state, updated in place
 *   Q      [count][n][r]      auxiliary basis Q_{t-1}; persistent state, updated in place
 *   P_hat  [count][m][r]      orthonormal projection P~_t            (output)
 *   D_hat  [count][m][n]      global reconstruction P~ Q^T           (optional output)
 *
 * Ownership: every DEVICE buffer is allocated and owned by the caller; the
 * library never allocates or frees device memory.  `psgd_attach` hands it E, Q
 * and an opaque workspace whose size `psgd_sizes` reports.  Pointers marked
 * DEVICE must be device pointers valid on the current device; pointers marked
 * HOST are ordinary host pointers.
 *
 * Errors: argument problems return a negative psgd_status synchronously and
 * leave all state untouched.  Numerical conditions (rank-deficient P, Jacobi
 * sweeps exhausted) never abort a step: they set warning bits in a device-side
 * status word that `psgd_last_status` returns after synchronising the stream.
 * All step calls are stream-ordered and never synchronise.  A handle is not
 * thread-safe.
 */
#ifndef PSGD_H
#define PSGD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct psgd_handle psgd_handle;

/* CUDA stream passed as an opaque pointer (a cudaStream_t); NULL = default stream. */
typedef void* psgd_stream;

typedef enum {
    PSGD_OK = 0,
    PSGD_E_INVALID = -1,    /* argument out of range (m < n, r > n, r > 128, ...) */
    PSGD_E_NULL = -2,       /* required pointer is NULL */
    PSGD_E_WORKSPACE = -3,  /* workspace too small or buffers not attached */
    PSGD_E_CUDA = -4,       /* a CUDA runtime call failed; see psgd_last_cuda_error */
    PSGD_E_STATE = -5,      /* call not valid in the handle's current state */
    PSGD_E_TOO_LARGE = -6   /* problem does not fit the fixed scratch of psgd_backproject_static */
} psgd_status;

/* warning bits of the device status word */
#define PSGD_W_RANK_DEFICIENT 1 /* a pivot of the orthogonalisation fell below tolerance */
#define PSGD_W_NOT_CONVERGED 2  /* the eigen-solver of the refresh hit its sweep limit */
#define PSGD_W_TIMEOUT 4        /* a bounded wait inside a kernel ran out (results of that step are invalid) */

/* options for psgd_set_option */
#define PSGD_OPT_ERROR_FORM 1   /* 0 (default): e_i <- Delta_i - P~ Q_i^T  (Algorithm 2, last line)
                                   1: e_i <- Delta_i - P~ Q^T with the node-averaged Q */
#define PSGD_OPT_MODE 2         /* 0: eager (E holds the true residual after every step)
                                   1: deferred (E holds Delta_t = g_t + e_t; the subtraction of
                                      P~_t Q_i^T is folded into the next step's first pass;
                                      psgd_materialize_error produces the true residual).  Up to 8 columns the
                                      whole SSP step is then one pass over G and E, up to 16 two passes; above,
                                      and on refresh steps, the three-pass kernels run as in mode 0 */
#define PSGD_OPT_REFRESH_ITERS 3   /* subspace iterations q of the refresh; 0 (default): where the early sweeps run on the tensor cores 12 (blocks of
                                      32 columns and more) or 20 (8 to 31 columns), else at most 20 with the stopping test.  The start block is [Q_{t-1} | random columns] */
#define PSGD_OPT_REFRESH_OVERSAMPLE 4 /* extra columns of the refresh block (default max(8, r)) */
#define PSGD_OPT_REFRESH_TC 5      /* 1 (default): the early sweeps of a refresh whose block has >= 8 columns run
                                      on the tensor cores in TF32, the last 4 in float32; 0: float32 throughout */
#define PSGD_OPT_POWER_STEPS 6     /* K >= 1 power steps per SSP iteration (Eq. (8)); 1 (default) is PowerSGD's single
                                      step (Eq. (9)); K > 1 runs the three-pass kernels */
#define PSGD_OPT_REFRESH_ADAPTIVE 7 /* 1 (default): a refresh whose block has <= 48 columns stops its sweeps once the top-r
                                      basis has stopped moving (movement d between two checks, q = d / d_prev < 1 and d q / (1 - q) <= 1e-5,
                                      or d <= 3e-6); 0: all the sweeps */

#define PSGD_OPT_GRAD_BF16 8        /* 0 (default): the gradients G are float32; 1: bfloat16 (the same [count][N][m][n] layout, 2 bytes
                                      per element), widened exactly to float32 as they are read.  The single-pass kernel then moves
                                      10 instead of 12 bytes per element; the other paths first form M = G + E in the E buffer */

#define PSGD_OPT_SINGLE_PASS 9       /* which kernels serve the SSP steps of the deferred mode.  0 (default): the fastest known for the
                                      shape (the cluster single-pass kernel up to 4 columns, and up to 8 where its clusters have at most 4 CTAs;
                                      the two-pass kernels otherwise);
                                      1: the cluster single-pass kernel where it applies (up to 8 columns; also bfloat16 gradients);
                                      2: the two-pass kernels; 3: the L2-pipelined single-pass kernel where it applies (up to 16
                                      columns, n % 4 == 0, float32 gradients).  A choice that does not apply falls back to two passes */

#define PSGD_OPT_TRANSPOSED 10       /* 1: G, E (and D_hat, X, mom) are stored as [count][N][n][m], i.e. each matrix as the row-major
                                      n x m transpose of the m x n problem (Sec. 1: X in R^{m x n}, m >= n): a weight kept as its transpose
                                      needs no copy.  P_hat [m][r] and Q [n][r] keep their layouts.  Runs the three-pass kernels with their
                                      roles exchanged (28 bytes per element); the deferred mode and bfloat16 gradients do not apply */

#define PSGD_OPT_PENDING_TC 11       /* two-pass form of the deferred mode: which projection folds in the pending residual
                                      e = Delta - P~ Qsub^T.  0 (default): the tensor-core kernel (the rank-r product as extra MMAs,
                                      up to 32 columns, n % 4 == 0) from the number of columns on where it is the faster one, the float32
                                      kernel (up to 16 columns) below; 1: the tensor-core kernel wherever it fits; 2: never (more than 16
                                      columns then take three passes) */

#define PSGD_OPT_BACKPROJECT_TMA 12   /* 1 (default): the float32 back-projection Q_i = M_i^T P~ of 4, 8 or 16 columns stages its tiles of M
                                      by TMA in shared memory (n >= 256, n % 4 == 0, aligned pointers); 0: always the kernel that
                                      prefetches into registers.  The two add the same products in a different order */

/* buffers that psgd_debug_ptr exposes (test use only; valid until the next step) */
#define PSGD_BUF_P_NODE 1   /* P^(i)   [count][N][m][r] */
#define PSGD_BUF_Q_NODE 2   /* Q^(i)   [count][N][n][r] */
#define PSGD_BUF_P_HAT 3    /* P~      [count][m][r]    */
#define PSGD_BUF_DBAR 4     /* node mean of Delta (refresh only) [count][m][n] */
#define PSGD_BUF_P_MEAN 5   /* P       [count][m][r]    */

/* kernel families for psgd_profile_read */
#define PSGD_K_PROJECT 0
#define PSGD_K_ORTH 1
#define PSGD_K_BACKPROJECT 2
#define PSGD_K_RESIDUAL 3
#define PSGD_K_REFRESH 4
#define PSGD_K_MISC 5
#define PSGD_K_COUNT 6

/*
 * Create a handle for one matrix variable (Sec. 1: N nodes, X in R^{m x n}, m >= n;
 * Algorithm 2 "Require": rank r, restart period tau = refresh_period, N workers).
 * Requires m >= n >= r >= 1, r <= 128, N >= 1, refresh_period >= 0 (0 = never
 * refresh: plain PowerSGD, the first branch of Algorithm 2).  `seed` keys the
 * counter-based generator used for Q_{-1} (psgd_reset) and for the random start
 * block of the refresh.  Allocates host memory only.  *out is set on success.
 */
psgd_status psgd_create(int64_t m, int64_t n, int r, int N, int refresh_period, uint64_t seed,
                        psgd_handle** out);

/* Same, for `count` >= 1 independent matrices of equal shape processed by the same launches. */
psgd_status psgd_create_batch(int64_t m, int64_t n, int r, int N, int count, int refresh_period,
                              uint64_t seed, psgd_handle** out);

/* Set an option (see PSGD_OPT_*).  Must precede psgd_sizes/psgd_attach. */
psgd_status psgd_set_option(psgd_handle* h, int option, int value);

/* Byte sizes of E, Q and the workspace the caller must provide.  Any pointer may be NULL. */
psgd_status psgd_sizes(const psgd_handle* h, size_t* e_bytes, size_t* q_bytes, size_t* workspace_bytes);

/*
 * Hand the handle its DEVICE buffers: E and Q (persistent state, Algorithm 2
 * "Initialize") and the workspace.  All three must be 256-byte aligned and stay
 * valid until psgd_destroy.  The contents of E and Q are taken as the current
 * state (e_t, Q_{t-1}); call psgd_reset to initialise them.
 */
psgd_status psgd_attach(psgd_handle* h, float* E /*DEVICE*/, float* Q /*DEVICE*/,
                        void* workspace /*DEVICE*/, size_t workspace_bytes);

/* e_0 = 0, Q_{-1} ~ N(0,1) from the seed (same on every node), t = 0.  (Algorithm 2, "Initialize") */
psgd_status psgd_reset(psgd_handle* h, psgd_stream stream);

/*
 * One iteration t of Algorithm 2 without the optimizer update:
 *   Delta_i = g_i + e_i (Eq. (7a));  SVD-Comp if refresh_period > 0 and
 *   t mod refresh_period == 0, else SSP-Comp (Algorithm 1);  e_i <- Delta_i - Delta^_i;  t <- t + 1.
 * G: DEVICE, read-only, float32 (bfloat16 with PSGD_OPT_GRAD_BF16).  P_hat (DEVICE, may be NULL) receives P~_t.  D_hat
 * (DEVICE, may be NULL) receives the dense global reconstruction P~_t Q_t^T.
 * Q (attached) is replaced by Q_t.  Enqueued on `stream`; does not synchronise.
 */
psgd_status psgd_step(psgd_handle* h, const void* G, float* P_hat, float* D_hat, psgd_stream stream);

/* The same iteration with SVD-Comp forced (Algorithm 1, second function; Definition 3). */
psgd_status psgd_refresh(psgd_handle* h, const void* G, float* P_hat, float* D_hat, psgd_stream stream);

/*
 * The optimizer step after the iteration, for momentum SGD (Eq. (7c)):  m_t = mu m_{t-1} + D^_t,
 * X_{t+1} = X_t - eta m_t,  with D^_t = P~_t Q_t^T of the last psgd_step / psgd_refresh, formed on the fly and
 * never stored.  X, mom: DEVICE, [count][m][n] float32, updated in place.  PSGD_E_STATE before the first step.
 */
psgd_status psgd_msgd_update(psgd_handle* h, float* X, float* mom, float eta, float mu, psgd_stream stream);

/*
 * psgd_step with HOST buffers: copies G_host into the caller's DEVICE staging
 * buffer G_stage (same size as G), runs the step, copies P~ and Q_t back to
 * P_hat_host / Q_host (either may be NULL) and synchronises the stream.
 * Pinned host memory makes the copies asynchronous with respect to the host.
 */
psgd_status psgd_step_host(psgd_handle* h, const void* G_host /*HOST*/, void* G_stage /*DEVICE*/,
                           float* P_hat_host /*HOST*/, float* Q_host /*HOST*/, psgd_stream stream);

/*
 * Deferred mode only: turn the stored Delta_t back into the true residual
 * e_{t+1} = Delta_t - P~_t Q_i^T (Algorithm 2, last line) in place.  A no-op when
 * E already holds the residual.  Call before reading or checkpointing E.
 */
psgd_status psgd_materialize_error(psgd_handle* h, psgd_stream stream);

/* Tell the handle that the caller overwrote E (and Q) with a true residual / basis. */
psgd_status psgd_state_written(psgd_handle* h);

psgd_status psgd_get_step(const psgd_handle* h, int64_t* t);
psgd_status psgd_set_step(psgd_handle* h, int64_t t);

/* Synchronise `stream`, return the warning bits accumulated since the last call in *flags, clear them. */
psgd_status psgd_last_status(psgd_handle* h, psgd_stream stream, int* flags /*HOST*/);

/* Test hook: DEVICE address and byte size of an internal buffer (PSGD_BUF_*). */
psgd_status psgd_debug_ptr(psgd_handle* h, int which, void** ptr, size_t* bytes);

/*
 * Launch plan and deferred-mode state of the handle, 12 ints (HOST): [0] 1 if the single-pass kernel
 * serves this shape in deferred mode, [1] rank padding, [2] columns per CTA, [3] CTAs per cluster,
 * [4] row slots per matrix, [5] clusters resident at once (-1 before the first single-pass launch),
 * [6] its dynamic shared memory in bytes, [7] row chunks of the eager back-projection, [8] 1 while E
 * holds Delta_t and the residual is still pending (deferred mode), [9] 1 if that pending residual is
 * the single-pass kernel's (padded factors in place), [10] multiprocessors of the device that was
 * current when the handle was created (148 when none was visible), [11] what ran the last
 * step: 0 the three- or two-pass kernels, 1 the cluster single-pass kernel, 2 the L2-pipelined single-pass kernel,
 * 3 the two-pass kernels with the pending residual folded in on the tensor cores (PSGD_OPT_PENDING_TC).
 */
psgd_status psgd_plan_info(const psgd_handle* h, int* info /*HOST*/);

/* Number of kernels this handle has launched since creation. */
psgd_status psgd_launch_count(const psgd_handle* h, int64_t* launches);

/*
 * Per-family kernel timing with CUDA events recorded on the launching stream.
 * psgd_profile_begin enables it; psgd_profile_read synchronises the events,
 * returns accumulated milliseconds and launch counts per family
 * (arrays of PSGD_K_COUNT entries, HOST) and disables it again.
 */
psgd_status psgd_profile_begin(psgd_handle* h);
psgd_status psgd_profile_read(psgd_handle* h, float* ms /*HOST*/, int* launches /*HOST*/);

/* Text of the last CUDA error seen by this handle (static storage; never NULL). */
const char* psgd_last_cuda_error(const psgd_handle* h);

/* Frees host memory of the handle.  Never touches caller-owned device buffers. */
psgd_status psgd_destroy(psgd_handle* h);

/*
 * One iteration of Algorithm 2 with the nodes spread over several processes (one or more nodes per GPU).  Algorithm 2
 * averages three arrays over the nodes: P = mean_i P_i, Q = mean_i Q_i and, when t mod tau = 0, Delta = mean_i (g_i + e_i).
 * A handle created with N nodes forms the mean over ITS nodes; the caller averages over the processes between the phases
 * (an all-reduce with the mean as its operation, every process holding the same N) and hands the result back:
 *
 *   psgd_exchange_plan   whether the next step is a refresh (t mod tau = 0, or force_refresh) and how many floats each exchange carries:
 *                        first = count*m*r (P), or count*m*n at a refresh (Delta); second = count*n*r (Q)
 *   psgd_exchange_begin  M_i = G_i + e_i, then `first` <- local mean of P_i = M_i Q_{t-1} (at a refresh: of M_i,
 *                        in storage orientation)
 *        ... caller: first <- mean over processes of first ...
 *   psgd_exchange_orth   P~ = orth(first) (at a refresh: SVD-Comp on first), then `second` <- local mean of Q_i = M_i^T P~
 *        ... caller: second <- mean over processes of second ...
 *   psgd_exchange_end    Q_t <- second, e_{t+1,i} = M_i - P~ Q_i^T (or - P~ Q_t^T, PSGD_OPT_ERROR_FORM = 1), P_hat and
 *                        D_hat as in psgd_step, t <- t + 1
 *
 * `first` and `second` are DEVICE arrays of the caller (16-byte aligned; typically slots of one flat buffer per exchange that
 * serves all handles of a model, so that each exchange is one all-reduce); the library reads and writes them in stream
 * order and keeps no pointer to them.  All processes must use the same seed, options and step count: each then factorises
 * the same averaged array with the same deterministic kernels and obtains the same P~.  With one process the three phases
 * equal psgd_step (eager mode) or its two-pass form (PSGD_OPT_MODE = 1: up to 16 columns the residual stays pending in E);
 * the single-pass kernels are not used.  PSGD_E_INVALID: phases out of order, PSGD_OPT_POWER_STEPS > 1, misaligned arrays.
 */
psgd_status psgd_exchange_plan(const psgd_handle* h, int force_refresh, int* refresh, size_t* first_floats, size_t* second_floats);
psgd_status psgd_exchange_begin(psgd_handle* h, const void* G, int force_refresh, float* first, psgd_stream stream);
psgd_status psgd_exchange_orth(psgd_handle* h, const float* first, float* second, psgd_stream stream);
psgd_status psgd_exchange_end(psgd_handle* h, const float* second, float* P_hat, float* D_hat, psgd_stream stream);

/*
 * Several handles of different shapes stepped by ONE call (a model's matrices come in a few shape classes: Sec. 5 trains
 * LLaMA- and RoBERTa-style stacks).  Each handle runs on a stream of the group's own, forked from `stream` and joined back into
 * it, so that the small finishing kernels and the ragged last wave of one class overlap the streaming kernels of the others; for
 * the caller's stream the call is one stream-ordered operation.  The handles share nothing, so the results equal those of
 * stepping them one after the other bit for bit.  psgd_group_create creates CUDA streams and events on the current device (no
 * device memory); handles must outlive the group.  G[i] / P_hat[i] (DEVICE; P_hat[i] and P_hat itself may be NULL) belong to handle i.
 */
typedef struct psgd_group psgd_group;
psgd_status psgd_group_create(psgd_handle* const* handles /*HOST*/, int count, psgd_group** out);
psgd_status psgd_group_step(psgd_group* g, const void* const* G /*HOST array of DEVICE pointers*/,
                            float* const* P_hat /*HOST array of DEVICE pointers, or NULL*/, psgd_stream stream);
psgd_status psgd_group_destroy(psgd_group* g);

/*
 * The tensor-core contraction the refresh uses for its early subspace sweeps (SVD-Comp of
 * Algorithm 1 computed by block subspace iteration; Definition 3 fixes what it converges to):
 *     C[c] = A[c] B[c]^T,   A [count][M][K],  B [count][Nc][K],  C [count][M][Nc],
 * all DEVICE, float32, row-major.  Operands are read as TF32 (the 13 low mantissa bits are
 * ignored), products are accumulated in float32.  Requires Nc <= 256, K % 4 == 0, A and B
 * 16-byte aligned.  `scratch` (DEVICE, 256-byte aligned) must hold the bytes that
 * psgd_gemm_nt_tf32_scratch reports; its first word is used as a status word.  Synchronises the
 * stream before returning; PSGD_E_STATE means a bounded wait inside the kernel ran out.
 */
psgd_status psgd_gemm_nt_tf32_scratch(int64_t M, int64_t Nc, int64_t K, int count, size_t* scratch_bytes /*HOST*/);
psgd_status psgd_gemm_nt_tf32(const float* A /*DEVICE*/, const float* B /*DEVICE*/, float* C /*DEVICE*/, int64_t M,
                              int64_t Nc, int64_t K, int count, void* scratch /*DEVICE*/, size_t scratch_bytes,
                              psgd_stream stream);

/*
 * Back-projection without a workspace.  (An addition of this library: the paper has no
 * counterpart; the operation itself is the Q^(i) <- Delta^(i)^T P~ / All-Reduce-Mean pair of
 * Algorithm 1.)
 *
 * Some callers cannot allocate device memory at all: a plug-in running inside a serving
 * process whose memory pool already owns the whole GPU, code that runs where cudaMalloc is
 * not allowed or would stall every stream on the device, or a tightly budgeted job that was
 * given fixed input/output buffers and nothing else.  The handle API above needs a workspace
 * from them; this call does not.  It computes, for ONE matrix on N nodes,
 *     Q_node[i] = M[i]^T P_hat   (i = 0..N-1)      and      Q_mean = (1/N) sum_i Q_node[i]
 * with M [N][m][n], P_hat [m][r], Q_node [N][n][r] (may be NULL), Q_mean [n][r]; all DEVICE,
 * float32, row-major, caller-owned.  The partial sums over row chunks go to a fixed array of
 * PSGD_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU that loads the
 * library gives up that much memory until the process exits.
 *
 * Limits and rules:
 *  - N * n * r * 4 bytes must not exceed PSGD_STATIC_SCRATCH_BYTES, otherwise PSGD_E_TOO_LARGE
 *    is returned and nothing is launched; m >= n >= r >= 1, r <= 128 as elsewhere.
 *  - The first call on each device looks up the array's device address (a CUDA runtime query,
 *    no allocation); make that first call outside any stream capture.
 *  - The call allocates and frees nothing and does not synchronise.
 *  - All calls on a device share the one array, and it keeps whatever the previous call left
 *    there.  Each call overwrites every entry it later reads, so stale contents are harmless,
 *    but two calls that may run at the same time on the GPU (different streams) race on it:
 *    keep all calls on one stream or order them yourself.
 */
#define PSGD_STATIC_SCRATCH_BYTES (8u << 20)
psgd_status psgd_backproject_static(const float* M /*DEVICE*/, const float* P_hat /*DEVICE*/,
                                    float* Q_node /*DEVICE*/, float* Q_mean /*DEVICE*/,
                                    int64_t m, int64_t n, int r, int N, psgd_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* PSGD_H */
