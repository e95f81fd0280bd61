/*
 * tgrad.h -- C ABI of the B200 (sm_100a) TensorGRaD optimizer-step library.
 *
 * One state object per complex weight tensor W in C^{I_1 x ... x I_N}.  A step
 * is Algorithm 1 of the paper ("Adam with Sparse and Low-Rank Gradient
 * Compression"): the gradient is split into an unstructured sparse part
 * (magnitude top-k index set Omega, Section 2.2 "Unstructured sparse gradient
 * tensor") and a low-rank Tucker part (factor matrices U^(n), Section 2.2
 * "Low-rank gradient tensor decomposition"); Adam runs on the k sparse values
 * and on the Tucker core; the core is expanded back through the U^(n), the
 * sparse update is scatter-added, and W is updated in place.
 *
 * Conventions
 *  - All tensors are dense, row-major (last index fastest).  TGRAD_C64 stores
 *    each entry as two fp32 (re, im); TGRAD_C32H as two IEEE fp16 (re, im) and
 *    TGRAD_C32B as two bfloat16 (the paper's mixed-precision recipe, Section 2.3:
 *    weights and gradients in half precision, every optimizer state in fp32; the
 *    paper does not name the 16-bit format).
 *  - The caller passes grad = d(phi)/dW.  Algorithm 1 is written for
 *    G = -grad and W <- W + eta*Gtilde(G); the library evaluates the same
 *    stages on grad and subtracts, which is bit-identical.
 *  - Pointers named d_* are DEVICE pointers, everything else is host memory.
 *  - The library never allocates or frees device memory and, but for the
 *    side streams of tgrad_step_batched and the one a refresh uses (below),
 *    never creates streams.  The caller owns: the weight, the gradient, one persistent
 *    block (Omega, U^(n), moments, status words, a split copy of U^(N-1)
 *    laid out for the compression kernel) and one workspace block
 *    (scratch; contents need not survive between calls, but the same
 *    workspace must not be used by two states concurrently).  Sizes come
 *    from tgrad_state_bytes().  Both blocks must be 256-byte aligned.
 *  - All device work is enqueued asynchronously on the given stream
 *    (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *  - Argument errors are detected on the host before anything is enqueued and
 *    leave every buffer untouched.  Conditions found on the device (Jacobi
 *    sweep cap reached, non-finite gradient seen by the selection) set sticky
 *    bits that tgrad_query_status() reads.  Nothing aborts or traps.
 *  - A state is not thread-safe; distinct states may be used from distinct
 *    threads.
 */
#ifndef TGRAD_H_
#define TGRAD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tgrad_state tgrad_state;   /* opaque host handle; owns no device memory */

typedef enum {
  TGRAD_OK = 0,
  TGRAD_ERR_INVALID_ARG = 1,
  TGRAD_ERR_UNSUPPORTED = 2,
  TGRAD_ERR_BUFFER_TOO_SMALL = 3,
  TGRAD_ERR_CUDA = 4,
  TGRAD_ERR_NO_CONVERGE = 5,
  TGRAD_ERR_NONFINITE = 6,
  TGRAD_ERR_BAD_STATE = 7,
  TGRAD_ERR_TOO_LARGE = 8      /* tgrad_select_topk_noalloc: more entries than its built-in scratch covers */
} tgrad_status;

/* sticky device flags reported by tgrad_query_status() */
#define TGRAD_FLAG_NO_CONVERGE 1   /* the Jacobi eigensolver hit jacobi_max_sweeps */
#define TGRAD_FLAG_NONFINITE   2   /* a NaN/Inf magnitude was seen while selecting Omega */
#define TGRAD_FLAG_COPY_TIMEOUT 4  /* a streaming kernel gave up waiting for one of its own asynchronous copies
                                      (every device-side wait is bounded); the blocks that saw it returned early,
                                      so W and the moments of that step are undefined.  Not expected in normal
                                      operation; treat the state as lost */

typedef enum {
  TGRAD_C64 = 0,   /* interleaved 2 x fp32 */
  TGRAD_C32H = 1,  /* interleaved 2 x IEEE fp16 */
  TGRAD_C32B = 2   /* interleaved 2 x bfloat16 (general kernels only: no fp16 tensor-core fast path) */
} tgrad_dtype;

#define TGRAD_MAX_NDIM 8

/* Hyper-parameters of Algorithm 1 (its "Require" line) plus storage options. */
typedef struct {
  int32_t ndim;                     /* N, 2 <= ndim <= TGRAD_MAX_NDIM (N = 2: the matrix case,  */
                                    /* where the Tucker factors are the singular subspaces)     */
  int64_t dims[TGRAD_MAX_NDIM];     /* I_1..I_N, row-major; prod(dims) < 2^32                   */
  int32_t ranks[TGRAD_MAX_NDIM];    /* Tucker ranks, 1 <= r_n <= I_n                            */
  int64_t k;                        /* |Omega| = ceil(rho*I), computed exactly by the caller;   */
                                    /* k < 2^31                                                 */
  int32_t T;                        /* subspace change frequency, >= 1                          */
  float lr;                         /* eta                                                      */
  float alpha;                      /* scale of the reconstructed low-rank update               */
  float lambda;                     /* scale of the sparse update                               */
  float beta1, beta2, eps;          /* Adam decay rates and epsilon                             */
  float weight_decay;               /* decoupled decay W <- (1 - eta*wd) W before the update    */
  int32_t wg_dtype;                 /* tgrad_dtype of W and grad; all states are fp32           */
  int32_t auto_refresh;             /* 1: tgrad_step refreshes Omega and U^(n) when t % T == 0  */
  int32_t jacobi_max_sweeps;        /* sweep cap of the eigensolver (0 -> default 30)           */
  float jacobi_tol;                 /* off-diagonal tolerance relative to max diag (0 -> 1e-6)  */
  int32_t warm_refresh;             /* 1: a refresh starts its eigenvector iteration from the factor matrices
                                       the state holds (the paper's "warm restart" of the factors, appendix
                                       "Tensor Decomposition / Implementation") instead of a fixed pseudo-random
                                       start; if the subspace moved little this saves iterations, and the result
                                       is the same eigen-decomposition to the same tolerance.  Stored factors
                                       that are unusable (never set, not finite) are noticed on the device and
                                       that refresh starts cold.  0: every refresh starts cold               */
  int32_t hooi_iters;               /* refinement sweeps of TuckerFactors after the truncated-SVD factors (higher-
                                       order orthogonal iteration, the paper's appendix "Tensor Decomposition /
                                       Implementation"): per sweep and mode, the residual is compressed in every
                                       other mode with the current factors and U^(n) becomes the leading left
                                       singular vectors of the result.  0: none.  With warm_refresh = 1 and
                                       factors in the state, the sweeps start from those factors and the
                                       truncated-SVD stage is skipped (the warm restart of the decomposition).
                                       Needs extra workspace, and each trailing slab must still fit in shared
                                       memory with one of its two factors replaced by the identity            */
  int32_t composition;              /* order of the two parts (Section 2.2 "Residual and composition"):
                                       0: sparse part first, low-rank part on its residual (Algorithm 1);
                                       1: low-rank part first, the sparse part selected from and fed with
                                          G - P_U(G), P_U(G) the low-rank approximation of the gradient;
                                       2: both parts applied to the gradient itself and added                 */
  int32_t sparse_strategy;          /* how Omega is chosen at a refresh (Section 2.2 "Unstructured sparse gradient
                                       tensor"): 0 top-k magnitude; 1 uniform random k-subset; 2 sampling without
                                       replacement with probabilities proportional to |g|.  1 and 2 rank the
                                       entries by a key built from one Philox-4x32-10 word per entry (counter =
                                       flat index, refresh number t / T) and take the k largest                */
  uint64_t seed;                    /* key of that generator                                                   */
} tgrad_config;

/* Selectors for tgrad_export_state / tgrad_import_state.  FACTOR_BASE + n is
 * U^(n+1), an I_n x r_n row-major complex64 matrix. */
enum {
  TGRAD_WHAT_OMEGA = 1,        /* k x uint32, strictly ascending flat indices */
  TGRAD_WHAT_M_L = 2,          /* prod(r_n) x complex64, row-major core order */
  TGRAD_WHAT_V_L = 3,          /* prod(r_n) x fp32                            */
  TGRAD_WHAT_M_S = 4,          /* k x complex64, slot j <-> Omega[j]          */
  TGRAD_WHAT_V_S = 5,          /* k x fp32                                    */
  TGRAD_WHAT_CORE = 6,         /* last step's compressed gradient (export only; workspace) */
  TGRAD_WHAT_N_L = 7,          /* last step's normalised core update (export only)         */
  TGRAD_WHAT_N_S = 8,          /* last step's normalised sparse update (export only)       */
  TGRAD_WHAT_GRAM_BASE = 32,   /* + n: the Gram matrix the last refresh took U^(n+1) from, I_n x I_n complex64 (export
                                  only): A_n = R_(n) R_(n)^H, or with refinement sweeps that of the residual
                                  compressed in every other mode */
  TGRAD_WHAT_FACTOR_BASE = 64  /* + n */
};

/* Sizes of the two caller-owned device blocks for a configuration.
 * Counts follow the state inventory of Algorithm 1 (its initialisation
 * statements) and of the appendix "Parameter Complexity Analysis":
 * prod(r_n) core-shaped entries for each low-rank moment, sum I_n r_n factor
 * entries, k indices and k entries for each sparse moment.
 * The sizes do not depend on the device the state will run on.
 *
 * Limits of this implementation; a configuration outside them returns
 * TGRAD_ERR_UNSUPPORTED here and from tgrad_init_state:
 *   prod(dims) < 2^32 (flat indices are uint32) and k < 2^31;
 *   every I_n <= 1024 (size of the on-device eigensolver);
 *   r_N <= 32 (rank of the last mode);
 *   one trailing slab of I_{N-1} x I_N entries, with the operand tables of
 *   its two mode products, must fit in the 227 KB of shared memory of one SM
 *   (roughly I_{N-1} * (I_N + r_N) complex64 entries <= 28,000). */
tgrad_status tgrad_state_bytes(const tgrad_config* cfg, size_t* persistent_bytes, size_t* workspace_bytes);

/* Algorithm 1 initialisation: t <- 0, M_L, V_L, M_S, V_S <- 0 (enqueued on
 * the stream).  Omega and U^(n) are undefined until the first refresh.
 * Returns a host handle in *out that refers to, but does not own, the two
 * device blocks. */
tgrad_status tgrad_init_state(const tgrad_config* cfg, void* d_persistent, size_t persistent_bytes,
                              void* d_workspace, size_t workspace_bytes, void* cuda_stream, tgrad_state** out);

/* One pass of the loop body of Algorithm 1 for one tensor: (refresh if
 * auto_refresh and t mod T == 0), sparse gather, residual, Tucker compression
 * (chained mode-n products with U^(n)H, Section 2.2), AdamUpdate on the sparse
 * values and on the core, reconstruction scaled by alpha, scaled sparse add,
 * W <- W - eta*Gtilde, t <- t+1.
 * d_weight: in/out, prod(dims) entries of wg_dtype.  d_grad: input of the same
 * shape and dtype; it is restored to its input value before the call's work
 * completes, but is written temporarily during a refresh.
 * Returns TGRAD_ERR_BAD_STATE if no refresh has happened yet and auto_refresh
 * is 0. */
tgrad_status tgrad_step(tgrad_state* st, void* d_weight, void* d_grad, void* cuda_stream);

/* The `t mod T = 0` branch of Algorithm 1 on the supplied gradient:
 * Omega <- magnitude top-k of grad (key = fp32 re*re + im*im without fused
 * multiply-add, ties to the lower flat index, stored ascending);
 * R <- grad with Omega zeroed; U^(n) <- eigenvectors of the r_n largest
 * eigenvalues of R_(n) R_(n)^H (Jacobi), descending, each column scaled by the
 * unit phase that makes its largest-modulus component real positive.
 * Moments are not touched.  d_grad is modified while the call's work runs and
 * restored at its end.
 * Part of a refresh (the eigenvectors of the leading modes, while the Gram
 * matrices of the trailing modes are accumulated) runs on one side stream per
 * device, created at the first refresh on that device and kept for the life of
 * the process.  It is forked from and joined back into the caller's stream with
 * events: work enqueued on that stream before the call happens before all of
 * the refresh, work enqueued after it happens after all of it.  If the stream
 * cannot be created everything runs on the caller's stream.  The same holds
 * for a refresh that tgrad_step runs by itself. */
tgrad_status tgrad_refresh_subspace(tgrad_state* st, void* d_grad, void* cuda_stream);

/* Batched variants over a list of layers: semantically n independent calls
 * (the tensors of an FNO's spectral layers are independent).  Arrays are HOST
 * arrays of handles / device pointers.
 * tgrad_step_batched and tgrad_refresh_subspace_batched run the tensors' kernel chains side by side: they fork
 * them onto up to four streams that the library creates per device at the
 * first batched call (an exception to "creates no streams") and join
 * them back into the given stream, so for the caller the call orders like
 * any other work on that stream.  The states must have distinct workspaces,
 * and d_weights / d_grads must not overlap between tensors. */
tgrad_status tgrad_step_batched(tgrad_state* const* states, void* const* d_weights, void* const* d_grads,
                                int32_t n_tensors, void* cuda_stream);
tgrad_status tgrad_refresh_subspace_batched(tgrad_state* const* states, void* const* d_grads, int32_t n_tensors,
                                            void* cuda_stream);

/* Synchronises the stream, then reports the sticky flags (TGRAD_FLAG_*), the
 * step counter t and the number of Jacobi sweeps the last refresh used per
 * mode (sweeps may be NULL; otherwise ndim int32). */
tgrad_status tgrad_query_status(tgrad_state* st, void* cuda_stream, int32_t* sticky_flags, int64_t* t,
                                int32_t* sweeps);

/* Checkpoint / inspection: copy one state component to or from HOST memory.
 * `bytes` must equal the component's size exactly.  Both calls synchronise the
 * stream.  tgrad_set_step sets the counter t (host side). */
tgrad_status tgrad_export_state(tgrad_state* st, int32_t what, void* host_dst, size_t bytes, void* cuda_stream);
tgrad_status tgrad_import_state(tgrad_state* st, int32_t what, const void* host_src, size_t bytes,
                                void* cuda_stream);
tgrad_status tgrad_set_step(tgrad_state* st, int64_t t);

/* Optional diagnostics of the last step, not part of the timed path (synchronises the stream).  d_grad must be the
 * gradient that step was given.  out[0] = ||G||_F;  out[1] = ||G_S||_F / ||G||_F, the share of the gradient the
 * sparse part took;  out[2] = || X - P_U X ||_F / ||G||_F, the part the low-rank compression lost, X being what the
 * low-rank part was given (the residual of the sparse part in Algorithm 1's order, the gradient otherwise) -- with
 * orthonormal factors this is sqrt(||X||^2 - ||core||^2), the reconstruction error Section 2.2 reports for its
 * decompositions;  out[3] = max over modes and entries of |U^(n)H U^(n) - I|.
 * TGRAD_ERR_BAD_STATE before the first step. */
tgrad_status tgrad_diagnostics(tgrad_state* st, const void* d_grad, void* cuda_stream, double* out);

/* Frees the host handle only. */
tgrad_status tgrad_destroy_state(tgrad_state* st);

const char* tgrad_status_string(tgrad_status s);

/* Magnitude top-k selection for callers that cannot allocate device memory.
 * (The paper has no counterpart of this call; it computes the same Omega as
 * the refresh, "Unstructured sparse gradient tensor" with the top-k strategy.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a
 * framework's allocator callback or memory-pool hook (allocating there
 * re-enters the allocator), in a process whose device memory was handed out
 * in full at start-up, or in a latency-critical loop that must not take the
 * driver's allocation lock.  The other entry points need a workspace block
 * that somebody allocated; this one needs none.
 *
 * The scratch of the selection (radix histograms, threshold state, per-block
 * counts) lives in a fixed array inside the library's device image, about
 * 290 KB, which every GPU that loads the library holds until the process
 * exits.  That fixes the largest input: numel <= TGRAD_NOALLOC_MAX_NUMEL,
 * otherwise TGRAD_ERR_TOO_LARGE and nothing is enqueued.
 *
 * d_grad, d_omega and d_values must be 16-byte aligned, like the pointers of
 * the other entry points (TGRAD_ERR_INVALID_ARG otherwise, nothing enqueued).
 * d_grad:   device, numel entries of wg_dtype (tgrad_dtype), read only.
 * d_omega:  device, out, k x uint32: the flat indices of the k entries of
 *           largest |g|^2 (fp32 re*re + im*im without fused multiply-add),
 *           ties to the lower index, ascending.
 * d_values: device, out, k x complex64: grad at those indices (widened to
 *           fp32 if stored as fp16), i.e. Sparse(G, Omega) as index-value pairs.
 * Work is enqueued on the stream; nothing is allocated or freed, on the
 * device or by any library, and the stream is not synchronised.
 *
 * First call on a device: the library looks up the device address of its
 * scratch array once per device (the device that is current at the call) and
 * remembers it.  Make that first call outside any stream capture.
 * Sharing: all calls on a device use the same scratch, which keeps what the
 * last call left there; each call clears what it needs zeroed on its own
 * stream first.  Two calls whose work overlaps on the GPU (different streams,
 * or different threads and streams) race on it -- keep them on one stream or
 * order them with events.  Non-finite inputs give an unspecified result. */
#define TGRAD_NOALLOC_MAX_NUMEL (1ll << 26)
tgrad_status tgrad_select_topk_noalloc(const void* d_grad, int64_t numel, int64_t k, int32_t wg_dtype,
                                       uint32_t* d_omega, void* d_values, void* cuda_stream);

/* Kernels launched by this library since it was loaded (host-side counter). */
int64_t tgrad_launch_count(void);

/* Optional per-stage device timing of tgrad_step (CUDA events recorded on the
 * caller's stream between the stages of a non-refresh step).  Stages, in
 * order: 0 trailing-mode compression fused with the sparse gather (streams
 * grad), 1 mode products of the compression except the first mode, 2 first-mode
 * compression + Adam on the core and on the sparse values + first-mode
 * reconstruction, 3 remaining mode products of the reconstruction, 4
 * trailing-mode reconstruction fused with the weight update and sparse add
 * (streams W).
 * tgrad_get_stage_times synchronises the stream and returns, for the steps
 * since the last call (at most the 64 most recent), the summed milliseconds
 * per stage in ms_sum[5] and the number of steps in *n_steps. */
#define TGRAD_NUM_STAGES 5
tgrad_status tgrad_set_stage_timing(tgrad_state* st, int32_t enable);
tgrad_status tgrad_get_stage_times(tgrad_state* st, void* cuda_stream, float* ms_sum, int32_t* n_steps);

#ifdef __cplusplus
}
#endif
#endif /* TGRAD_H_ */
