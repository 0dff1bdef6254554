/*
 * zeno.h -- C ABI of the Zeno aggregation step on one NVIDIA B200 (sm_100a).
 *
 * The step is the server side of "Zeno: Distributed Stochastic Gradient
 * Descent with Suspicion-based Fault-tolerance" (Algorithm 1, the line
 * "v = Zeno_b({v_i})"):
 *
 *   Definition 2   Score_{gamma,rho}(v_i, x) = f_r(x) - f_r(x - gamma v_i) - rho ||v_i||^2,
 *                  f_r = mean loss over the server's n_r samples, l2 norm;
 *   Definition 3   rank the m candidates by score (descending) and return the
 *                  average of the m - b best.
 *
 * Conventions for every call
 *   - All data pointers are DEVICE pointers owned by the caller (x, V, the batch,
 *     and every output).  Inputs are never written (the one exception is x in
 *     zeno_step_update, which is that call's output too); outputs are overwritten
 *     in full.  The library allocates device memory only inside zeno_create.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls are asynchronous on it: they enqueue kernels and return; there is
 *     no host synchronisation and no device-to-host copy inside a call.
 *   - Errors are return codes.  Nothing is thrown, aborted or trapped.  Argument
 *     errors are detected on the host before anything is enqueued.
 *   - A handle serialises its calls through one private workspace: calls that
 *     use the same handle must be ordered on the GPU (same stream, or events).
 *
 * Parameter-vector layout (x and every row of V):
 *   multi-layer perceptron: for layer l = 1..L, the weights W_l as
 *   [dims[l] x dims[l-1]] row-major (input index contiguous), then, if
 *   has_bias, the bias b_l[dims[l]]; layers concatenated in order.
 *   least squares: the d entries of x.
 *   V is [m x ldv] row-major with ldv >= d (in elements); columns >= d are
 *   padding and are never read.  Rows whose start is 16-byte aligned
 *   (ldv * element size a multiple of 16, base pointer 16-byte aligned) take
 *   the vectorised kernels; any other ldv >= d takes a slower scalar path.
 */
#ifndef ZENO_H_
#define ZENO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ZENO_MAX_LAYERS 8
#define ZENO_MAX_CANDIDATES 1024
#define ZENO_KRUM_MAX_M 128      /* most candidates zeno_krum accepts */
#define ZENO_STATIC_MAX_M 64    /* most candidates zeno_score_lsq_static accepts */
#define ZENO_STATIC_MAX_N_R 32  /* most server samples zeno_score_lsq_static accepts */

typedef enum {
    ZENO_OK = 0,
    ZENO_ERR_INVALID_ARG = 1, /* NULL required pointer, m/b/n_r/ldv out of range, non-finite gamma or rho */
    ZENO_ERR_UNSUPPORTED = 2, /* a (loss, dtype, shape) for which no kernel exists -- never a silent fallback */
    ZENO_ERR_WORKSPACE = 3,   /* the handle's workspace could not be allocated */
    ZENO_ERR_CUDA = 4,        /* a CUDA runtime call failed; see zeno_last_cuda_error */
    ZENO_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up */
} zeno_status;

typedef enum {
    /* f(x; (a, y)) = -log softmax(MLP_x(a))[y]: L >= 1 dense layers, ReLU between
     * them; L = 1 is softmax regression.  Cross-entropy is the loss the paper
     * trains and reports (Experiments, evaluation metrics). */
    ZENO_LOSS_SOFTMAX_MLP = 0,
    /* f(x; (a, y)) = (a.x - y)^2 / 2, so that f_r(x) = ||A x - y||^2 / (2 n_r). */
    ZENO_LOSS_LEAST_SQUARES = 1,
    /* f(x; (a, y)) = -log softmax(CNN_x(a))[y] for a small convolutional network.  The paper's experiments
     * train "a CNN with 4 convolutional layers followed by 1 fully connected layer" (Experiments, datasets and
     * evaluation metrics) and do not print its shape; the network here is this library's own:
     *   Lc convolutional layers (Lc even): 3 x 3 windows, stride 1, zero padding 1, as a cross-correlation
     *     out[co][y][x] = b[co] + sum_ci sum_dy sum_dx W[co][ci][dy][dx] in[ci][y + dy - 1][x + dx - 1],
     *   each followed by ReLU, every second one also by a 2 x 2 max pooling with stride 2 (a NaN in the window
     *   gives NaN); then one dense layer from the last planes, flattened [C][y][x], to the classes' logits.
     * Parameter vector: per convolutional layer W[C_l][C_{l-1}][3][3] then b[C_l]; then the dense layer's
     * W[classes][C_Lc * side * side] and b[classes] (side = S / 2^(Lc/2)). */
    ZENO_LOSS_SOFTMAX_CNN = 2
} zeno_loss_kind;

typedef enum {
    ZENO_F32 = 0, /* x and V stored as IEEE binary32 */
    ZENO_BF16 = 1 /* x and V stored as bfloat16; a candidate's parameters are
                     x - gamma v rounded (to binary32, then) to bfloat16;
                     features, activations and accumulation stay binary32 */
} zeno_dtype;

typedef struct {
    int32_t kind;        /* zeno_loss_kind */
    int32_t param_dtype; /* zeno_dtype */
    int32_t n_layers;    /* L; least squares: 1; convolutional network: Lc + 1 (its dense layer counts) */
    int32_t has_bias;    /* MLP and convolutional network */
    int64_t dims[ZENO_MAX_LAYERS + 1]; /* MLP: widths, e.g. {3072,512,512,10}; least squares: {d, 1};
                                          convolutional network: {S, C_0, C_1, .., C_Lc, classes}, e.g.
                                          {32,3,32,32,64,64,10}: S x S images of C_0 planes (S even, at most 32,
                                          and still even before each pooling), n_layers + 2 entries */
} zeno_model_desc;

/* The server's batch z_1..z_{n_r} (Definition 2), drawn by the caller after the
 * candidates arrive (Algorithm 1). */
typedef struct {
    const float *features; /* device, [n_r x dims[0]] row-major binary32 (least squares: A [n_r x d];
                              convolutional network: [n_r][C_0][S][S]) */
    const void *targets;   /* device, int32 labels[n_r] in [0, dims[L]) (MLP) or float y[n_r] (least squares) */
    int32_t n_r;
} zeno_batch;

typedef struct zeno_context *zeno_handle;

/* Number of parameters d implied by a model description (0 if it is invalid). */
int64_t zeno_param_count(const zeno_model_desc *desc);

/* Creates a handle for one model shape on CUDA device `device` and allocates its
 * workspace for up to m_max candidates and n_r_max server samples.
 * INVALID_ARG: NULL arguments, m_max outside [1, ZENO_MAX_CANDIDATES], n_r_max < 1,
 * bad layer sizes.  UNSUPPORTED: unknown kind/dtype, least squares with bfloat16.
 * WORKSPACE / CUDA: allocation failed (the handle is not created). */
zeno_status zeno_create(zeno_handle *out, const zeno_model_desc *desc, int32_t m_max,
                        int32_t n_r_max, int32_t device);

/* Frees the workspace.  The caller makes sure no call on the handle is in flight. */
zeno_status zeno_destroy(zeno_handle h);

/* Definition 2 for all m candidates:
 *   losses[0] = f_r(x), losses[1+i] = f_r(x - gamma v_i), norms[i] = ||v_i||^2,
 *   scores[i] = losses[0] - losses[1+i] - rho * norms[i].
 * f_r(x) is evaluated once and shared ((m+1) n_r sample evaluations in all,
 * the paper's cost model).  The m perturbed models are never materialised:
 * x - gamma v_i is formed inside the operand load, and ||v_i||^2 is accumulated
 * in the same pass over V.
 * x: [d]; V: [m x ldv]; scores: float[m] (required); losses: float[m+1] or NULL;
 * norms: float[m] or NULL.
 * INVALID_ARG: NULL x/V/batch/features/targets/scores, m < 1 or > m_max,
 * n_r < 1 or > n_r_max, ldv < d, rho < 0 (the theory uses rho = 0 for convex
 * losses, so 0 is accepted), gamma or rho not finite.
 * Labels outside [0, classes) are not detected; the loss of that sample is then
 * computed against class 0. */
zeno_status zeno_score(zeno_handle h, const void *x, const void *V, int64_t ldv, int32_t m,
                       const zeno_batch *batch, float gamma, float rho, float *scores,
                       float *losses, float *norms, void *stream);

/* Definition 3, the ranking: idx[0..m-b) = the candidates with the m - b highest
 * scores in rank order.  The paper's ">=" leaves ties open; here a higher score
 * comes first, equal scores keep index order, and a NaN score ranks as minus
 * infinity.  Runs in one thread block (bitonic network on (score, index) keys).
 * INVALID_ARG: NULL pointers, m < 1 or > m_max, b < 0 or b >= m (the paper needs
 * m > b >= q; q is unknown to the server, so only m > b >= 0 is checked). */
zeno_status zeno_select(zeno_handle h, const float *scores, int32_t m, int32_t b, int32_t *idx,
                        void *stream);

/* Definition 3, the average: out[j] = (1/k) sum_{r<k} V[idx[r]][j] for j < d,
 * in binary32 whatever the storage type of V.  Only the k selected rows are
 * read.  idx is a device array; entries outside [0, m) are skipped (their row
 * contributes zero) rather than dereferenced.
 * INVALID_ARG: NULL pointers, k < 1 or k > m, m > m_max, ldv < d. */
zeno_status zeno_aggregate(zeno_handle h, const void *V, int64_t ldv, int32_t m,
                           const int32_t *idx, int32_t k, float *out, void *stream);

/* The score pass for a parameter vector that is sharded over several GPUs by column slice (the paper's
 * model is m-way data parallel; Definition 2's score is what has to be put together across the slices).
 * For the least-squares loss the residual A (x - gamma v) - y is linear in the parameters, so each GPU can
 * take the products of its own columns and one sum over the GPUs gives the whole:
 *
 *   zeno_score_partial   on a handle made for the slice (dims[0] = the slice's length): x, V, features are
 *                        the slice's columns (x [d_s], V [m x ldv], features A[:, slice] as [n_r x d_s]);
 *                        writes sums[(m+1) x (n_r+1)] doubles on the device: row 0 = A_s x_s, row 1 + c =
 *                        A_s v_c, last column of row 1 + c = the slice's share of ||v_c||^2 (0 in row 0).
 *   (the caller adds the sums of all slices: an all-reduce of (m+1)(n_r+1) doubles)
 *   zeno_score_from_sums from the total: losses[0] = ||A x - y||^2 / (2 n_r), losses[1 + c] the same at
 *                        x - gamma v_c, norms, scores = Definition 2.  targets = y[n_r] (device).
 *
 * Every GPU then ranks the same scores (zeno_select) and averages its own slice (zeno_aggregate): no further
 * exchange.  UNSUPPORTED: a handle that is not least squares.  Otherwise as zeno_score. */
zeno_status zeno_score_partial(zeno_handle h, const void *x, const void *V, int64_t ldv, int32_t m,
                               const float *features, int32_t n_r, double *sums, void *stream);
zeno_status zeno_score_from_sums(zeno_handle h, const double *sums, const float *targets, int32_t m, int32_t n_r,
                                 float gamma, float rho, float *scores, float *losses, float *norms, void *stream);

/* The workers' side of Algorithm 1 and the experiments' failures, on the device, so that a whole synchronous
 * iteration (workers' gradients -> failures -> Zeno_b -> update) can be chained on one stream.  These calls
 * build the step's input V; they are no part of the scoring path.
 *
 * zeno_worker_gradients -- Algorithm 1, worker i: v_i = grad F_i(x), the gradient of the mean loss over the
 * worker's own n samples, written to row i of V (in V's storage type).  features: [m][n x dims[0]] binary32,
 * targets: [m][n] int32 labels or binary32 y, one batch per worker; label_flip: int32[m] on the device or
 * NULL -- where non-zero, that worker's labels are replaced by (classes - 1 - label) first (Experiments,
 * label-flipping failure: "9 - label" for ten classes).  UNSUPPORTED: losses whose gradient needs
 * back-propagation through hidden layers (only one-layer softmax models with at most 32 classes, and least
 * squares in binary32, are served), or n beyond what a block's shared memory holds.
 *
 * zeno_inject_faults -- rows faulty[0..n_faulty) (device int32, entries outside [0, m) are skipped) of V
 * are overwritten in place:
 *   ZENO_FAULT_BIT_FLIP  Experiments, bit-flipping failure: the negative of row faulty[0]'s gradient, copied
 *                        over every faulty row (all faulty gradients have the same value);
 *   ZENO_FAULT_SCALE     the failure model's example: eps times the row's own gradient (eps a large
 *                        negative constant). */
#define ZENO_FAULT_BIT_FLIP 0
#define ZENO_FAULT_SCALE 1
zeno_status zeno_worker_gradients(zeno_handle h, const void *x, const float *features, const void *targets, int32_t n,
                                  int32_t m, const int32_t *label_flip, void *V, int64_t ldv, void *stream);
zeno_status zeno_inject_faults(zeno_handle h, void *V, int64_t ldv, int32_t m, const int32_t *faulty, int32_t n_faulty,
                               int32_t mode, float eps, void *stream);

/* The paper's baseline aggregation rules on the same candidates (Experiments, "Baselines"), for comparing
 * them with Zeno_b on the same step.
 *
 * zeno_median -- Definition "Median", the marginal median: out[j] = the one-dimensional median of
 * V[0][j] .. V[m-1][j] (the middle one of the sorted values, the mean of the two middle ones for even m),
 * in binary32.  The paper does not say what a NaN entry is worth; here it counts as plus infinity.
 * V: [m x ldv] device; out: float[d] device.  INVALID_ARG: NULL pointers, m < 1 or > m_max, ldv < d. */
zeno_status zeno_median(zeno_handle h, const void *V, int64_t ldv, int32_t m, float *out, void *stream);

/* zeno_krum -- Definition "Krum": k = arg min_i sum_{i -> j} ||v_i - v_j||^2 over the m - b - 2 nearest
 * neighbours j of v_i among the other candidates (squared Euclidean distances, taken as sums of squared
 * differences); ties go to the lowest index; a NaN distance counts as plus infinity.
 * k: device int32[1], the winning candidate (required); out: float[d] device, a copy of row k, or NULL;
 * sums: float[m] device, the candidates' neighbour sums, or NULL.
 * INVALID_ARG: NULL V / k, m < 1 or > m_max, ldv < d, b < 0, m - b - 2 < 1 (no neighbour left).  The paper
 * notes that Krum's guarantee needs 2b + 2 < m; its own toy example does not meet that, so it is not
 * enforced.  UNSUPPORTED: m > ZENO_KRUM_MAX_M. */
zeno_status zeno_krum(zeno_handle h, const void *V, int64_t ldv, int32_t m, int32_t b, float *out, int32_t *k,
                      float *sums, void *stream);

/* Zeno_b({v_i}) = score -> select -> aggregate on one stream, no host round trip.
 * out: float[d] (required); scores: float[m] or NULL; idx: int32[m-b] or NULL.
 * The SGD update x <- x - gamma * out (Algorithm 1) is left to the caller; zeno_step_update
 * applies it in the same call. */
zeno_status zeno_step(zeno_handle h, const void *x, const void *V, int64_t ldv, int32_t m,
                      const zeno_batch *batch, float gamma, float rho, int32_t b, float *out,
                      float *scores, int32_t *idx, void *stream);

/* Algorithm 1's server lines v = Zeno_b({v_i}) and x <- x - gamma v in one call: zeno_step, and
 * in the pass that forms the average the parameter vector takes the update,
 *     x[j] <- RN(x[j] - gamma out[j])    (one fused multiply-add in binary32, rounded to the
 *                                          storage type of x: binary32, or bfloat16 to nearest even),
 * so the update costs no further pass over x.  gamma is the same learning rate that the score
 * uses (Definition 2).  x is read by the scoring pass and overwritten in place afterwards; out
 * (the average itself, [d] binary32) may be NULL when only the new x is wanted; scores and idx as
 * in zeno_step.  Same argument checks and errors as zeno_step. */
zeno_status zeno_step_update(zeno_handle h, void *x, const void *V, int64_t ldv, int32_t m,
                             const zeno_batch *batch, float gamma, float rho, int32_t b, float *out,
                             float *scores, int32_t *idx, void *stream);

/* Algorithm 1's server loop for `steps` iterations on one stream with no host synchronisation in between:
 * iteration t scores the candidates V_t against the batch z_t at the current x, ranks them, and applies
 * x <- x - gamma Zeno_b(V_t) in the pass that forms the average (zeno_step_update without the out vector).
 * The candidates and batches of all iterations are laid out one after the other:
 *   V:        iteration t's [m x ldv] matrix starts step_stride_v elements after iteration t - 1's
 *             (step_stride_v >= m * ldv);
 *   features: [steps][n_r x dims[0]] binary32, contiguous;   targets: [steps][n_r] (int32 or float);
 *   scores:   [steps][m] or NULL;   idx: [steps][m - b] or NULL.
 * x is read and updated in place by every iteration.  The candidates are inputs: they are what the workers
 * sent for these iterations, however the caller obtained them.  The profiler (zeno_profile) sees the whole
 * run as one call and keeps only the kernels that fit its per-call list.
 * INVALID_ARG: as zeno_step_update, or steps < 1, or step_stride_v < m * ldv. */
zeno_status zeno_run(zeno_handle h, void *x, const void *V, int64_t ldv, int64_t step_stride_v, int32_t m,
                     const float *features, const void *targets, int32_t n_r, int32_t steps, float gamma,
                     float rho, int32_t b, float *scores, int32_t *idx, void *stream);

/* The same step for a caller whose data lives in HOST memory (Algorithm 1's server receiving the
 * candidates over the network): x, V, features, targets, out, scores and idx are HOST pointers
 * (pinned memory makes the copies asynchronous).  The call copies the inputs to a device staging
 * area owned by the handle (allocated or grown on first need -- the only allocation outside
 * zeno_create), enqueues the step, copies out[d] (and scores[m], idx[m-b] if not NULL) back and
 * synchronises the stream before returning.  Same argument checks as zeno_step. */
zeno_status zeno_step_host(zeno_handle h, const void *x, const void *V, int64_t ldv, int32_t m,
                           const float *features, const void *targets, int32_t n_r, float gamma,
                           float rho, int32_t b, float *out, float *scores, int32_t *idx,
                           void *stream);

/* Least-squares scores for callers that must not allocate.  (The paper has no counterpart: this
 * is a packaging variant of zeno_score for the least-squares loss.  It always runs the CUDA-core
 * streaming kernel, whereas a handle takes the tensor-core stream for aligned shapes of up to 64
 * candidates: the two agree to the tolerances the tests use, not bit for bit.)
 * Some users of this library cannot call cudaMalloc at the point where they need a score: a
 * serving loop that promised its host framework not to touch the allocator after start-up
 * (cudaMalloc synchronises the whole device and would stall every other stream), or a process
 * whose framework has already claimed all device memory for its own pool.  zeno_create needs an
 * allocation for its workspace, so this call takes no handle: its scratch (per-slab partial
 * products, about 1.4 MB) is a fixed array inside the library image, present on every GPU that
 * loads the library for the life of the process.
 *   - All pointers are device pointers on `device`; x [d], V [m x ldv], A [n_r x d], y [n_r];
 *     scores[m] required, losses[m+1] and norms[m] optional (NULL).  Same quantities as
 *     zeno_score on a least-squares handle (equal within 1e-4 relative on the scores, see above).
 *   - m <= ZENO_STATIC_MAX_M and n_r <= ZENO_STATIC_MAX_N_R, else ZENO_ERR_WORKSPACE (the scratch
 *     is fixed).  Other argument errors: ZENO_ERR_INVALID_ARG, as for zeno_score.
 *   - The first call on a device looks up the array's device address, which makes the CUDA
 *     runtime load the library's code and data (this array included) onto that device if it has
 *     not done so yet -- the one moment at which device memory is claimed on the caller's behalf.
 *     Make that first call at start-up: before the process hands the rest of the device's memory
 *     to its own pool, and before any stream capture begins.  Later calls only launch kernels.
 *     First calls from several host threads are serialised inside the library.
 *   - The call itself invokes no cudaMalloc / cudaFree / allocating routine, ever.
 *   - All calls on a device share the one array and nothing in it needs clearing between calls
 *     (each call rewrites every partial it later reads), but two calls whose kernels overlap on
 *     the GPU (different streams, no ordering) race on it: order them. */
zeno_status zeno_score_lsq_static(int32_t device, const float *x, const float *V, int64_t ldv, int64_t d,
                                  int32_t m, const float *A, const float *y, int32_t n_r, float gamma,
                                  float rho, float *scores, float *losses, float *norms, void *stream);

/* Synchronises `stream` and reports whether any kernel enqueued through this handle gave up on a
 * bounded device-side wait (its outputs are then undefined): ZENO_ERR_TIMEOUT if so, else
 * ZENO_OK.  The condition is sticky for the life of the handle. */
zeno_status zeno_device_status(zeno_handle h, void *stream);

/* Test hook for the give-up path of the bounded device-side waits.  Every wait a tensor-core kernel
 * makes on one of its barriers polls at most `polls` times (default 2^22, a few tenths of a second)
 * before it gives up, raises the status word that zeno_device_status reads and lets the block leave
 * through its teardown (copies in flight awaited, tensor memory freed) -- the context stays usable.
 * polls = 0 makes every wait that is not already satisfied give up, and makes every block begin by
 * waiting, as briefly, for an arrival that never comes -- which is how the tests reach that path for
 * certain without anything going wrong on the device; the waits of the teardown itself keep the
 * default.  The outputs of a call that gave up are undefined and the handle's workspace may be left
 * inconsistent: destroy the handle afterwards. */
zeno_status zeno_debug_set_wait_limit(zeno_handle h, uint32_t polls);

/* Per-kernel timing for benchmarks.  zeno_profile(h, 1) makes every later call on the handle
 * record a CUDA event on the call's stream before each of its kernels and after the last one
 * (a few microseconds of overhead per call) and keeps the events of the last 64 calls;
 * zeno_profile(h, 0) switches it off again.  zeno_profile_read looks at the call made `back`
 * calls ago (0 = the most recent), waits for its last event (a host synchronisation) and
 * writes, for up to `cap` kernels in launch order, the elapsed milliseconds ms[i] and a static
 * name names[i] (either array may be NULL).  Enqueue many calls before reading, so that the
 * GPU is never waiting for the host between the events.  Returns the number of kernels
 * written, 0 if profiling is off or that call is not in the ring, -1 on a CUDA error. */
zeno_status zeno_profile(zeno_handle h, int32_t enable);
int32_t zeno_profile_read(zeno_handle h, int32_t back, float *ms, const char **names, int32_t cap);

/* Kernels launched by the most recent call on this handle (0 after an error). */
int32_t zeno_last_launch_count(zeno_handle h);

/* The cudaError_t (as int) behind the most recent ZENO_ERR_CUDA on this handle. */
int32_t zeno_last_cuda_error(zeno_handle h);

/* Which device-side wait was behind the most recent ZENO_ERR_TIMEOUT on this handle (0 if none): the
 * kernel in bits 24-27 (1 first-layer stream, 2 layer, 3 least squares), the index of the barrier in
 * that kernel's barrier array in bits 1-16, the awaited phase parity in bit 0.  For bug reports. */
int32_t zeno_last_wait_code(zeno_handle h);

const char *zeno_status_string(zeno_status s);

#ifdef __cplusplus
}
#endif
#endif /* ZENO_H_ */
