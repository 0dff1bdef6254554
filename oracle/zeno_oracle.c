/*
 * zeno_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, float64 statement of the Zeno aggregation rule
 * (Xie, Koyejo, Gupta: "Zeno: Distributed SGD with Suspicion-based
 * Fault-tolerance"), written from the paper's definitions so that it can be
 * checked against them by eye:
 *
 *   Definition 2 (stochastic descendant score)
 *       Score_{gamma,rho}(u, x) = f_r(x) - f_r(x - gamma u) - rho ||u||^2,
 *       f_r(x) = (1/n_r) sum_{i<=n_r} f(x; z_i),  all norms l2 (Table 1).
 *   Definition 3 (suspicion-based aggregation)
 *       sort the candidates by score, descending; average the first m-b.
 *
 * Every candidate is evaluated on its own, from the definition: the
 * perturbed parameter vector x - gamma*v_i is formed, the loss is evaluated
 * on it, nothing is shared between candidates except f_r(x), nothing is
 * blocked, fused or reordered.  All arithmetic is double precision; inputs
 * (float32 or bfloat16 storage) are promoted exactly.
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg use
 * this file.  It shares no code, header, table or constant with the CUDA
 * library.
 *
 * Pins (tests/test_oracle_pins.py): every function below is pinned -- see the
 * list in that file.  Nothing here is "parity unpinned".
 *
 * Parameter-vector layout (the one both sides agree on): x and every row of
 * V are the flat concatenation, layer by layer, of W_l stored [out_l x in_l]
 * row-major followed by b_l[out_l] (if has_bias).  Least squares: just x[d].
 *
 * Convolutional network (kind 2; the paper's experiments train "a CNN with 4 convolutional layers
 * followed by 1 fully connected layer" whose exact shape it does not print, so this one is this
 * project's own and is stated here in full):
 *   dims = {S, C_0, C_1, .., C_Lc, classes}, n_layers = Lc + 1 (Lc convolutional layers, Lc even, and the
 *   dense layer); the input is C_0 planes of S x S values, [C_0][S][S] row-major.
 *   Convolutional layer l (1-based): 3 x 3 windows, stride 1, zero padding 1, as a cross-correlation
 *     out[co][y][x] = b[co] + sum_ci sum_dy sum_dx W[co][ci][dy][dx] in[ci][y + dy - 1][x + dx - 1],
 *   followed by ReLU; after every second convolutional layer a 2 x 2 max pooling with stride 2 (a NaN in
 *   the window gives NaN).  The dense layer takes the last planes flattened [C][y][x] to `classes`
 *   logits; the loss is the softmax cross-entropy, as for kind 0.
 *   Parameters: per convolutional layer W[C_l][C_{l-1}][3][3] then b[C_l]; then the dense layer's
 *   W[classes][C_Lc (S / 2^(Lc/2))^2] and b[classes].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ZO_LOSS_SOFTMAX_MLP = 0, ZO_LOSS_LEAST_SQUARES = 1, ZO_LOSS_SOFTMAX_CNN = 2 };
enum { ZO_F32 = 0, ZO_BF16 = 1 };
enum { ZO_OK = 0, ZO_BAD_ARG = 1, ZO_NO_MEM = 2 };

/* number of single-sample loss evaluations f(.; z_j) performed since the last
 * reset; the paper's cost model is (m+1) * n_r of them per step (Discussion:
 * "21 x 4 = 84" for m = 20, n_r = 4). */
static long long zo_sample_evals = 0;
void zo_reset_eval_count(void) { zo_sample_evals = 0; }
long long zo_eval_count(void) { return zo_sample_evals; }

int zo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- storage formats ---------------------------------------------------- */

static double zo_bf16_bits_to_double(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16; /* bfloat16 = the upper half of a binary32 */
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* one stored parameter, promoted exactly */
static double zo_load(const void *p, int64_t i, int dtype)
{
    if (dtype == ZO_BF16)
        return zo_bf16_bits_to_double(((const uint16_t *)p)[i]);
    return (double)((const float *)p)[i];
}

/* Round a binary32 value to the nearest bfloat16 (8 significant bits, binary32
 * exponent range), ties to even, written from the format's definition:
 * find the spacing of bfloat16 numbers around |f| and round f to a multiple
 * of it with the current (to-nearest-even) rounding mode. */
double zo_round_to_bf16(float f)
{
    double a = fabs((double)f);
    if (!(a == a) || isinf(a) || a == 0.0)
        return (double)f;
    int e;
    frexp(a, &e);            /* a = frac * 2^e, frac in [0.5, 1)  =>  2^(e-1) <= a < 2^e */
    int ulp_exp = (e - 1) - 7; /* 8 significant bits */
    if (ulp_exp < -126 - 7)
        ulp_exp = -126 - 7;  /* subnormal range: fixed spacing 2^-133 */
    double q = nearbyint(ldexp(a, -ulp_exp)); /* exact scaling, ties to even */
    double r = ldexp(q, ulp_exp);
    if (r >= ldexp(1.0, 128))
        r = INFINITY;        /* past the largest finite bfloat16 */
    return f < 0 ? -r : r;
}

/* ---- the candidate's parameter vector ----------------------------------- */

/* w = x - gamma * v, element by element (Definition 2's argument x - gamma u).
 * v == NULL gives w = x.
 * float32 storage: exact double arithmetic on the promoted values.
 * bfloat16 storage: the candidate is itself a bfloat16 model; its entries are
 * the difference rounded once to binary32 (the precision the quantisation
 * decision is taken in) and then to bfloat16. */
void zo_candidate_params(const void *x, const void *v, int64_t d, int dtype,
                         double gamma, double *w)
{
    for (int64_t j = 0; j < d; ++j) {
        double xj = zo_load(x, j, dtype);
        if (!v) { w[j] = xj; continue; }
        double vj = zo_load(v, j, dtype);
        double diff = xj - gamma * vj;
        if (dtype == ZO_BF16)
            diff = zo_round_to_bf16((float)diff);
        w[j] = diff;
    }
}

/* side of the planes after all pooling steps, or 0 if the description is not a valid network */
static int64_t zo_cnn_final_side(int n_layers, const int64_t *dims)
{
    int lc = n_layers - 1;
    if (lc < 2 || (lc & 1))
        return 0;
    int64_t side = dims[0];
    for (int l = 2; l <= lc; l += 2) {
        if (side < 2 || (side & 1))
            return 0;
        side /= 2;
    }
    return side;
}

int64_t zo_param_count(int kind, int n_layers, const int64_t *dims, int has_bias)
{
    if (kind == ZO_LOSS_LEAST_SQUARES)
        return dims[0];
    if (kind == ZO_LOSS_SOFTMAX_CNN) {
        int lc = n_layers - 1;
        int64_t side = zo_cnn_final_side(n_layers, dims);
        if (side == 0)
            return 0;
        int64_t d = 0;
        for (int l = 1; l <= lc; ++l)
            d += dims[l + 1] * dims[l] * 9 + (has_bias ? dims[l + 1] : 0);
        int64_t classes = dims[lc + 2];
        d += classes * dims[lc + 1] * side * side + (has_bias ? classes : 0);
        return d;
    }
    int64_t d = 0;
    for (int l = 0; l < n_layers; ++l)
        d += dims[l + 1] * dims[l] + (has_bias ? dims[l + 1] : 0);
    return d;
}

/* ---- f_r ---------------------------------------------------------------- */

/* Softmax cross-entropy of a ReLU multi-layer perceptron, one sample.
 * h: the sample's features [dims[0]].  scratch: two buffers of max(dims). */
static double zo_mlp_sample_loss(const double *w, int n_layers, const int64_t *dims,
                                 int has_bias, const float *feat, int32_t label,
                                 double *buf0, double *buf1)
{
    double *h = buf0, *z = buf1;
    for (int64_t k = 0; k < dims[0]; ++k)
        h[k] = (double)feat[k];
    const double *p = w;
    for (int l = 0; l < n_layers; ++l) {
        int64_t in = dims[l], out = dims[l + 1];
        const double *W = p;
        const double *bias = has_bias ? p + out * in : NULL;
        for (int64_t o = 0; o < out; ++o) {
            double acc = 0.0;
            for (int64_t k = 0; k < in; ++k)
                acc += W[o * in + k] * h[k];
            if (bias)
                acc += bias[o];
            if (l + 1 < n_layers && !(acc > 0.0))
                acc = (acc == acc) ? 0.0 : acc; /* ReLU; a NaN stays a NaN */
            z[o] = acc;
        }
        p += out * in + (has_bias ? out : 0);
        double *t = h; h = z; z = t;
    }
    /* h now holds the logits: loss = log sum_c exp(z_c) - z_label */
    int64_t C = dims[n_layers];
    double zmax = h[0];
    for (int64_t c = 1; c < C; ++c)
        if (h[c] > zmax) zmax = h[c];
    double se = 0.0;
    for (int64_t c = 0; c < C; ++c)
        se += exp(h[c] - zmax);
    return zmax + log(se) - h[label];
}

/* the larger of two values; a NaN wins */
static double zo_max_nan(double a, double b)
{
    if (a != a) return a;
    if (b != b) return b;
    return a > b ? a : b;
}

/* Softmax cross-entropy of the convolutional network described at the top of this file, one sample.
 * feat: [C_0][S][S].  buf0, buf1: two buffers of the largest number of values any layer holds.
 * logits_out (optional): the dense layer's outputs. */
static double zo_cnn_sample_loss(const double *w, int n_layers, const int64_t *dims, int has_bias,
                                 const float *feat, int32_t label, double *buf0, double *buf1,
                                 double *logits_out)
{
    int lc = n_layers - 1;
    int64_t side = dims[0];
    double *h = buf0, *z = buf1;
    for (int64_t k = 0; k < dims[1] * side * side; ++k)
        h[k] = (double)feat[k];
    const double *p = w;
    for (int l = 1; l <= lc; ++l) {
        int64_t cin = dims[l], cout = dims[l + 1];
        const double *W = p;
        const double *bias = has_bias ? p + cout * cin * 9 : NULL;
        for (int64_t co = 0; co < cout; ++co)
            for (int64_t y = 0; y < side; ++y)
                for (int64_t x = 0; x < side; ++x) {
                    double acc = bias ? bias[co] : 0.0;
                    for (int64_t ci = 0; ci < cin; ++ci)
                        for (int dy = 0; dy < 3; ++dy)
                            for (int dx = 0; dx < 3; ++dx) {
                                int64_t yy = y + dy - 1, xx = x + dx - 1;
                                if (yy < 0 || yy >= side || xx < 0 || xx >= side)
                                    continue; /* zero padding */
                                acc += W[((co * cin + ci) * 3 + dy) * 3 + dx] * h[(ci * side + yy) * side + xx];
                            }
                    if (!(acc > 0.0))
                        acc = (acc == acc) ? 0.0 : acc; /* ReLU; a NaN stays a NaN */
                    z[(co * side + y) * side + x] = acc;
                }
        p += cout * cin * 9 + (has_bias ? cout : 0);
        double *t = h; h = z; z = t;
        if ((l & 1) == 0) { /* 2 x 2 max pooling, stride 2 */
            int64_t half = side / 2;
            for (int64_t c = 0; c < cout; ++c)
                for (int64_t y = 0; y < half; ++y)
                    for (int64_t x = 0; x < half; ++x) {
                        const double *q = h + (c * side + 2 * y) * side + 2 * x;
                        z[(c * half + y) * half + x] =
                            zo_max_nan(zo_max_nan(q[0], q[1]), zo_max_nan(q[side], q[side + 1]));
                    }
            side = half;
            t = h; h = z; z = t;
        }
    }
    int64_t flat = dims[lc + 1] * side * side, C = dims[lc + 2];
    const double *W = p;
    const double *bias = has_bias ? p + C * flat : NULL;
    for (int64_t c = 0; c < C; ++c) {
        double acc = 0.0;
        for (int64_t k = 0; k < flat; ++k)
            acc += W[c * flat + k] * h[k];
        if (bias)
            acc += bias[c];
        z[c] = acc;
        if (logits_out)
            logits_out[c] = acc;
    }
    double zmax = z[0];
    for (int64_t c = 1; c < C; ++c)
        if (z[c] > zmax) zmax = z[c];
    double se = 0.0;
    for (int64_t c = 0; c < C; ++c)
        se += exp(z[c] - zmax);
    return zmax + log(se) - z[label];
}

/* largest number of values a layer of the network holds (the input, any layer's planes, the logits) */
static int64_t zo_cnn_widest(int n_layers, const int64_t *dims)
{
    int lc = n_layers - 1;
    int64_t side = dims[0], widest = dims[1] * side * side;
    for (int l = 1; l <= lc; ++l) {
        if (dims[l + 1] * side * side > widest) widest = dims[l + 1] * side * side;
        if ((l & 1) == 0) side /= 2;
    }
    if (dims[lc + 2] > widest) widest = dims[lc + 2];
    return widest;
}

/* The network's logits for one sample (for the pins: the layers' arithmetic seen without the loss). */
int zo_cnn_logits(int n_layers, const int64_t *dims, int has_bias, const double *w, const float *feat,
                  double *logits)
{
    if (zo_cnn_final_side(n_layers, dims) == 0)
        return ZO_BAD_ARG;
    int64_t widest = zo_cnn_widest(n_layers, dims);
    double *buf0 = (double *)malloc(sizeof(double) * (size_t)widest);
    double *buf1 = (double *)malloc(sizeof(double) * (size_t)widest);
    if (!buf0 || !buf1) { free(buf0); free(buf1); return ZO_NO_MEM; }
    (void)zo_cnn_sample_loss(w, n_layers, dims, has_bias, feat, 0, buf0, buf1, logits);
    free(buf0);
    free(buf1);
    return ZO_OK;
}

/* f_r(w) = (1/n_r) sum_j f(w; z_j)   (Definition 2).
 * kind 0: targets = int32 labels[n_r]; features [n_r x dims[0]] float32.
 * kind 2: targets = int32 labels[n_r]; features [n_r x C_0 x S x S] float32 (see the top of the file).
 * kind 1: f(w; (a_j, y_j)) = (a_j . w - y_j)^2 / 2, features = A [n_r x d],
 *         targets = float32 y[n_r], so that f_r = ||A w - y||^2 / (2 n_r). */
double zo_loss(int kind, int n_layers, const int64_t *dims, int has_bias,
               const double *w, const float *features, const void *targets, int n_r)
{
    double total = 0.0;
    if (kind == ZO_LOSS_LEAST_SQUARES) {
        int64_t d = dims[0];
        const float *y = (const float *)targets;
        for (int j = 0; j < n_r; ++j) {
            double acc = 0.0;
            for (int64_t k = 0; k < d; ++k)
                acc += (double)features[(int64_t)j * d + k] * w[k];
            double r = acc - (double)y[j];
            total += 0.5 * r * r;
        }
    } else if (kind == ZO_LOSS_SOFTMAX_CNN) {
        if (zo_cnn_final_side(n_layers, dims) == 0)
            return NAN;
        int64_t widest = zo_cnn_widest(n_layers, dims);
        int64_t in_elems = dims[1] * dims[0] * dims[0];
        double *buf0 = (double *)malloc(sizeof(double) * (size_t)widest);
        double *buf1 = (double *)malloc(sizeof(double) * (size_t)widest);
        if (!buf0 || !buf1) { free(buf0); free(buf1); return NAN; }
        const int32_t *labels = (const int32_t *)targets;
        for (int j = 0; j < n_r; ++j)
            total += zo_cnn_sample_loss(w, n_layers, dims, has_bias, features + (int64_t)j * in_elems,
                                        labels[j], buf0, buf1, NULL);
        free(buf0);
        free(buf1);
    } else {
        int64_t widest = 0;
        for (int l = 0; l <= n_layers; ++l)
            if (dims[l] > widest) widest = dims[l];
        double *buf0 = (double *)malloc(sizeof(double) * (size_t)widest);
        double *buf1 = (double *)malloc(sizeof(double) * (size_t)widest);
        if (!buf0 || !buf1) { free(buf0); free(buf1); return NAN; }
        const int32_t *labels = (const int32_t *)targets;
        for (int j = 0; j < n_r; ++j)
            total += zo_mlp_sample_loss(w, n_layers, dims, has_bias,
                                        features + (int64_t)j * dims[0], labels[j], buf0, buf1);
        free(buf0);
        free(buf1);
    }
#pragma omp atomic
    zo_sample_evals += n_r;
    return total / (double)n_r;
}

/* ---- Definition 2: scores ------------------------------------------------ */

/* scores[i] = f_r(x) - f_r(x - gamma v_i) - rho ||v_i||^2 for i < m.
 * losses (optional, [m+1]): losses[0] = f_r(x), losses[1+i] = f_r(x - gamma v_i).
 * norms  (optional, [m])  : ||v_i||^2.
 * V is [m x ldv] row-major in the storage dtype; columns >= d are padding.
 * Candidates are independent; they are spread over the host threads. */
int zo_score(int kind, int dtype, int n_layers, const int64_t *dims, int has_bias,
             const void *x, const void *V, int64_t ldv, int m,
             const float *features, const void *targets, int n_r,
             double gamma, double rho,
             double *scores, double *losses, double *norms)
{
    if (m < 1 || n_r < 1 || !x || !V || !features || !targets || !scores)
        return ZO_BAD_ARG;
    int64_t d = zo_param_count(kind, n_layers, dims, has_bias);
    if (ldv < d)
        return ZO_BAD_ARG;
    size_t esz = dtype == ZO_BF16 ? 2 : 4;
    int rc = ZO_OK;

    double *w0 = (double *)malloc(sizeof(double) * (size_t)d);
    if (!w0) return ZO_NO_MEM;
    zo_candidate_params(x, NULL, d, dtype, 0.0, w0);
    double f0 = zo_loss(kind, n_layers, dims, has_bias, w0, features, targets, n_r);
    free(w0);
    if (losses) losses[0] = f0;

#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < m; ++i) {
        const void *vi = (const char *)V + (size_t)i * (size_t)ldv * esz;
        double *w = (double *)malloc(sizeof(double) * (size_t)d);
        if (!w) {
#pragma omp atomic write
            rc = ZO_NO_MEM;
            continue;
        }
        zo_candidate_params(x, vi, d, dtype, gamma, w);
        double fi = zo_loss(kind, n_layers, dims, has_bias, w, features, targets, n_r);
        free(w);
        double nrm = 0.0;
        for (int64_t j = 0; j < d; ++j) {
            double vj = zo_load(vi, j, dtype);
            nrm += vj * vj;
        }
        scores[i] = f0 - fi - rho * nrm;
        if (losses) losses[1 + i] = fi;
        if (norms) norms[i] = nrm;
    }
    return rc;
}

/* ---- Definition 3: ranking ----------------------------------------------- */

/* idx[0..m-b) = the candidates with the m-b highest scores, in rank order.
 * The paper's ">=" leaves ties open; the reading taken here: higher score
 * first, then lower index; a NaN score counts as minus infinity.
 * Plain stable insertion sort of the index list. */
int zo_select(const double *scores, int m, int b, int32_t *idx)
{
    if (m < 1 || b < 0 || b >= m || !scores || !idx)
        return ZO_BAD_ARG;
    int32_t *order = (int32_t *)malloc(sizeof(int32_t) * (size_t)m);
    double *key = (double *)malloc(sizeof(double) * (size_t)m);
    if (!order || !key) { free(order); free(key); return ZO_NO_MEM; }
    for (int i = 0; i < m; ++i)
        key[i] = (scores[i] == scores[i]) ? scores[i] : -INFINITY;
    for (int i = 0; i < m; ++i) {
        int pos = i;
        /* move left past strictly smaller keys only: equal keys keep index order */
        while (pos > 0 && key[order[pos - 1]] < key[i]) {
            order[pos] = order[pos - 1];
            --pos;
        }
        order[pos] = i;
    }
    for (int r = 0; r < m - b; ++r)
        idx[r] = order[r];
    free(order);
    free(key);
    return ZO_OK;
}

/* ---- Definition 3: trimmed average --------------------------------------- */

/* out[j] = (1/k) sum_{r<k} V[idx[r]][j],  j < d. */
int zo_aggregate(int dtype, const void *V, int64_t ldv, int64_t d, int m,
                 const int32_t *idx, int k, double *out)
{
    if (k < 1 || !V || !idx || !out || ldv < d)
        return ZO_BAD_ARG;
    size_t esz = dtype == ZO_BF16 ? 2 : 4;
    for (int r = 0; r < k; ++r)
        if (idx[r] < 0 || idx[r] >= m) return ZO_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < d; ++j) {
        double acc = 0.0;
        for (int r = 0; r < k; ++r) {
            const void *row = (const char *)V + (size_t)idx[r] * (size_t)ldv * esz;
            acc += zo_load(row, j, dtype);
        }
        out[j] = acc / (double)k;
    }
    return ZO_OK;
}

/* ---- Algorithm 1, the server's update line -------------------------------- */

/* xnew[j] = x[j] - gamma * vbar[j] with vbar the aggregated vector (the line after
 * v = Zeno_b({v_i}) in Algorithm 1).  float32 storage: the exact double value.
 * bfloat16 storage: the new parameter is a bfloat16 number, the difference rounded
 * once to binary32 and then to bfloat16, the same rule as for a candidate's parameters. */
void zo_update(const void *x, const double *vbar, int64_t d, int dtype, double gamma,
               double *xnew)
{
    for (int64_t j = 0; j < d; ++j) {
        double diff = zo_load(x, j, dtype) - gamma * vbar[j];
        if (dtype == ZO_BF16)
            diff = zo_round_to_bf16((float)diff);
        xnew[j] = diff;
    }
}

/* ---- the whole step: Zeno_b({v_i}) ---------------------------------------- */

int zo_step(int kind, int dtype, int n_layers, const int64_t *dims, int has_bias,
            const void *x, const void *V, int64_t ldv, int m,
            const float *features, const void *targets, int n_r,
            double gamma, double rho, int b,
            double *out, double *scores, int32_t *idx)
{
    if (b < 0 || b >= m) return ZO_BAD_ARG;
    int64_t d = zo_param_count(kind, n_layers, dims, has_bias);
    double *s = scores ? scores : (double *)malloc(sizeof(double) * (size_t)m);
    int32_t *ix = idx ? idx : (int32_t *)malloc(sizeof(int32_t) * (size_t)(m - b));
    if (!s || !ix) return ZO_NO_MEM;
    int rc = zo_score(kind, dtype, n_layers, dims, has_bias, x, V, ldv, m,
                      features, targets, n_r, gamma, rho, s, NULL, NULL);
    if (rc == ZO_OK) rc = zo_select(s, m, b, ix);
    if (rc == ZO_OK) rc = zo_aggregate(dtype, V, ldv, d, m, ix, m - b, out);
    if (!scores) free(s);
    if (!idx) free(ix);
    return rc;
}

/* ---- the baseline aggregation rules on the same candidates ----------------
 *
 * Experiments, "Baselines": the marginal median (Definition "Median") and Krum
 * (Definition "Krum"), written out as their definitions. */

static int zo_cmp_double(const void *a, const void *b)
{
    double x = *(const double *)a, y = *(const double *)b;
    return (x > y) - (x < y);
}

/* Marginal median: out[j] = the one-dimensional median of the j-th entries of the m
 * candidates -- the middle one of the sorted values for odd m, the mean of the two
 * middle ones for even m.  Reading where the paper is silent: a NaN entry (a faulty
 * worker may send anything) counts as plus infinity. */
int zo_median(int dtype, const void *V, int64_t ldv, int64_t d, int m, double *out)
{
    if (m < 1 || d < 1 || ldv < d) return ZO_BAD_ARG;
    const size_t esz = dtype == ZO_BF16 ? 2 : 4;
    int rc = ZO_OK;
#pragma omp parallel
    {
        double *col = (double *)malloc(sizeof(double) * (size_t)m);
        if (!col) {
#pragma omp critical
            rc = ZO_NO_MEM;
        } else {
#pragma omp for schedule(static)
            for (int64_t j = 0; j < d; ++j) {
                for (int i = 0; i < m; ++i) {
                    double v = zo_load((const char *)V + (size_t)i * (size_t)ldv * esz, j, dtype);
                    col[i] = v != v ? INFINITY : v;
                }
                qsort(col, (size_t)m, sizeof(double), zo_cmp_double);
                out[j] = (m & 1) ? col[m / 2] : (col[m / 2 - 1] + col[m / 2]) / 2.0;
            }
            free(col);
        }
    }
    return rc;
}

/* Krum_b: for every candidate i the sum of the squared Euclidean distances to its
 * m - b - 2 nearest neighbours among the other candidates; the candidate with the
 * smallest sum is returned (*k_out; ties: the lowest index).  sums[m] receives the
 * per-candidate sums, dist[m*m] (may be NULL) the squared distances.
 * The definition needs at least one neighbour: m - b - 2 >= 1.  (The paper notes that
 * Krum's guarantee needs 2b + 2 < m; its own toy example uses m = 6, b = 2, so that
 * bound is not enforced here.) */
int zo_krum(int dtype, const void *V, int64_t ldv, int64_t d, int m, int b,
            int32_t *k_out, double *sums, double *dist)
{
    if (m < 1 || b < 0 || m - b - 2 < 1 || d < 1 || ldv < d) return ZO_BAD_ARG;
    const size_t esz = dtype == ZO_BF16 ? 2 : 4;
    double *D = dist ? dist : (double *)malloc(sizeof(double) * (size_t)m * (size_t)m);
    double *row = (double *)malloc(sizeof(double) * (size_t)m);
    if (!D || !row) return ZO_NO_MEM;
#pragma omp parallel for schedule(dynamic)
    for (int i = 0; i < m; ++i) {
        const char *vi = (const char *)V + (size_t)i * (size_t)ldv * esz;
        for (int j = 0; j < m; ++j) {
            const char *vj = (const char *)V + (size_t)j * (size_t)ldv * esz;
            double s = 0.0;
            for (int64_t t = 0; t < d; ++t) {
                double df = zo_load(vi, t, dtype) - zo_load(vj, t, dtype);
                s += df * df;
            }
            D[(size_t)i * m + j] = s;
        }
    }
    const int nn = m - b - 2;
    int best = 0;
    for (int i = 0; i < m; ++i) {
        int c = 0;
        for (int j = 0; j < m; ++j)
            if (j != i) {
                double v = D[(size_t)i * m + j];
                row[c++] = v != v ? INFINITY : v;          /* a NaN distance is no neighbour */
            }
        qsort(row, (size_t)c, sizeof(double), zo_cmp_double);
        double s = 0.0;
        for (int t = 0; t < nn; ++t) s += row[t];
        sums[i] = s;
        if (s < sums[best]) best = i;
    }
    *k_out = best;
    free(row);
    if (!dist) free(D);
    return ZO_OK;
}

/* ---- the workers' side of Algorithm 1, and the experiments' failures -------
 *
 * Algorithm 1, worker i: v_i = grad F_i(x) on the worker's own samples.  Written out for the two
 * losses whose gradient has a closed form that needs no back-propagation through hidden layers:
 * softmax regression (a one-layer model of the softmax family) and least squares.
 *   softmax regression:  d/dW[c][k] = (1/n) sum_j (p_j[c] - [c = label_j]) a_j[k],
 *                        d/db[c]    = (1/n) sum_j (p_j[c] - [c = label_j]),  p_j = softmax(W a_j + b);
 *   least squares:       grad = A^T (A x - y) / n.
 * flip != 0 is the experiments' label-flipping failure: every label is replaced by (classes - 1 - label)
 * before the gradient is taken (the paper's "9 - label" for ten classes). */
int zo_worker_gradient(int kind, int n_layers, const int64_t *dims, int has_bias, const void *x, int dtype,
                       const float *features, const void *targets, int n, int flip, double *grad)
{
    if (kind == ZO_LOSS_SOFTMAX_CNN)
        return ZO_BAD_ARG; /* the workers' side is stated for the dense models and least squares only */
    if (n < 1) return ZO_BAD_ARG;
    if (kind == ZO_LOSS_LEAST_SQUARES) {
        const int64_t d = dims[0];
        const float *y = (const float *)targets;
        for (int64_t k = 0; k < d; ++k) grad[k] = 0.0;
        for (int j = 0; j < n; ++j) {
            double r = -(double)y[j];
            for (int64_t k = 0; k < d; ++k) r += (double)features[(size_t)j * d + k] * zo_load(x, k, dtype);
            for (int64_t k = 0; k < d; ++k) grad[k] += (double)features[(size_t)j * d + k] * r / (double)n;
        }
        return ZO_OK;
    }
    if (kind != ZO_LOSS_SOFTMAX_MLP || n_layers != 1) return ZO_BAD_ARG;
    const int64_t in = dims[0], classes = dims[1];
    const int32_t *labels = (const int32_t *)targets;
    const int64_t d = classes * in + (has_bias ? classes : 0);
    double *z = (double *)malloc(sizeof(double) * (size_t)classes);
    if (!z) return ZO_NO_MEM;
    for (int64_t k = 0; k < d; ++k) grad[k] = 0.0;
    for (int j = 0; j < n; ++j) {
        const float *a = features + (size_t)j * in;
        double zmax = -INFINITY;
        for (int64_t c = 0; c < classes; ++c) {
            double s = has_bias ? zo_load(x, classes * in + c, dtype) : 0.0;
            for (int64_t k = 0; k < in; ++k) s += zo_load(x, c * in + k, dtype) * (double)a[k];
            z[c] = s;
            if (s > zmax) zmax = s;
        }
        double se = 0.0;
        for (int64_t c = 0; c < classes; ++c) se += exp(z[c] - zmax);
        int64_t label = labels[j];
        if (flip) label = classes - 1 - label;
        for (int64_t c = 0; c < classes; ++c) {
            const double delta = (exp(z[c] - zmax) / se - (c == label ? 1.0 : 0.0)) / (double)n;
            for (int64_t k = 0; k < in; ++k) grad[c * in + k] += delta * (double)a[k];
            if (has_bias) grad[classes * in + c] += delta;
        }
    }
    free(z);
    return ZO_OK;
}

/* The experiments' failures applied to the candidate matrix (float64 rows, [m][d]):
 *   mode 0, bit-flipping: a faulty worker pushes the negative of its gradient, and the first faulty
 *           row's (negated) gradient is copied over all other faulty rows;
 *   mode 1, scaling: a faulty row becomes eps times its gradient (the failure model's toy example,
 *           eps a large negative constant). */
int zo_inject_faults(double *V, int64_t d, int m, const int32_t *faulty, int n_faulty, int mode, double eps)
{
    if (n_faulty < 0 || (mode != 0 && mode != 1)) return ZO_BAD_ARG;
    for (int f = 0; f < n_faulty; ++f)
        if (faulty[f] < 0 || faulty[f] >= m) return ZO_BAD_ARG;
    if (n_faulty == 0) return ZO_OK;
    if (mode == 0) {
        double *first = V + (size_t)faulty[0] * d;
        for (int64_t k = 0; k < d; ++k) first[k] = -first[k];
        for (int f = 1; f < n_faulty; ++f)
            memcpy(V + (size_t)faulty[f] * d, first, sizeof(double) * (size_t)d);
    } else {
        for (int f = 0; f < n_faulty; ++f)
            for (int64_t k = 0; k < d; ++k) V[(size_t)faulty[f] * d + k] *= eps;
    }
    return ZO_OK;
}
