// C ABI of the Zeno aggregation step: argument checks, workspace, and the order in which the
// kernels are enqueued.  No arithmetic of the method lives here.
#include <math.h>
#include <new>
#include <stdlib.h>
#include <string.h>

#include <nvtx3/nvToolsExt.h>

#include "zeno_internal.h"

using zeno::Context;

struct zeno_context : public Context {};

namespace {

constexpr size_t kAlign = 256;

size_t round_up(size_t n, size_t q) { return (n + q - 1) / q * q; }

size_t elem_size(int dtype) { return dtype == ZENO_BF16 ? 2 : 4; }

// Convolutional network: dims = {S, C_0, C_1, .., C_Lc, classes}, n_layers = Lc + 1.  The side of the planes
// the dense layer sees, or 0 if the description is not a network the kernels take.
int64_t cnn_final_side(const zeno_model_desc *d) {
    const int lc = d->n_layers - 1;
    if (lc < 2 || (lc & 1) || d->n_layers + 1 > ZENO_MAX_LAYERS) return 0;
    for (int l = 0; l <= d->n_layers + 1; ++l)
        if (d->dims[l] < 1 || d->dims[l] > (int64_t)1 << 20) return 0;
    int64_t side = d->dims[0];
    for (int l = 1; l <= lc; ++l) {
        if (!zeno::cnn_side_ok((int)side)) return 0;
        if ((l & 1) == 0) side /= 2;
    }
    return side;
}

bool desc_ok(const zeno_model_desc *d) {
    if (!d) return false;
    if (d->kind == ZENO_LOSS_LEAST_SQUARES) return d->dims[0] >= 1;
    if (d->kind == ZENO_LOSS_SOFTMAX_CNN) return cnn_final_side(d) > 0;
    if (d->kind != ZENO_LOSS_SOFTMAX_MLP) return false;
    if (d->n_layers < 1 || d->n_layers > ZENO_MAX_LAYERS) return false;
    for (int l = 0; l <= d->n_layers; ++l)
        if (d->dims[l] < 1 || d->dims[l] > (int64_t)1 << 30) return false;
    return true;
}

// values of one sample's features
size_t feature_count(const zeno_model_desc &d) {
    if (d.kind == ZENO_LOSS_SOFTMAX_CNN) return (size_t)(d.dims[1] * d.dims[0] * d.dims[0]);
    return (size_t)d.dims[0];
}

bool is_aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// A named range around an entry point, visible on a profiler's timeline (a no-op without one attached).
struct Range {
    explicit Range(const char *name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
};

// Switches to the handle's device for the duration of a call and back afterwards.
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int dev) {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != dev) {
            err = cudaSetDevice(dev);
            switched = err == cudaSuccess;
        }
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

// Per-kernel timing: a call starts a fresh list of events and closes it after its last kernel.
void profile_begin(Context *c) { c->profiled = 0; }
void profile_end(Context *c, cudaStream_t s) {
    if (!c->profile) return;
    const int slot = (int)(c->call_seq % zeno::kProfileDepth);
    cudaEventRecord(c->events[slot][c->profiled], s);
    c->profiled_n[slot] = c->profiled;
    ++c->call_seq;
}

zeno_status fail_cuda(Context *c, cudaError_t e) {
    c->last_cuda_error = (int)e;
    c->last_launches = 0;
    return ZENO_ERR_CUDA;
}

// The 4-element vector loads of the scoring kernels need every row of every layer (and the
// rows of V) to start on a multiple of 4 elements.
bool score_rows_aligned(const Context &c, const void *x, const void *V, int64_t ldv,
                        const float *features) {
    const size_t vec_bytes = 4 * elem_size(c.desc.param_dtype);
    if (!is_aligned(x, vec_bytes) || !is_aligned(V, vec_bytes) || !is_aligned(features, 16)) return false;
    if (ldv % 4 != 0) return false;
    if (c.desc.kind == ZENO_LOSS_LEAST_SQUARES) return c.d % 4 == 0;
    if (c.desc.kind == ZENO_LOSS_SOFTMAX_CNN)      // only the dense layer takes vector loads
        return c.offW[c.desc.n_layers - 1] % 4 == 0 && c.cnn_flat % 4 == 0;
    for (int l = 0; l < c.desc.n_layers; ++l)
        if (c.offW[l] % 4 != 0 || c.desc.dims[l] % 4 != 0) return false;
    return true;
}

bool aggregate_rows_aligned(const Context &c, const void *V, int64_t ldv, const float *out, const void *xu) {
    return is_aligned(V, 16) && is_aligned(out, 16) && is_aligned(xu, 16) &&
           (ldv * elem_size(c.desc.param_dtype)) % 16 == 0;
}

zeno_status check_common(const Context *c, const void *V, int64_t ldv, int32_t m) {
    if (!c || !V) return ZENO_ERR_INVALID_ARG;
    if (m < 1 || m > c->m_max) return ZENO_ERR_INVALID_ARG;
    if (ldv < c->d) return ZENO_ERR_INVALID_ARG;
    return ZENO_OK;
}

// The convolutional network: its convolutional layers one launch each, then the dense layer with the
// cross-entropy and the scoring tail as for the dense models.
zeno_status enqueue_score_cnn(Context *c, const void *x, const void *V, int64_t ldv, int32_t m, const zeno_batch *batch,
                              float gamma, float rho, float *scores, float *loss_buf, float *norms, int keep,
                              int32_t *idx, bool *ranked, bool aligned, cudaStream_t s, int *launches) {
    const int n_r = batch->n_r, L = c->desc.n_layers, lc = L - 1;
    const int classes = (int)c->desc.dims[lc + 2];
    zeno::TailArgs tail;
    tail.normpart = c->normpart;
    tail.np_slots = c->np_slots;
    tail.used.layers = L;
    tail.m = m;
    tail.rho = rho;
    tail.scores = scores;
    tail.norms_out = norms;
    tail.norm_tot = c->norms;
    tail.loss_sum = c->loss_sum;
    tail.n_r = n_r;
    tail.idx = idx;
    tail.keep = keep;
    tail.ticket = c->tickets;
    int side = (int)c->desc.dims[0];
    cudaError_t e = cudaSuccess;
    for (int l = 0; l < lc; ++l) {
        zeno::CnnLayerArgs a;
        a.x = x;
        a.V = V;
        a.ldv = ldv;
        a.offW = c->offW[l];
        a.offB = c->offB[l];
        a.cin = (int)c->desc.dims[l + 1];
        a.cout = (int)c->desc.dims[l + 2];
        a.side = side;
        a.pool = (l & 1) == 1;
        a.Hin = l == 0 ? batch->features : c->act[(l - 1) & 1];
        a.hin_cand_stride = l == 0 ? 0 : (int64_t)n_r * a.cin * side * side;
        a.Hout = c->act[l & 1];
        a.n_r = n_r;
        a.m = m;
        a.gamma = gamma;
        a.normpart = c->normpart;
        a.np_slots = c->np_slots;
        a.np_base = c->np_base[l];
        tail.used.base[l] = c->np_base[l];
        tail.used.count[l] = zeno::cnn_norm_slots(a.cout);
        e = zeno::launch_cnn_conv(*c, a, s, launches);
        if (e != cudaSuccess) return fail_cuda(c, e);
        if (a.pool) side /= 2;
    }
    const bool fuse_loss = zeno::mlp_can_fuse_loss(classes, n_r);
    zeno::LayerArgs a;
    a.x = x;
    a.V = V;
    a.ldv = ldv;
    a.offW = c->offW[lc];
    a.offB = c->offB[lc];
    a.in = (int)c->cnn_flat;
    a.out = classes;
    a.Hin = c->act[(lc - 1) & 1];
    a.hin_cand_stride = (int64_t)n_r * a.in;
    a.Hout = c->act[lc & 1];
    a.n_r = n_r;
    a.m = m;
    a.gamma = gamma;
    a.relu = 0;
    a.normpart = c->normpart;
    a.np_slots = c->np_slots;
    a.np_base = c->np_base[lc];
    a.fuse_loss = fuse_loss;
    a.first_in_call = 0;
    tail.used.base[lc] = c->np_base[lc];
    tail.used.count[lc] = zeno::mlp_norm_slots(a.out);
    a.labels = static_cast<const int32_t *>(batch->targets);
    a.losses = loss_buf;
    a.tail = tail;
    e = zeno::launch_mlp_layer(*c, a, aligned, s, launches);
    if (e != cudaSuccess) return fail_cuda(c, e);
    if (!fuse_loss) {
        e = zeno::launch_mlp_loss(*c, c->act[lc & 1], static_cast<const int32_t *>(batch->targets), n_r, m, classes,
                                  loss_buf, tail, s, launches);
        if (e != cudaSuccess) return fail_cuda(c, e);
    }
    *ranked = keep > 0;
    return ZENO_OK;
}

// keep > 0 asks for the ranking as well (idx[0..keep)); *ranked tells whether the scoring pass
// delivered it (the MLP tail does) or a separate select launch is still needed.
zeno_status enqueue_score(Context *c, const void *x, const void *V, int64_t ldv, int32_t m,
                          const zeno_batch *batch, float gamma, float rho, float *scores,
                          float *losses, float *norms, int keep, int32_t *idx, bool *ranked,
                          cudaStream_t s, int *launches) {
    *ranked = false;
    zeno_status st = check_common(c, V, ldv, m);
    if (st != ZENO_OK) return st;
    if (!x || !batch || !batch->features || !batch->targets || !scores) return ZENO_ERR_INVALID_ARG;
    if (batch->n_r < 1 || batch->n_r > c->n_r_max) return ZENO_ERR_INVALID_ARG;
    if (!isfinite(gamma) || !isfinite(rho) || rho < 0.f) return ZENO_ERR_INVALID_ARG;

    const int n_r = batch->n_r;
    const bool aligned = score_rows_aligned(*c, x, V, ldv, batch->features);
    float *loss_buf = losses ? losses : c->losses;
    cudaError_t e = cudaSuccess;

    if (c->desc.kind == ZENO_LOSS_LEAST_SQUARES) {
        zeno::LsqArgs a;
        a.x = static_cast<const float *>(x);
        a.V = static_cast<const float *>(V);
        a.ldv = ldv;
        a.d = c->d;
        a.A = batch->features;
        a.n_r = n_r;
        a.m = m;
        a.part = c->lsq_part;
        a.slabs = c->lsq_slabs;
        e = zeno::launch_lsq_score(*c, a, static_cast<const float *>(batch->targets), gamma, rho,
                                   aligned, loss_buf, norms, scores, s, launches);
        return e == cudaSuccess ? ZENO_OK : fail_cuda(c, e);
    }

    if (c->desc.kind == ZENO_LOSS_SOFTMAX_CNN)
        return enqueue_score_cnn(c, x, V, ldv, m, batch, gamma, rho, scores, loss_buf, norms, keep, idx, ranked, aligned, s, launches);

    const int L = c->desc.n_layers;
    zeno::TailArgs tail;
    tail.normpart = c->normpart;
    tail.np_slots = c->np_slots;
    tail.used.layers = L;
    tail.m = m;
    tail.rho = rho;
    tail.scores = scores;
    tail.norms_out = norms;
    tail.norm_tot = c->norms;
    tail.loss_sum = c->loss_sum;
    tail.n_r = n_r;
    tail.idx = idx;
    tail.keep = keep;
    tail.ticket = c->tickets;
    const float *xf = static_cast<const float *>(x);
    const float *Vf = static_cast<const float *>(V);
    const int classes = (int)c->desc.dims[L];
    const bool fuse_loss = zeno::mlp_can_fuse_loss(classes, n_r);
    const size_t esz0 = elem_size(c->desc.param_dtype);
    const bool tc_rows = aligned && is_aligned(x, 16) && is_aligned(V, 16) && (ldv * esz0) % 16 == 0 &&
                         c->use_tc;
    // layers served by the streamed tensor-core kernel: every layer of a bfloat16 model it can take,
    // the wide later layers of an fp32 model (the first one goes to the stream that shares the batch)
    auto layer_tc_serves = [&](int l) {
        if (l < 0 || l >= L || !tc_rows) return false;
        const int in_l = (int)c->desc.dims[l], out_l = (int)c->desc.dims[l + 1];
        if ((l + 1 == L) && fuse_loss) return false;
        if (!zeno::layer_tc_usable((zeno_dtype)c->desc.param_dtype, in_l, out_l, n_r) || n_r > c->n_r_max) return false;
        if ((c->offW[l] * esz0) % 16 != 0) return false;
        if (c->desc.param_dtype == ZENO_BF16) return true;
        if (in_l < 128 || out_l < 128) return false;
        if (l > 0) return true;
        // first layer: the stream that shares the batch reads V once and nothing else, but it needs
        // split-K partials to fill the SMs; with enough whole tiles for every SM this kernel wins, and
        // beyond the stream's 64 samples it is the only tensor-core kernel there is
        return (m + 1) * ((out_l + 127) / 128) >= 2 * c->sm_count || n_r > 64;
    };
    // the layer before a small last layer takes that layer, the loss and the tail along
    auto head_folds_into = [&](int l) {
        if (l + 2 != L || c->head_zpart == nullptr || classes > zeno::kHeadMaxClasses || !layer_tc_serves(l)) return false;
        if (c->desc.dims[l] < 128) return false;     // at least two k-blocks: both converter sets take part in every tile
        // measured: the finish costs each tile about 9 us of its epilogue warps' time (two rounds of
        // fence, ticket and reads); that is cheaper than a further launch while every block has one
        // tile, and dearer once blocks take several tiles in a row
        if ((m + 1) * ((int)((c->desc.dims[l + 1] + 127) / 128)) > c->sm_count) return false;
        return !(l == 0 && c->desc.param_dtype == ZENO_F32 && c->tc_part != nullptr);      // not the linear first layer
    };
    bool have_split = false;               // the previous layer left its output in the stacked form
    for (int l = 0; l < L; ++l) {
        const int in_l = (int)c->desc.dims[l], out_l = (int)c->desc.dims[l + 1];
        const bool last_fused = (l + 1 == L) && fuse_loss;
        if (layer_tc_serves(l)) {
            const bool with_head = head_folds_into(l);
            zeno::HeadFuse hf;
            void *hs_in = c->act_split[(l + 1) & 1];
            if (!have_split) {
                const float *plain = l == 0 ? batch->features : c->act[(l - 1) & 1];
                e = zeno::launch_split_acts(*c, plain, l == 0 ? 1 : m + 1, n_r, in_l, hs_in, s, launches);
                if (e != cudaSuccess) return fail_cuda(c, e);
            }
            const bool next_tc = layer_tc_serves(l + 1);
            zeno::LayerTcLaunch t;
            t.x = x;
            t.V = V;
            t.ldv = ldv;
            t.offW = c->offW[l];
            t.offB = c->offB[l];
            t.K = in_l;
            t.out = out_l;
            t.n_r = n_r;
            t.n_pad = zeno::layer_tc_n_pad(n_r);
            t.m = m;
            t.h_shared = l == 0;
            // an fp32 first layer is linear in its weights and shares its activations: raw products,
            // then the combine kernel (one k-range) forms z_0 - gamma (P_c + b(v_c))
            t.linear = l == 0 && c->desc.param_dtype == ZENO_F32 && c->tc_part != nullptr;
            t.Hsplit_in = hs_in;
            t.Hout = t.linear ? c->tc_part : next_tc ? nullptr : c->act[l & 1];
            t.Hsplit_out = next_tc && !t.linear ? c->act_split[l & 1] : nullptr;
            t.relu = l + 1 < L;
            t.gamma = gamma;
            t.np_base = c->np_base[l];
            t.head = nullptr;
            tail.used.base[l] = c->np_base[l];
            tail.used.count[l] = zeno::layer_tc_norm_slots(out_l);
            if (with_head) {
                tail.used.base[l + 1] = c->np_base[l + 1];
                tail.used.count[l + 1] = zeno::layer_tc_head_slots(out_l);
                hf.classes = classes;
                hf.offW = c->offW[l + 1];
                hf.offB = c->offB[l + 1];
                hf.zpart = c->head_zpart;
                hf.model_ticket = c->head_tickets;
                hf.labels = static_cast<const int32_t *>(batch->targets);
                hf.losses = loss_buf;
                hf.np_base = c->np_base[l + 1];
                hf.tail = tail;                          // complete: this is the last launch of the pass
                t.head = &hf;
                t.Hout = nullptr;
                t.Hsplit_out = nullptr;
            }
            e = zeno::launch_layer_tc(*c, t, s, launches);
            if (e != cudaSuccess) return fail_cuda(c, e);
            if (with_head) {
                *ranked = keep > 0;
                return ZENO_OK;
            }
            if (t.linear) {
                zeno::StreamTcPlan one;
                one.R = 1;
                e = zeno::launch_stream_combine(*c, one, c->tc_part, xf, Vf, ldv, c->offB[l], out_l, n_r, m, gamma,
                                                l + 1 < L, next_tc ? nullptr : c->act[l & 1],
                                                next_tc ? static_cast<float *>(c->act_split[l & 1]) : nullptr, s,
                                                launches);
                if (e != cudaSuccess) return fail_cuda(c, e);
            }
            tail.used.base[l] = c->np_base[l];
            tail.used.count[l] = zeno::layer_tc_norm_slots(out_l);
            have_split = next_tc;
            continue;
        }
        have_split = false;
        // the first layer of an fp32 model on the tcgen05 stream against the shared batch, when the
        // shape and the alignment allow it
        zeno::StreamTcPlan plan;
        if (l == 0 && c->tc_ok && aligned && !last_fused &&
            zeno::stream_tc_plan(c->sm_count, in_l, out_l, n_r, m, &plan) && plan.R <= c->tc_r_max) {
            e = zeno::launch_stream_tc(*c, plan, xf, Vf, ldv, c->offW[l], c->offB[l], in_l, out_l, batch->features,
                                       n_r, m, c->tc_part, c->np_base[l], s, launches);
            if (e != cudaSuccess) return fail_cuda(c, e);
            // a following tensor-core layer takes its operand straight from the combine
            const bool next_tc = layer_tc_serves(l + 1);
            e = zeno::launch_stream_combine(*c, plan, c->tc_part, xf, Vf, ldv, c->offB[l], out_l, n_r, m, gamma,
                                            l + 1 < L, next_tc ? nullptr : c->act[l & 1],
                                            next_tc ? static_cast<float *>(c->act_split[l & 1]) : nullptr, s,
                                            launches);
            if (e != cudaSuccess) return fail_cuda(c, e);
            have_split = next_tc;
            tail.used.base[l] = c->np_base[l];
            tail.used.count[l] = zeno::stream_tc_norm_slots(plan);
            continue;
        }
        zeno::LayerArgs a;
        a.x = x;
        a.V = V;
        a.ldv = ldv;
        a.offW = c->offW[l];
        a.offB = c->offB[l];
        a.in = (int)c->desc.dims[l];
        a.out = (int)c->desc.dims[l + 1];
        a.Hin = l == 0 ? batch->features : c->act[(l - 1) & 1];
        a.hin_cand_stride = l == 0 ? 0 : (int64_t)n_r * a.in;
        a.Hout = c->act[l & 1];
        a.n_r = n_r;
        a.m = m;
        a.gamma = gamma;
        a.relu = l + 1 < L;
        a.normpart = c->normpart;
        a.np_slots = c->np_slots;
        a.np_base = c->np_base[l];
        a.fuse_loss = (l + 1 == L) && fuse_loss;
        a.first_in_call = l == 0;
        // 16-byte aligned rows of eight-parameter multiples take the warp-MMA kernel
        const size_t esz = elem_size(c->desc.param_dtype);
        const bool mma = !a.fuse_loss && aligned && c->use_tc &&
                         zeno::mlp_mma_usable(a.in, a.out) && is_aligned(x, 16) && is_aligned(V, 16) &&
                         (ldv * esz) % 16 == 0 && (a.offW * esz) % 16 == 0;
        tail.used.base[l] = c->np_base[l];
        tail.used.count[l] = mma ? zeno::mlp_mma_norm_slots(a.out) : zeno::mlp_norm_slots(a.out);
        a.labels = static_cast<const int32_t *>(batch->targets);
        a.losses = loss_buf;
        a.tail = tail;                               // complete by the time the last layer is reached
        e = mma ? zeno::launch_mlp_layer_mma(*c, a, s, launches) : zeno::launch_mlp_layer(*c, a, aligned, s, launches);
        if (e != cudaSuccess) return fail_cuda(c, e);
    }
    if (!fuse_loss) {
        e = zeno::launch_mlp_loss(*c, c->act[(L - 1) & 1], static_cast<const int32_t *>(batch->targets),
                                  n_r, m, classes, loss_buf, tail, s, launches);
        if (e != cudaSuccess) return fail_cuda(c, e);
    }
    *ranked = keep > 0;
    return ZENO_OK;
}

zeno_status enqueue_select(Context *c, const float *scores, int32_t m, int32_t b, int32_t *idx,
                           cudaStream_t s, int *launches) {
    if (!c || !scores || !idx) return ZENO_ERR_INVALID_ARG;
    if (m < 1 || m > c->m_max || b < 0 || b >= m) return ZENO_ERR_INVALID_ARG;
    cudaError_t e = zeno::launch_select(*c, scores, m, b, idx, s, launches);
    return e == cudaSuccess ? ZENO_OK : fail_cuda(c, e);
}

// xu: NULL, or the parameter vector that takes Algorithm 1's update in the same pass (out may then be NULL)
zeno_status enqueue_aggregate(Context *c, const void *V, int64_t ldv, int32_t m, const int32_t *idx,
                              int32_t k, float *out, void *xu, float gamma, cudaStream_t s, int *launches) {
    zeno_status st = check_common(c, V, ldv, m);
    if (st != ZENO_OK) return st;
    if (!idx || (!out && !xu) || k < 1 || k > m) return ZENO_ERR_INVALID_ARG;
    cudaError_t e = zeno::launch_aggregate(*c, V, ldv, m, idx, k, out, xu, gamma,
                                           aggregate_rows_aligned(*c, V, ldv, out, xu), s, launches);
    return e == cudaSuccess ? ZENO_OK : fail_cuda(c, e);
}

}  // namespace

extern "C" {

int64_t zeno_param_count(const zeno_model_desc *desc) {
    if (!desc_ok(desc)) return 0;
    if (desc->kind == ZENO_LOSS_LEAST_SQUARES) return desc->dims[0];
    if (desc->kind == ZENO_LOSS_SOFTMAX_CNN) {
        const int lc = desc->n_layers - 1;
        const int64_t side = cnn_final_side(desc), classes = desc->dims[lc + 2];
        int64_t d = 0;
        for (int l = 1; l <= lc; ++l) d += desc->dims[l + 1] * desc->dims[l] * 9 + (desc->has_bias ? desc->dims[l + 1] : 0);
        return d + classes * desc->dims[lc + 1] * side * side + (desc->has_bias ? classes : 0);
    }
    int64_t d = 0;
    for (int l = 0; l < desc->n_layers; ++l)
        d += desc->dims[l + 1] * desc->dims[l] + (desc->has_bias ? desc->dims[l + 1] : 0);
    return d;
}

zeno_status zeno_create(zeno_handle *out, const zeno_model_desc *desc, int32_t m_max,
                        int32_t n_r_max, int32_t device) {
    Range range("zeno_create");
    if (!out) return ZENO_ERR_INVALID_ARG;
    *out = nullptr;
    if (!desc) return ZENO_ERR_INVALID_ARG;
    if (desc->kind != ZENO_LOSS_SOFTMAX_MLP && desc->kind != ZENO_LOSS_LEAST_SQUARES &&
        desc->kind != ZENO_LOSS_SOFTMAX_CNN)
        return ZENO_ERR_UNSUPPORTED;
    if (desc->param_dtype != ZENO_F32 && desc->param_dtype != ZENO_BF16) return ZENO_ERR_UNSUPPORTED;
    if (desc->kind == ZENO_LOSS_LEAST_SQUARES && desc->param_dtype != ZENO_F32)
        return ZENO_ERR_UNSUPPORTED;
    if (!desc_ok(desc)) return ZENO_ERR_INVALID_ARG;
    if (m_max < 1 || m_max > ZENO_MAX_CANDIDATES || n_r_max < 1 || device < 0)
        return ZENO_ERR_INVALID_ARG;

    zeno_context *c = new (std::nothrow) zeno_context();
    if (!c) return ZENO_ERR_WORKSPACE;
    memset(static_cast<Context *>(c), 0, sizeof(Context));
    c->desc = *desc;
    c->d = zeno_param_count(desc);
    c->device = device;
    c->m_max = m_max;
    c->n_r_max = n_r_max;
    // the environment switches are read here, once: no call on the handle looks at them again
    c->chain = getenv("ZENO_DISABLE_PDL") == nullptr;
    c->use_tc = getenv("ZENO_DISABLE_TENSOR_CORES") == nullptr;
    c->spin_limit = zeno::kSpinLimit;

    DeviceGuard guard(device);
    cudaDeviceProp prop;
    cudaError_t e = guard.err != cudaSuccess ? guard.err : cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) {
        delete c;
        return ZENO_ERR_CUDA;
    }
    c->sm_count = prop.multiProcessorCount;

    const size_t rows = (size_t)m_max + 1;
    size_t act_elems = 0, norm_elems = 0, lsq_elems = 0, tc_elems = 0, ticket_elems = 1, split_elems = 0;
    size_t head_elems = 0;
    if (desc->kind == ZENO_LOSS_SOFTMAX_MLP) {
        int64_t off = 0, widest = 0;
        int slots = 0;
        for (int l = 0; l < desc->n_layers; ++l) {
            const int64_t in = desc->dims[l], o = desc->dims[l + 1];
            c->offW[l] = off;
            off += o * in;
            c->offB[l] = desc->has_bias ? off : -1;
            if (desc->has_bias) off += o;
            c->np_base[l] = slots;
            int layer_slots = zeno::mlp_norm_slots((int)o);
            if (l == 0 && desc->param_dtype == ZENO_F32 && c->use_tc) {
                // the tensor-core stream may serve the first layer: size its partials and norm slots
                // for the shortest k-range any plan may pick
                zeno::StreamTcPlan probe;
                if (zeno::stream_tc_plan(c->sm_count, (int)in, (int)o, n_r_max < 64 ? n_r_max : 64, m_max, &probe)) {
                    c->tc_ok = true;
                    c->tc_r_max = (int)((in + zeno::kStreamTcMinKR - 1) / zeno::kStreamTcMinKR);
                    probe.R = c->tc_r_max;
                    const int tc_slots = zeno::stream_tc_norm_slots(probe);
                    if (tc_slots > layer_slots) layer_slots = tc_slots;
                    const size_t need = (size_t)c->tc_r_max * rows * (size_t)n_r_max * (size_t)o;
                    if (need > tc_elems) tc_elems = need;
                }
            }
            if (zeno::layer_tc_usable((zeno_dtype)desc->param_dtype, (int)in, (int)o, n_r_max < 128 ? n_r_max : 128) &&
                c->use_tc) {
                if (zeno::layer_tc_norm_slots((int)o) > layer_slots) layer_slots = zeno::layer_tc_norm_slots((int)o);
                const size_t need = (l == 0 ? 1 : rows) * 2 * (size_t)zeno::layer_tc_n_pad(n_r_max < 128 ? n_r_max : 128) *
                                    (size_t)in;
                if (need > split_elems) split_elems = need;
                // an fp32 first layer leaves its raw products where the stream leaves its partials
                const size_t raw = rows * (size_t)n_r_max * (size_t)o;
                if (l == 0 && desc->param_dtype == ZENO_F32 && raw > tc_elems) tc_elems = raw;
            }
            // a small last layer may be folded into a tensor-core layer before it: partial logits and
            // norm partials per (128-row tile of that layer, epilogue warp)
            if (l >= 1 && l + 1 == desc->n_layers && o <= zeno::kHeadMaxClasses && c->use_tc &&
                zeno::layer_tc_usable((zeno_dtype)desc->param_dtype, (int)desc->dims[l - 1], (int)in,
                                      n_r_max < 128 ? n_r_max : 128)) {
                const int hs = zeno::layer_tc_head_slots((int)in);
                if (hs > layer_slots) layer_slots = hs;
                head_elems = rows * (size_t)(hs / 4) * zeno::kHeadMaxClasses * (size_t)zeno::layer_tc_n_pad(n_r_max < 128 ? n_r_max : 128);
            }
            slots += layer_slots;
            if (o > widest) widest = o;
        }
        c->np_slots = slots;
        act_elems = rows * (size_t)n_r_max * (size_t)widest;
        norm_elems = (size_t)m_max * (size_t)slots;
    } else if (desc->kind == ZENO_LOSS_SOFTMAX_CNN) {
        // layers 0 .. Lc - 1: the convolutional ones; layer Lc: the dense one (served by the dense kernels)
        const int lc = desc->n_layers - 1;
        int64_t off = 0, side = desc->dims[0], widest = 0;
        int slots = 0;
        for (int l = 0; l < lc; ++l) {
            const int64_t cin = desc->dims[l + 1], cout = desc->dims[l + 2];
            c->offW[l] = off;
            off += cout * cin * 9;
            c->offB[l] = desc->has_bias ? off : -1;
            if (desc->has_bias) off += cout;
            c->np_base[l] = slots;
            slots += zeno::cnn_norm_slots((int)cout);
            if ((l & 1) == 1) side /= 2;                 // the pooling is folded into every second layer
            if (cout * side * side > widest) widest = cout * side * side;
        }
        const int64_t classes = desc->dims[lc + 2];
        c->cnn_flat = desc->dims[lc + 1] * side * side;
        c->offW[lc] = off;
        off += classes * c->cnn_flat;
        c->offB[lc] = desc->has_bias ? off : -1;
        c->np_base[lc] = slots;
        slots += zeno::mlp_norm_slots((int)classes);
        if (classes > widest) widest = classes;
        c->np_slots = slots;
        act_elems = rows * (size_t)n_r_max * (size_t)widest;
        norm_elems = (size_t)m_max * (size_t)slots;
    } else {
        c->lsq_slabs = zeno::lsq_slab_count(*c);
        lsq_elems = ((size_t)c->lsq_slabs + 1) * rows * ((size_t)n_r_max + 1);
    }

    size_t bytes = 0;
    auto reserve = [&](size_t elems, size_t esz) {
        size_t at = bytes;
        bytes += round_up(elems * esz, kAlign);
        return at;
    };
    const size_t at_act0 = reserve(act_elems, 4), at_act1 = reserve(act_elems, 4);
    const size_t at_norm = reserve(norm_elems, 4), at_lsq = reserve(lsq_elems, 4);
    const size_t at_loss = reserve(rows, 4), at_norms = reserve(m_max, 4);
    const size_t at_scores = reserve(m_max, 4), at_idx = reserve(m_max, 4);
    const size_t at_status = reserve(1, 4), at_tc = reserve(tc_elems, 4);
    const size_t at_tickets = reserve(ticket_elems, 4);
    const size_t at_split0 = reserve(split_elems, 4), at_split1 = reserve(split_elems, 4);
    const size_t at_losspart = reserve(rows * 8, 8), at_losssum = reserve(rows, 8);
    const size_t at_headz = reserve(head_elems, 4), at_headt = reserve(rows, 4);
    c->krum_blocks = 8 * c->sm_count;
    const size_t krum_elems = m_max <= ZENO_KRUM_MAX_M ? zeno::krum_part_floats(m_max, c->krum_blocks) : 0;
    const size_t at_krum = reserve(krum_elems, 4), at_krums = reserve(m_max, 4);

    e = cudaMalloc(&c->arena, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        delete c;
        return ZENO_ERR_WORKSPACE;
    }
    char *base = static_cast<char *>(c->arena);
    c->act[0] = reinterpret_cast<float *>(base + at_act0);
    c->act[1] = reinterpret_cast<float *>(base + at_act1);
    c->normpart = reinterpret_cast<float *>(base + at_norm);
    c->lsq_part = reinterpret_cast<float *>(base + at_lsq);
    c->losses = reinterpret_cast<float *>(base + at_loss);
    c->norms = reinterpret_cast<float *>(base + at_norms);
    c->scores = reinterpret_cast<float *>(base + at_scores);
    c->idx = reinterpret_cast<int32_t *>(base + at_idx);
    c->dev_status = reinterpret_cast<int *>(base + at_status);
    c->tc_part = reinterpret_cast<float *>(base + at_tc);
    c->tickets = reinterpret_cast<unsigned *>(base + at_tickets);
    c->loss_part = reinterpret_cast<double *>(base + at_losspart);
    c->loss_sum = reinterpret_cast<double *>(base + at_losssum);
    c->act_split[0] = base + at_split0;
    c->act_split[1] = base + at_split1;
    c->head_zpart = head_elems ? reinterpret_cast<float *>(base + at_headz) : nullptr;
    c->head_tickets = reinterpret_cast<unsigned *>(base + at_headt);
    c->krum_part = krum_elems ? reinterpret_cast<float *>(base + at_krum) : nullptr;
    c->krum_sums = reinterpret_cast<float *>(base + at_krums);
    e = cudaMemset(c->dev_status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(c->tickets, 0, ticket_elems * sizeof(unsigned));
    if (e == cudaSuccess) e = cudaMemset(c->head_tickets, 0, rows * sizeof(unsigned));
    if (e != cudaSuccess) {
        cudaFree(c->arena);
        delete c;
        return ZENO_ERR_CUDA;
    }
    *out = c;
    return ZENO_OK;
}

zeno_status zeno_destroy(zeno_handle h) {
    Range range("zeno_destroy");
    if (!h) return ZENO_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    cudaError_t e = cudaFree(h->arena);
    if (h->host_stage) cudaFree(h->host_stage);
    free(h->tmap_cache);
    if (h->profile)
        for (int d = 0; d < zeno::kProfileDepth; ++d)
            for (int i = 0; i <= zeno::kMaxProfiled; ++i) cudaEventDestroy(h->events[d][i]);
    delete h;
    return e == cudaSuccess ? ZENO_OK : ZENO_ERR_CUDA;
}

zeno_status zeno_score(zeno_handle h, const void *x, const void *V, int64_t ldv, int32_t m,
                       const zeno_batch *batch, float gamma, float rho, float *scores,
                       float *losses, float *norms, void *stream) {
    Range range("zeno_score");
    if (!h) return ZENO_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    int launches = 0;
    profile_begin(h);
    bool ranked = false;
    zeno_status st = enqueue_score(h, x, V, ldv, m, batch, gamma, rho, scores, losses, norms, 0, nullptr,
                                   &ranked, static_cast<cudaStream_t>(stream), &launches);
    profile_end(h, static_cast<cudaStream_t>(stream));
    h->last_launches = st == ZENO_OK ? launches : 0;
    return st;
}

zeno_status zeno_select(zeno_handle h, const float *scores, int32_t m, int32_t b, int32_t *idx,
                        void *stream) {
    Range range("zeno_select");
    if (!h) return ZENO_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    int launches = 0;
    profile_begin(h);
    zeno_status st = enqueue_select(h, scores, m, b, idx, static_cast<cudaStream_t>(stream), &launches);
    profile_end(h, static_cast<cudaStream_t>(stream));
    h->last_launches = st == ZENO_OK ? launches : 0;
    return st;
}

zeno_status zeno_aggregate(zeno_handle h, const void *V, int64_t ldv, int32_t m, const int32_t *idx,
                           int32_t k, float *out, void *stream) {
    Range range("zeno_aggregate");
    if (!h) return ZENO_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    int launches = 0;
    profile_begin(h);
    zeno_status st = enqueue_aggregate(h, V, ldv, m, idx, k, out, nullptr, 0.f, static_cast<cudaStream_t>(stream),
                                       &launches);
    profile_end(h, static_cast<cudaStream_t>(stream));
    h->last_launches = st == ZENO_OK ? launches : 0;
    return st;
}

zeno_status zeno_score_partial(zeno_handle h, const void *x, const void *V, int64_t ldv, int32_t m,
                               const float *features, int32_t n_r, double *sums, void *stream) {
    Range range("zeno_score_partial");
    if (!h || !sums) return ZENO_ERR_INVALID_ARG;
    zeno_status st = check_common(h, V, ldv, m);
    if (st != ZENO_OK) return st;
    if (!x || !features || n_r < 1 || n_r > h->n_r_max) return ZENO_ERR_INVALID_ARG;
    if (h->desc.kind != ZENO_LOSS_LEAST_SQUARES) return ZENO_ERR_UNSUPPORTED;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    zeno::LsqArgs a;
    a.x = static_cast<const float *>(x);
    a.V = static_cast<const float *>(V);
    a.ldv = ldv;
    a.d = h->d;
    a.A = features;
    a.n_r = n_r;
    a.m = m;
    a.part = h->lsq_part;
    a.slabs = h->lsq_slabs;
    int launches = 0;
    profile_begin(h);
    cudaError_t e = zeno::launch_lsq_partial(*h, a, score_rows_aligned(*h, x, V, ldv, features), sums,
                                             static_cast<cudaStream_t>(stream), &launches);
    profile_end(h, static_cast<cudaStream_t>(stream));
    h->last_launches = e == cudaSuccess ? launches : 0;
    return e == cudaSuccess ? ZENO_OK : fail_cuda(h, e);
}

zeno_status zeno_score_from_sums(zeno_handle h, const double *sums, const float *targets, int32_t m, int32_t n_r,
                                 float gamma, float rho, float *scores, float *losses, float *norms, void *stream) {
    Range range("zeno_score_from_sums");
    if (!h || !sums || !targets || !scores) return ZENO_ERR_INVALID_ARG;
    if (m < 1 || m > h->m_max || n_r < 1 || n_r > h->n_r_max) return ZENO_ERR_INVALID_ARG;
    if (!isfinite(gamma) || !isfinite(rho) || rho < 0.f) return ZENO_ERR_INVALID_ARG;
    if (h->desc.kind != ZENO_LOSS_LEAST_SQUARES) return ZENO_ERR_UNSUPPORTED;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    int launches = 0;
    profile_begin(h);
    cudaError_t e = zeno::launch_lsq_from_sums(*h, sums, m, n_r, targets, gamma, rho, losses, norms, scores,
                                               static_cast<cudaStream_t>(stream), &launches);
    profile_end(h, static_cast<cudaStream_t>(stream));
    h->last_launches = e == cudaSuccess ? launches : 0;
    return e == cudaSuccess ? ZENO_OK : fail_cuda(h, e);
}

zeno_status zeno_worker_gradients(zeno_handle h, const void *x, const float *features, const void *targets, int32_t n,
                                  int32_t m, const int32_t *label_flip, void *V, int64_t ldv, void *stream) {
    Range range("zeno_worker_gradients");
    if (!h || !x || !features || !targets) return ZENO_ERR_INVALID_ARG;
    zeno_status st = check_common(h, V, ldv, m);
    if (st != ZENO_OK) return st;
    if (n < 1) return ZENO_ERR_INVALID_ARG;
    if (!zeno::worker_gradients_supported(*h, n)) return ZENO_ERR_UNSUPPORTED;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    int launches = 0;
    profile_begin(h);
    cudaError_t e = zeno::launch_worker_gradients(*h, x, features, targets, n, m, label_flip, V, ldv,
                                                  static_cast<cudaStream_t>(stream), &launches);
    profile_end(h, static_cast<cudaStream_t>(stream));
    h->last_launches = e == cudaSuccess ? launches : 0;
    return e == cudaSuccess ? ZENO_OK : fail_cuda(h, e);
}

zeno_status zeno_inject_faults(zeno_handle h, void *V, int64_t ldv, int32_t m, const int32_t *faulty, int32_t n_faulty,
                               int32_t mode, float eps, void *stream) {
    Range range("zeno_inject_faults");
    if (!h) return ZENO_ERR_INVALID_ARG;
    zeno_status st = check_common(h, V, ldv, m);
    if (st != ZENO_OK) return st;
    if (n_faulty < 0 || n_faulty > m || (n_faulty > 0 && !faulty)) return ZENO_ERR_INVALID_ARG;
    if (mode != ZENO_FAULT_BIT_FLIP && mode != ZENO_FAULT_SCALE) return ZENO_ERR_INVALID_ARG;
    if (mode == ZENO_FAULT_SCALE && !isfinite(eps)) return ZENO_ERR_INVALID_ARG;
    if (n_faulty == 0) {
        h->last_launches = 0;
        return ZENO_OK;
    }
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    int launches = 0;
    profile_begin(h);
    cudaError_t e = zeno::launch_inject_faults(*h, V, ldv, m, faulty, n_faulty, mode, eps, static_cast<cudaStream_t>(stream),
                                               &launches);
    profile_end(h, static_cast<cudaStream_t>(stream));
    h->last_launches = e == cudaSuccess ? launches : 0;
    return e == cudaSuccess ? ZENO_OK : fail_cuda(h, e);
}

zeno_status zeno_median(zeno_handle h, const void *V, int64_t ldv, int32_t m, float *out, void *stream) {
    Range range("zeno_median");
    if (!h || !out) return ZENO_ERR_INVALID_ARG;
    zeno_status st = check_common(h, V, ldv, m);
    if (st != ZENO_OK) return st;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    int launches = 0;
    profile_begin(h);
    cudaError_t e = zeno::launch_median(*h, V, ldv, m, out, static_cast<cudaStream_t>(stream), &launches);
    profile_end(h, static_cast<cudaStream_t>(stream));
    h->last_launches = e == cudaSuccess ? launches : 0;
    return e == cudaSuccess ? ZENO_OK : fail_cuda(h, e);
}

zeno_status zeno_krum(zeno_handle h, const void *V, int64_t ldv, int32_t m, int32_t b, float *out, int32_t *k,
                      float *sums, void *stream) {
    Range range("zeno_krum");
    if (!h || !k) return ZENO_ERR_INVALID_ARG;
    zeno_status st = check_common(h, V, ldv, m);
    if (st != ZENO_OK) return st;
    if (b < 0 || m - b - 2 < 1) return ZENO_ERR_INVALID_ARG;
    if (m > ZENO_KRUM_MAX_M || !h->krum_part) return ZENO_ERR_UNSUPPORTED;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    int launches = 0;
    profile_begin(h);
    cudaError_t e = zeno::launch_krum(*h, V, ldv, m, b, out, k, sums, static_cast<cudaStream_t>(stream), &launches);
    profile_end(h, static_cast<cudaStream_t>(stream));
    h->last_launches = e == cudaSuccess ? launches : 0;
    return e == cudaSuccess ? ZENO_OK : fail_cuda(h, e);
}

zeno_status zeno_step(zeno_handle h, const void *x, const void *V, int64_t ldv, int32_t m,
                      const zeno_batch *batch, float gamma, float rho, int32_t b, float *out,
                      float *scores, int32_t *idx, void *stream) {
    Range range("zeno_step");
    if (!h || !out) return ZENO_ERR_INVALID_ARG;
    if (m < 1 || m > h->m_max || b < 0 || b >= m) return ZENO_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float *score_buf = scores ? scores : h->scores;
    int32_t *idx_buf = idx ? idx : h->idx;
    int launches = 0;
    profile_begin(h);
    bool ranked = false;
    zeno_status st = enqueue_score(h, x, V, ldv, m, batch, gamma, rho, score_buf, nullptr, nullptr, m - b,
                                   idx_buf, &ranked, s, &launches);
    if (st == ZENO_OK && !ranked) st = enqueue_select(h, score_buf, m, b, idx_buf, s, &launches);
    if (st == ZENO_OK) st = enqueue_aggregate(h, V, ldv, m, idx_buf, m - b, out, nullptr, 0.f, s, &launches);
    profile_end(h, s);
    h->last_launches = st == ZENO_OK ? launches : 0;
    return st;
}

zeno_status zeno_step_update(zeno_handle h, void *x, const void *V, int64_t ldv, int32_t m,
                             const zeno_batch *batch, float gamma, float rho, int32_t b, float *out,
                             float *scores, int32_t *idx, void *stream) {
    Range range("zeno_step_update");
    if (!h || !x) return ZENO_ERR_INVALID_ARG;
    if (m < 1 || m > h->m_max || b < 0 || b >= m) return ZENO_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float *score_buf = scores ? scores : h->scores;
    int32_t *idx_buf = idx ? idx : h->idx;
    int launches = 0;
    profile_begin(h);
    bool ranked = false;
    zeno_status st = enqueue_score(h, x, V, ldv, m, batch, gamma, rho, score_buf, nullptr, nullptr, m - b,
                                   idx_buf, &ranked, s, &launches);
    if (st == ZENO_OK && !ranked) st = enqueue_select(h, score_buf, m, b, idx_buf, s, &launches);
    // the scoring pass has read x by the time the average is formed: the update goes in place
    if (st == ZENO_OK) st = enqueue_aggregate(h, V, ldv, m, idx_buf, m - b, out, x, gamma, s, &launches);
    profile_end(h, s);
    h->last_launches = st == ZENO_OK ? launches : 0;
    return st;
}

zeno_status zeno_run(zeno_handle h, void *x, const void *V, int64_t ldv, int64_t step_stride_v, int32_t m,
                     const float *features, const void *targets, int32_t n_r, int32_t steps, float gamma,
                     float rho, int32_t b, float *scores, int32_t *idx, void *stream) {
    Range range("zeno_run");
    if (!h || !x || !V || !features || !targets) return ZENO_ERR_INVALID_ARG;
    if (steps < 1 || m < 1 || m > h->m_max || b < 0 || b >= m) return ZENO_ERR_INVALID_ARG;
    if (n_r < 1 || n_r > h->n_r_max || ldv < h->d || step_stride_v < (int64_t)m * ldv) return ZENO_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t esz = elem_size(h->desc.param_dtype);
    const size_t feat_stride = (size_t)n_r * feature_count(h->desc);
    int launches = 0;
    profile_begin(h);
    zeno_status st = ZENO_OK;
    for (int32_t t = 0; t < steps && st == ZENO_OK; ++t) {
        // iteration t of Algorithm 1's server loop: its own candidates and its own batch, the x of iteration t - 1
        const void *Vt = static_cast<const char *>(V) + (size_t)t * (size_t)step_stride_v * esz;
        zeno_batch batch;
        batch.features = features + (size_t)t * feat_stride;
        batch.targets = static_cast<const char *>(targets) + (size_t)t * (size_t)n_r * 4;
        batch.n_r = n_r;
        float *score_buf = scores ? scores + (size_t)t * m : h->scores;
        int32_t *idx_buf = idx ? idx + (size_t)t * (m - b) : h->idx;
        bool ranked = false;
        st = enqueue_score(h, x, Vt, ldv, m, &batch, gamma, rho, score_buf, nullptr, nullptr, m - b, idx_buf, &ranked,
                           s, &launches);
        if (st == ZENO_OK && !ranked) st = enqueue_select(h, score_buf, m, b, idx_buf, s, &launches);
        if (st == ZENO_OK) st = enqueue_aggregate(h, Vt, ldv, m, idx_buf, m - b, nullptr, x, gamma, s, &launches);
    }
    profile_end(h, s);
    h->last_launches = st == ZENO_OK ? launches : 0;
    return st;
}

zeno_status zeno_step_host(zeno_handle h, const void *x, const void *V, int64_t ldv, int32_t m,
                           const float *features, const void *targets, int32_t n_r, float gamma,
                           float rho, int32_t b, float *out, float *scores, int32_t *idx,
                           void *stream) {
    Range range("zeno_step_host");
    if (!h || !x || !V || !features || !targets || !out) return ZENO_ERR_INVALID_ARG;
    if (m < 1 || m > h->m_max || b < 0 || b >= m || ldv < h->d) return ZENO_ERR_INVALID_ARG;
    if (n_r < 1 || n_r > h->n_r_max) return ZENO_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t esz = elem_size(h->desc.param_dtype);
    const size_t in0 = feature_count(h->desc);
    const size_t x_bytes = round_up((size_t)h->d * esz, kAlign);
    const size_t v_bytes = round_up((size_t)m * (size_t)ldv * esz, kAlign);
    const size_t f_bytes = round_up((size_t)n_r * in0 * 4, kAlign);
    const size_t t_bytes = round_up((size_t)n_r * 4, kAlign);
    const size_t o_bytes = round_up((size_t)h->d * 4, kAlign);
    const size_t need = x_bytes + v_bytes + f_bytes + t_bytes + o_bytes;
    cudaError_t e;
    if (need > h->host_stage_bytes) {
        // grown on demand; the previous staging area may still be in use by earlier work
        e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return fail_cuda(h, e);
        if (h->host_stage) cudaFree(h->host_stage);
        h->host_stage = nullptr;
        h->host_stage_bytes = 0;
        e = cudaMalloc(&h->host_stage, need);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return ZENO_ERR_WORKSPACE;
        }
        h->host_stage_bytes = need;
    }
    char *p = static_cast<char *>(h->host_stage);
    void *dx = p;
    void *dV = p + x_bytes;
    float *df = reinterpret_cast<float *>(p + x_bytes + v_bytes);
    void *dt = p + x_bytes + v_bytes + f_bytes;
    float *dout = reinterpret_cast<float *>(p + x_bytes + v_bytes + f_bytes + t_bytes);
    e = cudaMemcpyAsync(dx, x, (size_t)h->d * esz, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dV, V, (size_t)m * (size_t)ldv * esz, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(df, features, (size_t)n_r * in0 * 4, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dt, targets, (size_t)n_r * 4, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return fail_cuda(h, e);
    zeno_batch batch;
    batch.features = df;
    batch.targets = dt;
    batch.n_r = n_r;
    int launches = 0;
    profile_begin(h);
    bool ranked = false;
    zeno_status st = enqueue_score(h, dx, dV, ldv, m, &batch, gamma, rho, h->scores, nullptr, nullptr, m - b,
                                   h->idx, &ranked, s, &launches);
    if (st == ZENO_OK && !ranked) st = enqueue_select(h, h->scores, m, b, h->idx, s, &launches);
    if (st == ZENO_OK) st = enqueue_aggregate(h, dV, ldv, m, h->idx, m - b, dout, nullptr, 0.f, s, &launches);
    profile_end(h, s);
    if (st != ZENO_OK) {
        h->last_launches = 0;
        return st;
    }
    e = cudaMemcpyAsync(out, dout, (size_t)h->d * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && scores)
        e = cudaMemcpyAsync(scores, h->scores, (size_t)m * 4, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && idx)
        e = cudaMemcpyAsync(idx, h->idx, (size_t)(m - b) * 4, cudaMemcpyDeviceToHost, s);
    int dev_status = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&dev_status, h->dev_status, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail_cuda(h, e);
    h->last_launches = launches;
    if (dev_status) h->last_wait_code = dev_status;
    return dev_status ? ZENO_ERR_TIMEOUT : ZENO_OK;
}

zeno_status zeno_device_status(zeno_handle h, void *stream) {
    if (!h) return ZENO_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int dev_status = 0;
    cudaError_t e = cudaMemcpyAsync(&dev_status, h->dev_status, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return fail_cuda(h, e);
    if (dev_status) h->last_wait_code = dev_status;
    return dev_status ? ZENO_ERR_TIMEOUT : ZENO_OK;
}

zeno_status zeno_profile(zeno_handle h, int32_t enable) {
    if (!h) return ZENO_ERR_INVALID_ARG;
    DeviceGuard guard(h->device);
    if (guard.err != cudaSuccess) return fail_cuda(h, guard.err);
    const int total = zeno::kProfileDepth * (zeno::kMaxProfiled + 1);
    cudaEvent_t *flat = &h->events[0][0];
    if (enable && !h->profile) {
        for (int i = 0; i < total; ++i) {
            cudaError_t e = cudaEventCreate(&flat[i]);
            if (e != cudaSuccess) {
                for (int j = 0; j < i; ++j) cudaEventDestroy(flat[j]);
                return fail_cuda(h, e);
            }
        }
        h->profile = true;
    } else if (!enable && h->profile) {
        for (int i = 0; i < total; ++i) cudaEventDestroy(flat[i]);
        h->profile = false;
    }
    h->profiled = 0;
    h->call_seq = 0;
    for (int d = 0; d < zeno::kProfileDepth; ++d) h->profiled_n[d] = 0;
    return ZENO_OK;
}

int32_t zeno_profile_read(zeno_handle h, int32_t back, float *ms, const char **names, int32_t cap) {
    if (!h || !h->profile || back < 0 || back >= zeno::kProfileDepth || back >= h->call_seq) return 0;
    const int slot = (int)((h->call_seq - 1 - back) % zeno::kProfileDepth);
    const int count = h->profiled_n[slot];
    if (count == 0) return 0;
    DeviceGuard guard(h->device);
    if (cudaEventSynchronize(h->events[slot][count]) != cudaSuccess) return -1;
    int n = count < cap ? count : cap;
    for (int i = 0; i < n; ++i) {
        float t = 0.f;
        if (cudaEventElapsedTime(&t, h->events[slot][i], h->events[slot][i + 1]) != cudaSuccess) return -1;
        if (ms) ms[i] = t;
        if (names) names[i] = h->kernel_names[slot][i];
    }
    return n;
}

zeno_status zeno_debug_set_wait_limit(zeno_handle h, uint32_t polls) {
    if (!h) return ZENO_ERR_INVALID_ARG;
    h->spin_limit = polls;
    return ZENO_OK;
}

int32_t zeno_last_launch_count(zeno_handle h) { return h ? h->last_launches : 0; }

int32_t zeno_last_cuda_error(zeno_handle h) { return h ? h->last_cuda_error : 0; }

int32_t zeno_last_wait_code(zeno_handle h) { return h ? h->last_wait_code : 0; }

const char *zeno_status_string(zeno_status s) {
    switch (s) {
        case ZENO_OK: return "ok";
        case ZENO_ERR_INVALID_ARG: return "invalid argument";
        case ZENO_ERR_UNSUPPORTED: return "unsupported loss / dtype / shape";
        case ZENO_ERR_WORKSPACE: return "workspace allocation failed";
        case ZENO_ERR_CUDA: return "CUDA runtime error";
        case ZENO_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

}  // extern "C"
