// Internal declarations shared by the translation units of libzeno.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "zeno.h"

namespace zeno {

// Rows of V (and x) handled per warp in the CUDA-core kernels.
constexpr int kRowsPerWarp = 4;
// Warps per block in the layer kernel; one block covers kRowsPerWarp * kLayerWarps output rows.
constexpr int kLayerWarps = 8;
// Number of k-slabs the least-squares stream is cut into is at most this.
constexpr int kMaxSlabs = 1024;
// Most kernels one call can enqueue (layers + loss + finalize + select + aggregate).
constexpr int kMaxProfiled = ZENO_MAX_LAYERS + 8;
// Calls whose per-kernel events are kept for zeno_profile_read.
constexpr int kProfileDepth = 64;

// cudaFuncSetAttribute acts on the current device only, so "already done" is remembered per device
// (one of these per kernel instantiation; devices beyond the table are simply set again each time).
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
    bool done[kMaxDevices] = {};
    bool need(int device) const { return device < 0 || device >= kMaxDevices || !done[device]; }
    void mark(int device) { if (device >= 0 && device < kMaxDevices) done[device] = true; }
};

// Polls of a barrier before a bounded device-side wait gives up: the default of a handle, and the
// limit of the waits a block's teardown makes after an abort whatever the handle says.
constexpr uint32_t kSpinLimit = 1u << 22;

// Launch shape of the tensor-core stream: k-range length, number of k-ranges, blocks per
// k-range, padded sample count, 128-row tiles per model, dynamic shared memory, ring depth.
struct StreamTcPlan { int KR, R, G, n_pad, tiles_per_model, smem_bytes, stages; };
constexpr int kStreamTcMinKR = 128;

// Which norm-partial slots a call filled: per layer (first slot, count).
struct NormSlots { int base[ZENO_MAX_LAYERS]; int count[ZENO_MAX_LAYERS]; int layers; };

struct Context {
    zeno_model_desc desc;
    int64_t d;
    int device;
    int m_max, n_r_max;
    int sm_count;
    int64_t offW[ZENO_MAX_LAYERS];  // element offset of W_l inside a parameter vector
    int64_t offB[ZENO_MAX_LAYERS];  // element offset of b_l, -1 without bias
    int np_base[ZENO_MAX_LAYERS];   // first norm-partial slot of layer l
    int np_slots;                   // norm-partial slots per candidate
    int64_t cnn_flat;               // convolutional network: inputs of its dense layer
    void *arena;                    // the one device allocation everything below is carved from
    float *act[2];                  // activations [m_max+1][n_r_max][widest layer output]
    double *loss_part;              // [m_max + 1][8] per-block sums of the sample losses
    double *loss_sum;               // [m_max + 1] per-model sums of the sample losses
    void *act_split[2];             // two-term stacked activations for the streamed tensor-core layers
    float *normpart;                // [m_max][np_slots] partial sums of v^2
    float *lsq_part;                // [slabs][m_max+1][n_r_max+1] partial A.v and v^2
    int lsq_slabs;
    float *losses;                  // [m_max+1]
    float *norms;                   // [m_max]
    float *scores;                  // [m_max]
    int32_t *idx;                   // [m_max]
    int *dev_status;                // raised by a kernel whose bounded wait gave up
    uint32_t spin_limit;            // polls a bounded device-side wait may take before it gives up
    bool tc_ok;                     // the tensor-core stream can serve the first layer (fp32 storage)
    int tc_r_max;                   // most k-ranges any plan for it may use
    float *tc_part;                 // [R][m_max+1][n_r_max][dims[1]] split-K partials
    unsigned *tickets;              // the tail's arrival counter, zero between launches
    float *head_zpart;              // partial logits of a last layer folded into the layer before it, or NULL
    unsigned *head_tickets;         // [m_max + 1] per-model arrival counters of that mode, zero between launches
    // Krum: per-block partial sums of the pairs' squared distances, and the candidates' sums
    float *krum_part;               // NULL when m_max is beyond ZENO_KRUM_MAX_M
    float *krum_sums;               // [m_max]
    int krum_blocks;                // blocks the partials were sized for
    void *host_stage;               // device copies of host inputs (zeno_step_host), grown on demand
    void *tmap_cache;               // encoded tensor maps of the tensor-core kernels (host memory, malloc'ed), or NULL
    size_t host_stage_bytes;
    int last_launches;
    int last_cuda_error;
    int last_wait_code;             // status word read back after a kernel gave up on a bounded wait
    // optional per-kernel timing (zeno_profile): a ring of the last kProfileDepth calls; in a
    // call's slot events[i] is recorded before kernel i and events[n] after the last one
    bool use_tc;                    // tensor-core kernels allowed (ZENO_DISABLE_TENSOR_CORES unset at zeno_create)
    bool chain;                     // chain a step's kernels with programmatic dependent launch
    bool profile;
    cudaEvent_t events[kProfileDepth][kMaxProfiled + 1];
    const char *kernel_names[kProfileDepth][kMaxProfiled];
    int profiled_n[kProfileDepth];
    int profiled;                   // kernels marked so far in the current call
    long long call_seq;             // calls completed since profiling was switched on
};

// Kernels overlap their set-up with the previous kernel's tail unless per-kernel events are wanted.
inline bool chain_launches(const Context &c) { return c.chain && !c.profile; }

// Records the event that closes the previous kernel and opens the next one.
inline void profile_mark(Context &c, const char *name, cudaStream_t s) {
    if (!c.profile || c.profiled >= kMaxProfiled) return;
    const int slot = (int)(c.call_seq % kProfileDepth);
    cudaEventRecord(c.events[slot][c.profiled], s);
    c.kernel_names[slot][c.profiled++] = name;
}

// What the last block of the scoring pass needs to turn losses and norm partials into scores
// (and, if keep > 0, into the ranking).
struct TailArgs {
    const float *normpart;
    int np_slots;
    NormSlots used;
    int m;
    float rho;
    float *scores;
    float *norms_out;   // may be NULL
    float *norm_tot;    // [m] workspace: ||v_i||^2 summed over the layers' partials
    double *loss_sum;   // [m+1] workspace: each model's sample losses added up in double (not yet divided by n_r)
    int n_r;
    int32_t *idx;       // used if keep > 0
    int keep;           // m - b, or 0: no ranking wanted
    unsigned *ticket;   // zero between launches
};

// One dense layer of all m+1 models (candidate 0 is x itself).
struct LayerArgs {
    const void *x;
    const void *V;
    int64_t ldv;
    int64_t offW, offB;
    int in, out;
    const float *Hin;         // input activations [m+1][n_r][in] (shared features: stride 0)
    int64_t hin_cand_stride;
    float *Hout;              // [m+1][n_r][out]
    int n_r, m;
    float gamma;
    int relu;
    float *normpart;
    int np_slots, np_base;
    // last layer only: fold the cross-entropy (and the tail) into this launch
    int fuse_loss;
    // this launch is the first of the call: whatever precedes it on the stream is the caller's and may
    // be producing x or V, so nothing is read before the preceding kernel has completed
    int first_in_call;
    const int32_t *labels;
    float *losses;
    TailArgs tail;
};

struct LsqArgs {
    const float *x;
    const float *V;
    int64_t ldv;
    int64_t d;
    const float *A;
    int n_r, m;
    float *part;      // [slabs][m+1][n_r+1]; the last column holds the partial sum of squares
    int slabs;
};

// Launchers return the cudaError_t of the launch; *launches is incremented per kernel.
cudaError_t launch_mlp_layer(Context &c, const LayerArgs &a, bool aligned, cudaStream_t s,
                             int *launches);
cudaError_t launch_mlp_loss(Context &c, const float *logits, const int32_t *labels, int n_r,
                            int m, int classes, float *losses, const TailArgs &tail, cudaStream_t s,
                            int *launches);
cudaError_t launch_lsq_partial(Context &c, const LsqArgs &a, bool aligned, double *sums, cudaStream_t s,
                               int *launches);
cudaError_t launch_lsq_from_sums(Context &c, const double *sums, int m, int n_r, const float *y, float gamma,
                                 float rho, float *losses, float *norms, float *scores, cudaStream_t s,
                                 int *launches);
bool mlp_can_fuse_loss(int out, int n_r);
// Warp-MMA version of the layer kernel (16-byte aligned rows, in % 8 == 0).
cudaError_t launch_mlp_layer_mma(Context &c, const LayerArgs &a, cudaStream_t s, int *launches);
int mlp_mma_norm_slots(int out);
bool mlp_mma_usable(int in, int out);
cudaError_t launch_lsq_score(Context &c, const LsqArgs &a, const float *y, float gamma,
                             float rho, bool aligned, float *losses, float *norms, float *scores,
                             cudaStream_t s, int *launches);
cudaError_t launch_select(Context &c, const float *scores, int m, int b, int32_t *idx, cudaStream_t s,
                          int *launches);
// xu != NULL: the parameter vector to update in the same pass, xu <- xu - gamma out (out may be NULL)
cudaError_t launch_aggregate(Context &c, const void *V, int64_t ldv, int m,
                             const int32_t *idx, int k, float *out, void *xu, float gamma, bool aligned,
                             cudaStream_t s, int *launches);

// One convolutional layer (3 x 3, stride 1, zero padding 1, ReLU, optionally followed by a 2 x 2 max
// pooling) of all m + 1 models of a ZENO_LOSS_SOFTMAX_CNN handle.
struct CnnLayerArgs {
    const void *x;
    const void *V;
    int64_t ldv;
    int64_t offW, offB;       // W[cout][cin][3][3], b[cout] (-1: none)
    int cin, cout, side;      // input planes, output planes, the planes' side (before the pooling)
    int pool;
    const float *Hin;         // [m+1][n_r][cin][side][side] (the shared batch: stride 0)
    int64_t hin_cand_stride;
    float *Hout;              // [m+1][n_r][cout][side or side / 2]^2
    int n_r, m;
    float gamma;
    float *normpart;
    int np_slots, np_base;
};
bool cnn_side_ok(int side);
int cnn_norm_slots(int cout);
cudaError_t launch_cnn_conv(Context &c, const CnnLayerArgs &a, cudaStream_t s, int *launches);

// Tensor-core stream for the first layer (fp32 storage).
bool stream_tc_plan(int sms, int K, int out, int n_r, int m, StreamTcPlan *p);
int stream_tc_norm_slots(const StreamTcPlan &p);
cudaError_t launch_stream_tc(Context &c, const StreamTcPlan &p, const float *x, const float *V, int64_t ldv,
                             int64_t offW, int64_t offB, int K, int out, const float *X, int n_r, int m,
                             float *part, int np_base, cudaStream_t s, int *launches);
cudaError_t launch_stream_combine(Context &c, const StreamTcPlan &p, const float *part, const float *x,
                                  const float *V, int64_t ldv, int64_t offB, int out, int n_r, int m,
                                  float gamma, int relu, float *H, float *Hsplit, cudaStream_t s, int *launches);

// A small last layer (at most kHeadMaxClasses outputs) folded into the tensor-core layer before it:
// that layer's epilogue multiplies its activations, still in registers, against the last layer's
// weights and leaves per-tile partial logits; the block that completes a model (a ticket per
// model) adds them up and takes the cross-entropy, and the block that completes the last model
// runs the scoring tail.  Neither the hidden activations nor the logits of that pair of layers
// are written out in full, and no further kernel is launched.
constexpr int kHeadMaxClasses = 16;
struct HeadFuse {
    int classes;             // outputs of the last layer; 0: not fused
    int64_t offW, offB;      // element offsets of its weights [classes][out] and bias (-1: none)
    float *zpart;            // [m+1][tiles][kHeadMaxClasses][n_pad] partial logits, one set per 128-row tile
    unsigned *model_ticket;  // [m+1], zero between launches
    const int32_t *labels;
    float *losses;           // [m+1]
    int np_base;             // first norm-partial slot of the last layer (one per tile and epilogue warp)
    TailArgs tail;
};
int layer_tc_head_slots(int out);

// Dense layer on the tensor cores with both operands streamed (any layer of a bfloat16 model, the
// later layers of an fp32 model).  Its input activations come as the two-term stacked operand
// [models][2 n_pad][K] that launch_split_acts, or a preceding layer of this kind, writes.
struct LayerTcLaunch {
    const void *x, *V;
    int64_t ldv, offW, offB;
    int K, out, n_r, n_pad, m;
    int h_shared;            // first layer: one set of activations for every model
    int linear;              // fp32 first layer: raw products H v_c^T into Hout, finished by the combine kernel
    const void *Hsplit_in;
    float *Hout;             // plain fp32 output [m+1][n_r][out], or NULL
    void *Hsplit_out;        // stacked two-term output for a following layer of this kind, or NULL
    int relu;
    float gamma;
    int np_base;
    const HeadFuse *head;    // the last layer folded in (Hout and Hsplit_out are then unused), or NULL
};
bool layer_tc_usable(zeno_dtype dtype, int K, int out, int n_r);
int layer_tc_n_pad(int n_r);
int layer_tc_norm_slots(int out);
cudaError_t launch_layer_tc(Context &c, const LayerTcLaunch &l, cudaStream_t s, int *launches);
cudaError_t launch_split_acts(Context &c, const float *H, int models, int n_r, int K, void *out, cudaStream_t s,
                              int *launches);

// The paper's baseline aggregation rules on the same V (zeno_baselines.cu).
size_t krum_part_floats(int m, int blocks);
cudaError_t launch_median(Context &c, const void *V, int64_t ldv, int m, float *out, cudaStream_t s, int *launches);
cudaError_t launch_krum(Context &c, const void *V, int64_t ldv, int m, int b, float *out, int32_t *k, float *sums,
                        cudaStream_t s, int *launches);

// The workers' side of Algorithm 1 and the experiments' failures (zeno_workers.cu): builders of the step's input.
bool worker_gradients_supported(const Context &c, int n);
cudaError_t launch_worker_gradients(Context &c, const void *x, const float *features, const void *targets, int n, int m,
                                    const int32_t *flip, void *V, int64_t ldv, cudaStream_t s, int *launches);
cudaError_t launch_inject_faults(Context &c, void *V, int64_t ldv, int m, const int32_t *faulty, int n_faulty, int mode,
                                 float eps, cudaStream_t s, int *launches);

int lsq_slab_count(const Context &c);
// Tensor-core version of the least-squares stream (zeno_lsq_tc.cu): one slab per block into a.part.
bool lsq_tc_usable(const LsqArgs &a, bool aligned);
cudaError_t launch_lsq_tc(Context &c, const LsqArgs &a, int max_slabs, int *slabs, cudaStream_t s);
int mlp_norm_slots(int out);

// ---- device helpers shared by the kernels ------------------------------------------------

#ifdef __CUDACC__

// Programmatic dependent launch.  Consecutive kernels of a step are chained so that a kernel's
// blocks may become resident, and run their on-chip set-up, while the kernel before it drains.
// Every kernel calls pdl_wait() before it reads or writes any global memory that a kernel of this
// library writes; pdl_wait() returns once the preceding kernel has completed and its writes are
// visible (it is a no-op for a kernel launched the ordinary way).  pdl_launch_dependents() comes
// only AFTER the kernel's own pdl_wait(): a kernel's successor can then start no earlier than the
// completion of the kernel's predecessor, so whatever a successor reads ahead of its own wait (the
// head kernel reads x and V there) cannot still be written by a kernel two places up the chain --
// the in-place update of x by the previous step's averaging pass in particular.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                  bool overlap, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t hi16_in_low) {
    return __uint_as_float(hi16_in_low << 16);
}

__device__ __forceinline__ float load_elem(const float *p) { return __ldg(p); }
__device__ __forceinline__ float load_elem(const __nv_bfloat16 *p) {
    return bf16_bits_to_float(__ldg(reinterpret_cast<const unsigned short *>(p)));
}

// four consecutive elements starting at p (p must be aligned to 4 elements)
__device__ __forceinline__ void load_vec4(const float *p, float (&o)[4]) {
    float4 t = __ldg(reinterpret_cast<const float4 *>(p));
    o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w;
}
__device__ __forceinline__ void load_vec4(const __nv_bfloat16 *p, float (&o)[4]) {
    uint2 t = __ldg(reinterpret_cast<const uint2 *>(p));
    o[0] = __uint_as_float(t.x << 16);
    o[1] = __uint_as_float(t.x & 0xffff0000u);
    o[2] = __uint_as_float(t.y << 16);
    o[3] = __uint_as_float(t.y & 0xffff0000u);
}

// value rounded to tf32 (10 explicit mantissa bits), ties away from zero in magnitude
__device__ __forceinline__ float tf32_hi(float a) {
    return __uint_as_float((__float_as_uint(a) + 0x1000u) & 0xffffe000u);
}

// (score, index) packed so that unsigned order is "higher score first, then lower index":
// the score's bits mapped to an order-preserving unsigned integer (NaN ranks with minus
// infinity, -0 is folded into +0), the index stored complemented in the low half.
__device__ __forceinline__ unsigned long long rank_key(float s, int index) {
    if (s != s) s = -INFINITY;   // a NaN score ranks with minus infinity
    s += 0.0f;                   // -0 -> +0
    unsigned u = __float_as_uint(s);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)u << 32) | (unsigned)(0xffffffffu - (unsigned)index);
}

// ReLU that lets a NaN through
__device__ __forceinline__ float relu_keep_nan(float z) { return (z > 0.f || z != z) ? z : 0.f; }

template <typename T> struct is_bf16 { static constexpr bool value = false; };
template <> struct is_bf16<__nv_bfloat16> { static constexpr bool value = true; };

// One entry of the candidate's parameter vector, x - gamma v (Definition 2's argument).
// bfloat16 models: the difference is rounded to binary32 by the fused multiply-add and then
// to bfloat16, because the candidate is itself a bfloat16 model.
template <typename T>
__device__ __forceinline__ float candidate_param(float x, float v, float gamma) {
    float w = fmaf(-gamma, v, x);
    if (is_bf16<T>::value) w = __bfloat162float(__float2bfloat16_rn(w));
    return w;
}

#endif  // __CUDACC__

}  // namespace zeno
