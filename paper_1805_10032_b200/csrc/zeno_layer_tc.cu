// Dense layers of all m+1 models on the 5th-generation tensor cores, both operands streamed.
//
// For every model c the layer is  Z_c = H_c (x - gamma v_c)^T + b_c  with H_c the model's own input
// activations [n_r x K] (the shared server batch for the first layer).  A block takes whole
// 128-row tiles of one model's weight matrix over the full input range K, so there are no split-K
// partial sums: the epilogue adds the bias, applies the activation and writes the layer's output.
//
// Per k-block (128 bytes of every row: 32 floats or 64 bfloat16) TMA fills a stage of each of two rings:
//   the weight ring: the x tile and the v tile (128 rows each, 128-byte swizzled), free again as soon
//   as a converter set has read them, and
//   the activation ring: the k-block of the activations, already split into two terms and stacked --
//   rows 0..n_pad-1 hold h_hi, rows n_pad..2 n_pad-1 hold h_lo, so that one MMA yields w h_hi and
//   w h_lo side by side -- free once the MMAs that read it have finished.
// Converter warps form the candidate's weights w = x - gamma v from the two tiles (thread = row),
// accumulate v^2 for the score's norm term, and put w into TMEM as the MMA's A operand; the
// activations are the B operand, read from the stage by the tensor core itself.
//
//   fp32 storage : w is split too, w = w_hi + w_lo (tf32 + remainder); D1 += w_hi [h_hi; h_lo]^T,
//                  D2 += w_lo h_hi^T (kind::tf32, K = 8 per MMA); result D1[j] + D1[n_pad + j] + D2[j].
//   bf16 storage : the candidate is a bfloat16 model, w = RN_bf16(x - gamma v) is exact in the A
//                  operand; the fp32 activations are carried as two bfloat16 terms;
//                  D += w [h_hi; h_lo]^T (kind::f16, K = 16 per MMA); result D[j] + D[n_pad + j].
//
// Warp roles: warps 0 and 2 TMA producers (weight ring, activation ring), warp 1 MMA issuer and owner of
// TMEM (all three stay converged and issue from one elected lane; the issuer takes two k-blocks per turn), warps 4-11 two converter sets taking alternate k-blocks, warps
// 12-15 epilogue.  Accumulator sets alternate between consecutive tiles when two fit in TMEM, so
// a tile is drained while the next one is accumulated.  Every mbarrier wait is bounded; a wait that
// gives up raises a status word and the block leaves through the common teardown.
//
// HEAD mode (the layer before a small last layer): the epilogue thread of output row o holds that
// row's activations of all samples in registers, so it multiplies them against column o of the
// last layer's weights (formed as x - gamma v on the spot, v^2 accumulated); the four epilogue
// warps add their 128 rows up through shared memory and leave one set of partial logits per tile.
// The epilogue group then takes a ticket for the model: the group that completes a model sums the
// tiles' partial logits in tile order, takes the cross-entropy and the candidate's norm total, and
// takes the pass's ticket; the block that completes the last model forms the scores and the
// ranking after its teardown.  All of it runs beside the main loop of the block's next tile.
#include "zeno_internal.h"
#include "zeno_tail.cuh"
#include "zeno_tc.cuh"

namespace zeno {

namespace {

constexpr int kRows = 128;                  // weight rows per tile = TMEM lanes
constexpr int kRowBytes = 128;              // bytes of a row per k-block = one swizzle row
constexpr int kTileBytes = kRows * kRowBytes;
constexpr int kLThreads = 32 * 16;
constexpr int kLMaxStages = 12;               // weight ring (x and v tiles)
constexpr int kLMaxBStages = 6;               // activation ring
constexpr int kLMaxABufs = 8;
constexpr int kLMaxSets = 2;
constexpr int kLSmemBudget = 226 * 1024;
constexpr int kLTmemCols = 512;

// Depth of the activation ring: 96 KB worth of stages, three to six (measured: a copy from L2 takes
// two to three microseconds under load, and the MMAs consume a stage in well under one).
inline int layer_tc_b_stages(int n_pad) {
    const int fit = 96 * 1024 / (2 * n_pad * kRowBytes);
    return fit < 3 ? 3 : fit > kLMaxBStages ? kLMaxBStages : fit;
}

template <typename T> struct TcTraits;
template <> struct TcTraits<float> {
    static constexpr int kBlockK = 32;      // elements per k-block
    static constexpr int kACols = 64;       // TMEM columns of one A buffer: w_hi then w_lo
    static constexpr int kAccPerPad = 3;    // accumulator columns per padded sample
    static constexpr CUtensorMapDataType kMapType = CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
};
template <> struct TcTraits<__nv_bfloat16> {
    static constexpr int kBlockK = 64;
    static constexpr int kACols = 32;
    static constexpr int kAccPerPad = 2;
    static constexpr CUtensorMapDataType kMapType = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
};

__device__ __forceinline__ void tc_mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

struct LayerTcArgs {
    const void *xparams;   // the parameter vector x (bias entries)
    const void *V;
    int64_t ldv, offB;     // offB: element offset of the layer's bias inside a parameter vector, -1 if none
    float gamma;
    int K, out, n_r, n_pad, m;
    int tiles;             // ceil(out / 128)
    int h_shared;          // every model reads the same activations (first layer)
    int stages, b_stages, n_sets, n_abufs;   // stages: weight ring; b_stages: activation ring
    float *Hout;           // [m+1][n_r][out] fp32, or NULL
    void *Hsplit;          // [m+1][2 n_pad][out] two-term activations for a following layer of this kind, or NULL
    int relu;
    float *normpart;
    int np_slots, np_base;
    int *status;
    uint32_t spin_limit;   // polls a bounded wait may take
    HeadFuse head;         // used by the HEAD instantiations only
};

// Sum over the 32 lanes of each of 32 per-lane values; lane j ends up with the total of value j
// (recursive halving: 31 shuffles).
__device__ __forceinline__ float lane_transpose_sum32(float (&v)[32], int lane) {
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const bool upper = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < s; ++i) {
            const float send = upper ? v[i] : v[i + s];
            const float keep = upper ? v[i + s] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
        }
    }
    return v[0];
}

constexpr int kEpiThreads = 128;            // the four epilogue warps
constexpr int kEpiBarrier = 1;              // their named barrier

__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync %0, %1;" ::"n"(kEpiBarrier), "n"(kEpiThreads) : "memory"); }
// true iff `ok` holds in every thread of the epilogue group (a barrier as well)
__device__ __forceinline__ bool epi_all(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n.reg .pred p, q;\nsetp.ne.b32 p, %1, 0;\n"
        "bar.red.and.pred q, %2, %3, p;\nselp.u32 %0, 1, 0, q;\n}\n"
        : "=r"(r) : "r"((uint32_t)ok), "n"(kEpiBarrier), "n"(kEpiThreads) : "memory");
    return r != 0;
}

// HEAD mode, the 128 threads of the epilogue group that completed `model` (g = thread within the
// group): the model's logits from the tiles' partial sums in tile order plus the last layer's bias;
// then one warp takes the mean cross-entropy into losses[model] while another adds up the
// candidate's norm partials of all layers.  `zl` is group-shared scratch of classes x n_pad floats.
template <typename T>
__device__ __forceinline__ void head_finish_model(const LayerTcArgs &a, int model, float *zl, int g) {
    const HeadFuse &h = a.head;
    const int n_pad = a.n_pad, lane = g & 31, gw = g >> 5;
    const float *zp = h.zpart + (int64_t)model * a.tiles * kHeadMaxClasses * n_pad;
    for (int t = g; t < h.classes * n_pad; t += kEpiThreads) {
        const int cls = t / n_pad, j = t - cls * n_pad;
        const float *src = zp + (int64_t)cls * n_pad + j;
        const int64_t tstride = (int64_t)kHeadMaxClasses * n_pad;
        float z = 0.f;
        for (int t0 = 0; t0 < a.tiles; t0 += 4) {          // four loads in flight, added in tile order
            float part[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) part[u] = t0 + u < a.tiles ? __ldcg(src + (t0 + u) * tstride) : 0.f;
#pragma unroll
            for (int u = 0; u < 4; ++u) z += part[u];
        }
        if (h.offB >= 0) {
            const float bv = model > 0 ? load_elem(static_cast<const T *>(a.V) + (int64_t)(model - 1) * a.ldv + h.offB + cls) : 0.f;
            z += candidate_param<T>(load_elem(static_cast<const T *>(a.xparams) + h.offB + cls), bv, a.gamma);
        }
        zl[cls * n_pad + j] = z;
    }
    epi_sync();
    if (gw == 0) {
        double l = 0.0;
        for (int j = lane; j < a.n_r; j += 32) {
            float zmax = -INFINITY;
            for (int o = 0; o < h.classes; ++o) zmax = fmaxf(zmax, zl[o * n_pad + j]);
            float se = 0.f;
            for (int o = 0; o < h.classes; ++o) se += expf(zl[o * n_pad + j] - zmax);   // a NaN logit makes se NaN
            int lab = h.labels[j];
            if (lab < 0 || lab >= h.classes) lab = 0;
            l += (double)((zmax - zl[lab * n_pad + j]) + logf(se));
        }
#pragma unroll
        for (int sft = 16; sft >= 1; sft >>= 1) l += __shfl_xor_sync(0xffffffffu, l, sft);
        if (lane == 0) {
            h.tail.loss_sum[model] = l;
            h.losses[model] = (float)(l / (double)a.n_r);
            __threadfence();
        }
    } else if (gw == 1 && model > 0) {
        // the candidate's ||v||^2: the partial sums of every layer, eight loads per lane in flight
        float nv = 0.f;
        for (int l = 0; l < h.tail.used.layers; ++l) {
            const float *src = h.tail.normpart + (int64_t)(model - 1) * h.tail.np_slots + h.tail.used.base[l];
            const int count = h.tail.used.count[l];
            for (int s0 = 0; s0 < count; s0 += 256) {
                float v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int sl = s0 + u * 32 + lane;
                    v[u] = sl < count ? __ldcg(src + sl) : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) nv += v[u];
            }
        }
#pragma unroll
        for (int sft = 16; sft >= 1; sft >>= 1) nv += __shfl_xor_sync(0xffffffffu, nv, sft);
        if (lane == 0) {
            h.tail.norm_tot[model - 1] = nv;
            __threadfence();
        }
    }
    epi_sync();
}

template <typename T, bool LINEAR, bool HEAD>
__global__ void __launch_bounds__(kLThreads, 1)
layer_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_v,
                const __grid_constant__ CUtensorMap map_h, LayerTcArgs a) {
    using Tr = TcTraits<T>;
    constexpr bool kBf16 = is_bf16<T>::value;
    constexpr int kBlockK = Tr::kBlockK;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // full, empty [kLMaxStages] (weight ring); bfull, bempty [kLMaxBStages] (activation ring);
    // a_full, a_empty [kLMaxABufs]; d_full, d_empty [2]
    constexpr int kBars = 2 * kLMaxStages + 2 * kLMaxBStages + 2 * kLMaxABufs + 2 * kLMaxSets;
    __shared__ __align__(8) uint64_t bars[kBars];
    __shared__ __align__(8) uint64_t drain_bar;   // teardown after an abort: the issuer's last commit
    __shared__ __align__(8) uint64_t never_bar;   // nothing arrives here (test hook, see wait_for_nothing)
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_state[kAbortWords];
    int &abort_flag = abort_state[0];
    __shared__ int issued[kLMaxStages + kLMaxBStages];     // last round a copy was issued into a stage, plus one
    __shared__ int head_last;                  // HEAD: the epilogue group's ticket result
    __shared__ int head_final;                 // HEAD: this block completed the last model

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
    if (tid == 32) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    if (tid == 64) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_h) : "memory");

    const int nkb = (a.K + kBlockK - 1) / kBlockK;
    const int n_items = (a.m + 1) * a.tiles;
    const int n_stages = a.stages, n_bstages = a.b_stages, n_abufs = a.n_abufs, n_sets = a.n_sets;
    const int b_bytes = 2 * a.n_pad * kRowBytes;                // a stage of the activation ring
    constexpr int kWTiles = LINEAR ? 1 : 2;                     // weight tiles per stage
    constexpr int stage_bytes = kWTiles * kTileBytes;           // a stage of the weight ring: x tile, v tile
    const int acc_cols = Tr::kAccPerPad * a.n_pad;
    const int a_base = n_sets * acc_cols;                       // TMEM: accumulator sets, then the A buffers
    const float inv_stages = 1.0f / (float)n_stages, inv_abufs = 1.0f / (float)n_abufs;
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // HEAD: behind the ring, the epilogue warps' partial logits [4][classes rounded up to even][n_pad]
    uint8_t *bring = ring + (size_t)n_stages * stage_bytes;     // the activation ring follows the weight ring
    float *zq = reinterpret_cast<float *>(bring + (size_t)n_bstages * b_bytes);

    auto bar_full = [&](int s) { return smem_u32(&bars[s]); };
    auto bar_empty = [&](int s) { return smem_u32(&bars[kLMaxStages + s]); };
    constexpr int kBarB = 2 * kLMaxStages, kBarA = kBarB + 2 * kLMaxBStages, kBarD = kBarA + 2 * kLMaxABufs;
    auto bar_bfull = [&](int s) { return smem_u32(&bars[kBarB + s]); };
    auto bar_bempty = [&](int s) { return smem_u32(&bars[kBarB + kLMaxBStages + s]); };
    auto bar_afull = [&](int g) { return smem_u32(&bars[kBarA + g]); };
    auto bar_aempty = [&](int g) { return smem_u32(&bars[kBarA + kLMaxABufs + g]); };
    auto bar_dfull = [&](int q) { return smem_u32(&bars[kBarD + q]); };
    auto bar_dempty = [&](int q) { return smem_u32(&bars[kBarD + kLMaxSets + q]); };
    // item li of this block -> (model, tile); neighbouring blocks share a model's activations in L2
    auto get_item = [&](int li, int &model, int &tile) {
        const int item = blockIdx.x + li * gridDim.x;
        model = item / a.tiles;
        tile = item - model * a.tiles;
        return item < n_items;
    };

    if (tid == 0) {
        abort_flag = 0;
        abort_state[1] = (int)a.spin_limit;
        head_final = 0;
        for (int s = 0; s < kLMaxStages; ++s) {
            mbar_init(bar_full(s), 1);
            mbar_init(bar_empty(s), 4);        // the four warps of the converter set that read the tiles
            issued[s] = 0;
        }
        for (int s = 0; s < kLMaxBStages; ++s) {
            mbar_init(bar_bfull(s), 1);
            mbar_init(bar_bempty(s), 1);       // the commit of the MMAs that read the activations
            issued[kLMaxStages + s] = 0;
        }
        for (int g = 0; g < kLMaxABufs; ++g) {
            mbar_init(bar_afull(g), 4);
            mbar_init(bar_aempty(g), 1);
        }
        for (int q = 0; q < kLMaxSets; ++q) {
            mbar_init(bar_dfull(q), 1);
            mbar_init(bar_dempty(q), 4);
        }
        mbar_init(smem_u32(&drain_bar), 1);
        mbar_init(smem_u32(&never_bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // TMEM allocation by one full warp
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(kLTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_wait();                                        // the activations come from the preceding kernel
    pdl_launch_dependents();
    const uint32_t tmem = tmem_base_slot;
    volatile int *abortp = &abort_flag;

    if (warp == 0) wait_for_nothing(smem_u32(&never_bar), abortp);
    if (warp == 0 || warp == 2) {
        // ------------------------------------------------------------------ TMA producers
        // warp 0 feeds the weight ring (x tile, v tile), warp 2 the activation ring; the two rings
        // have their own depths because their stages live for different times: a weight stage is free
        // as soon as a converter set has read it, an activation stage only when its MMAs have finished.
        const bool acts = warp == 2;
        const int ring_stages = acts ? n_bstages : n_stages;
        int s = 0;
        uint32_t round = 0;
        int model, tile;
        for (int li = 0;; ++li) {
            if (!__all_sync(0xffffffffu, get_item(li, model, tile) && !*abortp)) break;
            const bool has_v = model > 0;                 // model 0 is x itself
            bool ok = true;
            for (int kb = 0; kb < nkb; ++kb) {
                const uint32_t empty = acts ? bar_bempty(s) : bar_empty(s), full = acts ? bar_bfull(s) : bar_full(s);
                ok = __all_sync(0xffffffffu, mbar_wait(empty, (round & 1) ^ 1, abortp));
                if (!ok) break;
                if (elect_one()) {
                    const uint32_t dst = acts ? smem_u32(bring + (size_t)s * b_bytes) : smem_u32(ring + (size_t)s * stage_bytes);
                    mbar_expect_tx(full, acts ? b_bytes : (has_v && !LINEAR ? 2 : 1) * kTileBytes);
                    issued[acts ? kLMaxStages + s : s] = (int)round + 1;
#pragma unroll 1
                    for (int w = acts ? 2 : 0; w < (acts ? 3 : 2); ++w) {     // x tile, v tile | activations: ONE issue site
                        // LINEAR: the only weight tile is x's for model 0, v's otherwise
                        if (LINEAR ? w == (has_v ? 0 : 1) : (w == 1 && !has_v)) continue;
                        const CUtensorMap *map = w == 0 ? &map_x : w == 1 ? &map_v : &map_h;
                        const int c1 = w == 2 ? 0 : tile * kRows;
                        const int c2 = w == 0 ? 0 : w == 1 ? model - 1 : (a.h_shared ? 0 : model);
                        const int slot = w == 2 ? 0 : (LINEAR ? 0 : w);
                        tma_load_3d(dst + slot * kTileBytes, map, kb * kBlockK, c1, c2, full);
                    }
                }
                __syncwarp();
                if (++s == ring_stages) {
                    s = 0;
                    ++round;
                }
            }
            if (!ok) break;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // instruction descriptor: D fp32, A and B tf32 (2) or bf16 (1), both K-major, M = 128
        const uint32_t fmt = kBf16 ? 1u : 2u;
        const uint32_t idesc_base = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(kRows >> 4) << 24);
        const uint32_t idesc_n = idesc_base | ((uint32_t)(a.n_pad >> 3) << 17);          // N = n_pad
        const uint32_t idesc_2n = idesc_base | ((uint32_t)((2 * a.n_pad) >> 3) << 17);   // N = 2 n_pad
        const int kb_step = n_bstages >= 4 ? 2 : 1;
        int bs = 0, ag = 0;                              // activation stage and A buffer of the next k-block
        uint32_t bph = 0, aph = 0;                       // and the phases their full barriers are awaited in
        int model, tile;
        for (int li = 0;; ++li) {
            if (!__all_sync(0xffffffffu, get_item(li, model, tile) && !*abortp)) break;
            const int set = li % n_sets;
            const uint32_t use = (uint32_t)(li / n_sets);        // earlier uses of this accumulator set
            if (!__all_sync(0xffffffffu, mbar_wait(bar_dempty(set), (use & 1) ^ 1, abortp))) break;
            tc_fence_after();
            const uint32_t d1 = tmem + set * acc_cols, d2 = d1 + 2 * a.n_pad;
            bool ok = true;
            // Two k-blocks per turn of the loop: by the time this warp gets there the operands of both
            // are long in place (cycle stamps put them ~800 cycles ahead), and the waits, the vote, the
            // fence, the election and the loop's own arithmetic cost this warp -- the one every other
            // role ends up waiting for -- as much as the sixteen MMAs it issues.  Only with an activation ring
            // of four stages or more: with three (128 samples), holding two back at a time measured slower.
            for (int kb = 0; kb < nkb; kb += kb_step) {
                const bool two = kb_step == 2 && kb + 1 < nkb;
                int s1 = bs + 1, g1 = ag + 1;
                uint32_t sph1 = bph, gph1 = aph;
                if (s1 == n_bstages) { s1 = 0; sph1 ^= 1; }
                if (g1 == n_abufs) { g1 = 0; gph1 ^= 1; }
                // all probes are issued before any result is looked at: each costs this warp a round trip to
                // shared memory, and one after the other they took longer than issuing the MMAs
                bool r0 = mbar_try_wait(bar_bfull(bs), bph), r1 = mbar_try_wait(bar_afull(ag), aph);
                bool r2 = !two || mbar_try_wait(bar_bfull(s1), sph1), r3 = !two || mbar_try_wait(bar_afull(g1), gph1);
                if (!r0) r0 = mbar_wait_poll(bar_bfull(bs), bph, abortp);
                if (!r1) r1 = mbar_wait_poll(bar_afull(ag), aph, abortp);
                if (!r2) r2 = mbar_wait_poll(bar_bfull(s1), sph1, abortp);
                if (!r3) r3 = mbar_wait_poll(bar_afull(g1), gph1, abortp);
                ok = __all_sync(0xffffffffu, r0 && r1 && r2 && r3);
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h == 1 && !two) break;
                        const int s = h ? s1 : bs, g = h ? g1 : ag;
                        const uint32_t a_tmem = tmem + a_base + g * Tr::kACols;
                        const uint32_t bx = smem_u32(bring + (size_t)s * b_bytes);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {            // 32 bytes of every row per MMA
                            const uint64_t db = smem_desc_sw128(bx + ks * 32);
                            const uint32_t acc = (uint32_t)(kb | h | ks);
                            if (kBf16) {
                                tc_mma_bf16_ts(d1, a_tmem + ks * 8, db, idesc_2n, acc);          // w [h_hi; h_lo]
                            } else {
                                tc_mma_tf32_ts(d1, a_tmem + ks * 8, db, idesc_2n, acc);          // w_hi [h_hi; h_lo]
                                tc_mma_tf32_ts(d2, a_tmem + 32 + ks * 8, db, idesc_n, acc);      // w_lo h_hi
                            }
                        }
                        tc_commit(bar_aempty(g));               // the A buffer and
                        tc_commit(bar_bempty(s));               // the stage's activations may be overwritten once these finish
                    }
                    if (kb + kb_step >= nkb) tc_commit(bar_dfull(set));
                }
                __syncwarp();
                // advance both rings by the k-blocks taken
                bs = two ? s1 + 1 : s1;
                bph = sph1;
                if (two && bs == n_bstages) { bs = 0; bph ^= 1; }
                ag = two ? g1 + 1 : g1;
                aph = gph1;
                if (two && ag == n_abufs) { ag = 0; aph ^= 1; }
            }
            if (!ok) break;
        }
    } else if (warp >= 4 && warp < 12) {
        // ------------------------------------------------------------------ converters
        const int cset = (warp - 4) >> 2;             // set 0 takes the even k-blocks of the stream, set 1 the odd
        const int quad = warp & 3;                    // TMEM lane quadrant this warp may access
        const int row = quad * 32 + lane;             // row of the tile = TMEM lane
        const uint32_t a_bufs = tmem + ((uint32_t)(quad * 32) << 16) + a_base;
        uint32_t it0 = 0;
        int model, tile;
        // partial sum of squares of this tile's rows (model 0 is x itself: not a candidate)
        auto store_norm = [&](const float (&n4)[4]) {
            if (model > 0) {
                float nrm = (n4[0] + n4[1]) + (n4[2] + n4[3]);
                const int o = tile * kRows + row;
                if (cset == 0 && a.offB >= 0 && o < a.out) {
                    const float bv = load_elem(static_cast<const T *>(a.V) + (int64_t)(model - 1) * a.ldv + a.offB + o);
                    nrm = fmaf(bv, bv, nrm);
                }
#pragma unroll
                for (int sft = 16; sft >= 1; sft >>= 1) nrm += __shfl_xor_sync(0xffffffffu, nrm, sft);
                if (lane == 0) {
                    a.normpart[(int64_t)(model - 1) * a.np_slots + a.np_base + (tile * 4 + quad) * 2 + cset] = nrm;
                    if (HEAD) __threadfence();
                }
            }
        };
        for (int li = 0; get_item(li, model, tile) && !*abortp; ++li, it0 += nkb) {
            float nrm4[4] = {0.f, 0.f, 0.f, 0.f};
            bool ok = true;
            for (int kb = (int)((cset - it0) & 1u); kb < nkb; kb += 2) {
                const uint32_t it = it0 + kb;
                const uint32_t sround = small_div(it, inv_stages), around = small_div(it, inv_abufs);
                const int s = (int)(it - sround * n_stages), g = (int)(it - around * n_abufs);
                if (!mbar_wait(bar_full(s), sround & 1, abortp)) { ok = false; break; }
                const uint8_t *src = ring + (size_t)s * stage_bytes + row * kRowBytes;
                uint4 xq[8], vq[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) xq[c] = *reinterpret_cast<const uint4 *>(src + ((c ^ (row & 7)) << 4));
                if (model > 0 && !LINEAR) {
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        vq[c] = *reinterpret_cast<const uint4 *>(src + kTileBytes + ((c ^ (row & 7)) << 4));
                } else {
#pragma unroll
                    for (int c = 0; c < 8; ++c) vq[c] = make_uint4(0u, 0u, 0u, 0u);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_empty(s));       // this set is done with the stage's weight tiles
                uint32_t wa[32], wb[32];                        // bf16: wa = packed pairs; fp32: wa = hi, wb = lo
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint32_t xw[4] = {xq[c].x, xq[c].y, xq[c].z, xq[c].w};
                    const uint32_t vw[4] = {vq[c].x, vq[c].y, vq[c].z, vq[c].w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (kBf16) {
                            const float x0 = __uint_as_float(xw[u] << 16), x1 = __uint_as_float(xw[u] & 0xffff0000u);
                            const float v0 = __uint_as_float(vw[u] << 16), v1 = __uint_as_float(vw[u] & 0xffff0000u);
                            nrm4[u] = fmaf(v0, v0, nrm4[u]);
                            nrm4[u] = fmaf(v1, v1, nrm4[u]);
                            const __nv_bfloat162 pk = __floats2bfloat162_rn(fmaf(-a.gamma, v0, x0), fmaf(-a.gamma, v1, x1));
                            wa[4 * c + u] = *reinterpret_cast<const uint32_t *>(&pk);
                        } else {
                            const float xv = __uint_as_float(xw[u]), vv = __uint_as_float(vw[u]);
                            nrm4[u] = LINEAR ? fmaf(xv, xv, nrm4[u]) : fmaf(vv, vv, nrm4[u]);   // LINEAR: the tile is v itself
                            const float w = LINEAR ? xv : fmaf(-a.gamma, vv, xv);
                            const float h = tf32_hi(w);
                            wa[4 * c + u] = __float_as_uint(h);
                            wb[4 * c + u] = __float_as_uint(w - h);
                        }
                    }
                }
                // HEAD: the norm partial must be in global memory before the epilogue group takes the
                // model's ticket, so it is written ahead of the set's last A buffer of the tile
                if (HEAD && kb + 2 >= nkb) store_norm(nrm4);
                if (!mbar_wait(bar_aempty(g), (around & 1) ^ 1, abortp)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_tmem = a_bufs + g * Tr::kACols;
                tc_st32(a_tmem, wa);
                if (!kBf16) tc_st32(a_tmem + 32, wb);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_afull(g));
            }
            if (!ok) break;
            if (!HEAD) store_norm(nrm4);          // HEAD: already written (every set has a k-block: K >= 2 k-blocks)
        }
    } else if (warp >= 12) {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        int model, tile;
        const int g = tid - (kLThreads - kEpiThreads);    // thread within the epilogue group
        const int cls_even = (a.head.classes + 1) & ~1;
        // HEAD: the group leaves the loop together (its named barrier needs all four warps)
        for (int li = 0; get_item(li, model, tile) && (HEAD || !*abortp); ++li) {
            const int set = li % n_sets;
            const uint32_t use = (uint32_t)(li / n_sets);
            const int o = tile * kRows + row;             // thread = output row o, column = sample j
            float bias = 0.f;
            if (!LINEAR && a.offB >= 0 && o < a.out) {    // asked for before the accumulator is awaited
                const float vb = model > 0 ? load_elem(static_cast<const T *>(a.V) + (int64_t)(model - 1) * a.ldv + a.offB + o) : 0.f;
                bias = candidate_param<T>(load_elem(static_cast<const T *>(a.xparams) + a.offB + o), vb, a.gamma);
            }
            // HEAD: column o of the last layer's weights for this model, and their share of ||v||^2
            float w3[kHeadMaxClasses];
            if (HEAD) {
                float nrm3 = 0.f;
                const T *x3 = static_cast<const T *>(a.xparams) + a.head.offW + o;
                const T *v3 = static_cast<const T *>(a.V) + (int64_t)(model > 0 ? model - 1 : 0) * a.ldv + a.head.offW + o;
#pragma unroll
                for (int cls = 0; cls < kHeadMaxClasses; ++cls) {
                    w3[cls] = 0.f;
                    if (cls < a.head.classes && o < a.out) {
                        const float vv = model > 0 ? load_elem(v3 + (int64_t)cls * a.out) : 0.f;
                        w3[cls] = candidate_param<T>(load_elem(x3 + (int64_t)cls * a.out), vv, a.gamma);
                        nrm3 = fmaf(vv, vv, nrm3);
                    }
                }
                if (model > 0) {
                    if (tile == 0 && quad == 0 && a.head.offB >= 0 && lane < a.head.classes) {
                        const float bv = load_elem(static_cast<const T *>(a.V) + (int64_t)(model - 1) * a.ldv + a.head.offB + lane);
                        nrm3 = fmaf(bv, bv, nrm3);
                    }
#pragma unroll
                    for (int sft = 16; sft >= 1; sft >>= 1) nrm3 += __shfl_xor_sync(0xffffffffu, nrm3, sft);
                    if (lane == 0) a.normpart[(int64_t)(model - 1) * a.np_slots + a.head.np_base + tile * 4 + quad] = nrm3;
                }
            }
            bool got = mbar_wait(bar_dfull(set), use & 1, abortp);
            if (HEAD) got = epi_all(got);
            if (!got) break;
            tc_fence_after();
            const uint32_t dset = tmem + lane_addr + set * acc_cols;
            for (int j0 = 0; j0 < a.n_pad; j0 += 16) {
                uint32_t t0[16], t1[16];
                float acc[16];
                tc_ld16(dset + j0, t0);                       // w(_hi) h_hi
                tc_ld16(dset + a.n_pad + j0, t1);             // w(_hi) h_lo
                tc_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) acc[j] = __uint_as_float(t1[j]);
                if (!kBf16) {
                    tc_ld16(dset + 2 * a.n_pad + j0, t1);     // w_lo h_hi
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) acc[j] += __uint_as_float(t1[j]);
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) acc[j] += __uint_as_float(t0[j]);
                if (j0 + 16 >= a.n_pad) {                     // everything is in registers: release the accumulator
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_dempty(set));
                }
                if (HEAD) {
                    // partial logits of this warp's 32 rows: lane l ends up with class cb + l / 16, sample j0 + l % 16
                    float zz[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        float z = acc[j] + bias;
                        if (a.relu) z = (z > 0.f || z != z) ? z : 0.f;
                        zz[j] = (j0 + j < a.n_r) ? z : 0.f;
                    }
                    float *zq_w = zq + (int64_t)quad * cls_even * a.n_pad;
#pragma unroll
                    for (int cb = 0; cb < kHeadMaxClasses; cb += 2) {
                        if (cb >= a.head.classes) break;
                        float pv[32];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            pv[j] = w3[cb] * zz[j];
                            pv[16 + j] = w3[cb + 1] * zz[j];
                        }
                        const float r = lane_transpose_sum32(pv, lane);
                        zq_w[(cb + (lane >> 4)) * a.n_pad + j0 + (lane & 15)] = r;
                    }
                } else if (o < a.out) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int jj = j0 + j;
                        float z = acc[j] + bias;
                        if (a.relu) z = (z > 0.f || z != z) ? z : 0.f;
                        if (jj >= a.n_r) z = 0.f;             // padded samples
                        if (a.Hout && jj < a.n_r) a.Hout[((int64_t)model * a.n_r + jj) * a.out + o] = z;
                        if (a.Hsplit) {
                            T *hs = static_cast<T *>(a.Hsplit) + (int64_t)model * 2 * a.n_pad * a.out + o;
                            if (kBf16) {
                                const __nv_bfloat16 hi = __float2bfloat16_rn(z);
                                const __nv_bfloat16 lo = __float2bfloat16_rn(z - __bfloat162float(hi));
                                reinterpret_cast<__nv_bfloat16 *>(hs)[(int64_t)jj * a.out] = hi;
                                reinterpret_cast<__nv_bfloat16 *>(hs)[(int64_t)(a.n_pad + jj) * a.out] = lo;
                            } else {
                                const float hi = tf32_hi(z);
                                reinterpret_cast<float *>(hs)[(int64_t)jj * a.out] = hi;
                                reinterpret_cast<float *>(hs)[(int64_t)(a.n_pad + jj) * a.out] = z - hi;
                            }
                        }
                    }
                }
            }
            if (HEAD) {
                // the four warps' partial logits added in warp order: one set per tile in global memory
                epi_sync();
                const int n_out = cls_even * a.n_pad;
                float *zp = a.head.zpart + ((int64_t)model * a.tiles + tile) * kHeadMaxClasses * a.n_pad;
                for (int t = g; t < n_out; t += kEpiThreads)
                    zp[t] = (zq[t] + zq[n_out + t]) + (zq[2 * n_out + t] + zq[3 * n_out + t]);
                __threadfence();
                epi_sync();
                if (g == 0) {
                    const unsigned tk = atomicAdd(a.head.model_ticket + model, 1u);
                    head_last = tk == (unsigned)a.tiles - 1;
                    if (head_last) a.head.model_ticket[model] = 0;       // ready for the next launch
                }
                epi_sync();
                if (head_last) {                       // uniform in the group; rewritten only after the barriers below
                    __threadfence();
                    head_finish_model<T>(a, model, zq, g);
                    if (g == 0) {
                        const unsigned tk = atomicAdd(a.head.tail.ticket, 1u);
                        if (tk == (unsigned)a.m) {
                            *a.head.tail.ticket = 0;
                            head_final = 1;
                        }
                    }
                }
                epi_sync();                            // zq and head_last may be reused
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1 && abort_flag) drain_mmas(smem_u32(&drain_bar));
    if (tid == 0 && abort_flag) {
        // bulk copies still in flight (only after an aborted run) must land before the block exits
        for (int s = 0; s < kLMaxStages + kLMaxBStages; ++s)
            if (issued[s] > 0) {
                const uint32_t bar = s < kLMaxStages ? bar_full(s) : bar_bfull(s - kLMaxStages);
                for (uint32_t i = 0; i < kSpinLimit; ++i) {
                    if (mbar_try_wait(bar, (uint32_t)(issued[s] - 1) & 1)) break;
                    __nanosleep(64);
                }
            }
        atomicCAS(a.status, 0, wait_code(2, abort_flag, smem_u32(bars)));   // the first block to give up is kept
    }
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kLTmemCols) : "memory");
    }
    if (HEAD && head_final) {               // block-uniform: written before the teardown's barrier
        __threadfence();
        finalize_and_select(a.head.tail);
    }
}

// Activations [models][n_r][K] fp32 -> the two-term stacked operand [models][2 n_pad][K]:
// rows 0..n_pad-1 the leading term, rows n_pad.. the remainder, zero rows for the padded samples.
template <typename T>
__global__ void __launch_bounds__(256) split_acts_kernel(const float *H, int models, int n_r, int n_pad, int K, T *out) {
    pdl_wait();
    pdl_launch_dependents();
    const int64_t total = (int64_t)models * n_pad * K;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int k = (int)(t % K);
        const int64_t cj = t / K;
        const int j = (int)(cj % n_pad);
        const int64_t c = cj / n_pad;
        const float h = j < n_r ? __ldg(H + (c * n_r + j) * K + k) : 0.f;
        T *dst = out + (c * 2 * n_pad + j) * (int64_t)K + k;
        if (is_bf16<T>::value) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(h);
            reinterpret_cast<__nv_bfloat16 *>(dst)[0] = hi;
            reinterpret_cast<__nv_bfloat16 *>(dst)[(int64_t)n_pad * K] = __float2bfloat16_rn(h - __bfloat162float(hi));
        } else {
            const float hi = tf32_hi(h);
            reinterpret_cast<float *>(dst)[0] = hi;
            reinterpret_cast<float *>(dst)[(int64_t)n_pad * K] = h - hi;
        }
    }
}

template <typename T>
cudaError_t encode_maps(Context &c, const LayerTcLaunch &l, CUtensorMap *map_x, CUtensorMap *map_v, CUtensorMap *map_h) {
    using Tr = TcTraits<T>;
    if (!encode_tiled_fn()) return cudaErrorNotSupported;
    const cuuint64_t es = sizeof(T);
    {
        cuuint64_t dims[3] = {(cuuint64_t)l.K, (cuuint64_t)l.out, 1};
        cuuint64_t strides[2] = {(cuuint64_t)l.K * es, (cuuint64_t)l.K * es * (cuuint64_t)l.out};
        cuuint32_t box[3] = {(cuuint32_t)Tr::kBlockK, kRows, 1};
        if (encode_cached(c, map_x, Tr::kMapType, static_cast<const T *>(l.x) + l.offW, dims, strides, box,
                          CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)l.K, (cuuint64_t)l.out, (cuuint64_t)l.m};
        cuuint64_t strides[2] = {(cuuint64_t)l.K * es, (cuuint64_t)l.ldv * es};
        cuuint32_t box[3] = {(cuuint32_t)Tr::kBlockK, kRows, 1};
        if (encode_cached(c, map_v, Tr::kMapType, static_cast<const T *>(l.V) + l.offW, dims, strides, box,
                          CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        const cuuint64_t rows = 2 * (cuuint64_t)l.n_pad, models = l.h_shared ? 1 : (cuuint64_t)l.m + 1;
        cuuint64_t dims[3] = {(cuuint64_t)l.K, rows, models};
        cuuint64_t strides[2] = {(cuuint64_t)l.K * es, (cuuint64_t)l.K * es * rows};
        cuuint32_t box[3] = {(cuuint32_t)Tr::kBlockK, (cuuint32_t)rows, 1};
        if (encode_cached(c, map_h, Tr::kMapType, l.Hsplit_in, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    return cudaSuccess;
}

template <typename T, bool LINEAR, bool HEAD>
cudaError_t launch_typed(Context &c, const LayerTcLaunch &l, cudaStream_t s) {
    using Tr = TcTraits<T>;
    CUtensorMap map_x, map_v, map_h;
    cudaError_t e = encode_maps<T>(c, l, &map_x, &map_v, &map_h);
    if (e != cudaSuccess) return e;
    LayerTcArgs a;
    a.xparams = l.x;
    a.V = l.V;
    a.ldv = l.ldv;
    a.offB = l.offB;
    a.gamma = l.gamma;
    a.K = l.K;
    a.out = l.out;
    a.n_r = l.n_r;
    a.n_pad = l.n_pad;
    a.m = l.m;
    a.tiles = (l.out + kRows - 1) / kRows;
    a.h_shared = l.h_shared;
    const int stage_bytes = (LINEAR ? 1 : 2) * kTileBytes, b_bytes = 2 * l.n_pad * kRowBytes;
    // HEAD: the ranking holds 9 KB of static shared memory, and the epilogue warps' partial logits
    // sit behind the ring
    const int zq_bytes = HEAD ? 4 * ((l.head->classes + 1) & ~1) * l.n_pad * 4 : 0;
    const int budget = HEAD ? kLSmemBudget - 10 * 1024 : kLSmemBudget;
    // the activation ring gets kBStages stages, the weight ring (whose tiles come from HBM) the rest
    a.b_stages = layer_tc_b_stages(l.n_pad);
    a.stages = (budget - 1024 - zq_bytes - a.b_stages * b_bytes) / stage_bytes;
    if (a.stages > kLMaxStages) a.stages = kLMaxStages;
    if (a.stages < 2) return cudaErrorInvalidConfiguration;
    const int acc_cols = Tr::kAccPerPad * l.n_pad;
    a.n_sets = 2 * acc_cols + 2 * Tr::kACols <= kLTmemCols ? 2 : 1;
    a.n_abufs = (kLTmemCols - a.n_sets * acc_cols) / Tr::kACols;
    if (a.n_abufs > kLMaxABufs) a.n_abufs = kLMaxABufs;
    a.Hout = l.Hout;
    a.Hsplit = l.Hsplit_out;
    a.relu = LINEAR ? 0 : l.relu;          // LINEAR: raw products, the combine kernel activates
    a.normpart = c.normpart;
    a.np_slots = c.np_slots;
    a.np_base = l.np_base;
    a.status = c.dev_status;
    a.spin_limit = c.spin_limit;
    if (HEAD) a.head = *l.head; else a.head = HeadFuse{};
    static PerDeviceOnce attr_set;      // per instantiation and device
    if (attr_set.need(c.device)) {
        e = cudaFuncSetAttribute(layer_tc_kernel<T, LINEAR, HEAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, budget);
        if (e != cudaSuccess) return e;
        attr_set.mark(c.device);
    }
    const int items = (l.m + 1) * a.tiles;
    const int sms = c.sm_count > 0 ? c.sm_count : 148;
    // equal shares: the fewest blocks that give the same number of rounds as one block per SM
    const int rounds = (items + sms - 1) / sms;
    const int blocks = (items + rounds - 1) / rounds;
    return launch_chained(layer_tc_kernel<T, LINEAR, HEAD>, dim3(blocks), dim3(kLThreads), (size_t)a.stages * stage_bytes + (size_t)a.b_stages * b_bytes + 1024 + zq_bytes, s,
                          chain_launches(c), map_x, map_v, map_h, a);
}

}  // namespace

// Shapes the kernel serves: rows of 16-byte multiples that a TMA box can step through, up to 128
// samples (N = 2 n_pad <= 256), at least two ring stages and two A buffers.
bool layer_tc_usable(zeno_dtype dtype, int K, int out, int n_r) {
    const int per16 = dtype == ZENO_BF16 ? 8 : 4;
    if (K % per16 != 0 || K < 64 || out < 32 || n_r < 1 || n_r > 128) return false;
    const int n_pad = layer_tc_n_pad(n_r);
    // two stages of the weight ring beside the activation ring, in the smallest budget any mode leaves
    const int head_room = 10 * 1024 + 4 * kHeadMaxClasses * n_pad * 4;
    if (kLSmemBudget - head_room - 1024 - layer_tc_b_stages(n_pad) * 2 * n_pad * kRowBytes < 2 * 2 * kTileBytes) return false;
    const int acc = (dtype == ZENO_BF16 ? 2 : 3) * n_pad, acols = dtype == ZENO_BF16 ? 32 : 64;
    return (kLTmemCols - acc) / acols >= 2;
}

int layer_tc_n_pad(int n_r) { return (n_r + 15) / 16 * 16; }

// one slot per (tile, warp of a converter set, converter set)
int layer_tc_norm_slots(int out) { return (out + kRows - 1) / kRows * 8; }

// HEAD mode: partial logits and the last layer's norm partials, one slot per (tile, epilogue warp)
int layer_tc_head_slots(int out) { return (out + kRows - 1) / kRows * 4; }

cudaError_t launch_layer_tc(Context &c, const LayerTcLaunch &l, cudaStream_t s, int *launches) {
    ++*launches;
    const bool head = l.head != nullptr && l.head->classes > 0 && !l.linear;
    profile_mark(c, head ? "layer_tc_head" : "layer_tc", s);
    if (c.desc.param_dtype == ZENO_BF16)
        return head ? launch_typed<__nv_bfloat16, false, true>(c, l, s) : launch_typed<__nv_bfloat16, false, false>(c, l, s);
    if (l.linear) return launch_typed<float, true, false>(c, l, s);
    return head ? launch_typed<float, false, true>(c, l, s) : launch_typed<float, false, false>(c, l, s);
}

cudaError_t launch_split_acts(Context &c, const float *H, int models, int n_r, int K, void *out, cudaStream_t s,
                              int *launches) {
    ++*launches;
    profile_mark(c, "split_acts", s);
    const int n_pad = layer_tc_n_pad(n_r);
    const int64_t total = (int64_t)models * n_pad * K;
    int blocks = (int)((total + 255) / 256);
    const int cap = (c.sm_count > 0 ? c.sm_count : 148) * 8;
    if (blocks > cap) blocks = cap;
    if (c.desc.param_dtype == ZENO_BF16)
        return launch_chained(split_acts_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, s, chain_launches(c), H,
                              models, n_r, n_pad, K, static_cast<__nv_bfloat16 *>(out));
    return launch_chained(split_acts_kernel<float>, dim3(blocks), dim3(256), 0, s, chain_launches(c), H, models, n_r,
                          n_pad, K, static_cast<float *>(out));
}

}  // namespace zeno
