// First dense layer of all m+1 models on the 5th-generation tensor cores (fp32 storage).
//
// The first layer's input activations are the server batch itself, shared by every candidate,
// and the layer is linear in its weights: X (W - gamma V_i)^T = X W^T - gamma X V_i^T.  So the
// layer for all models is ONE skinny GEMM of the shared batch X [n_r x K] against the stacked
// rows [W; V_1; ..; V_m] ([(m+1) out] x K), streamed from HBM exactly once, plus the row norms
// of V taken from the same registers (the rho ||v||^2 term of Definition 2).
//
// fp32 accuracy on tf32 tensor cores: both operands are split, a = a_hi + a_lo with a_hi the
// value rounded to tf32, and the product is accumulated as a_hi b_hi + a_lo b_hi + a_hi b_lo
// (the dropped a_lo b_lo term is below 2^-22 relative).  X_hi and X_lo are stacked along N: one
// MMA reads a_hi once and yields a_hi x_hi and a_hi x_lo side by side; a second one adds a_lo x_hi.
//
// The tensor core adds into its fp32 accumulator with truncation, so a long accumulation chain
// drifts; the two small products go to an accumulator of their own (their truncation error is
// 2^-11 smaller) and the k-range of a block bounds the length of the chain of large ones.
//
// Per block (one SM): a k-range of the input index, whose X_hi / X_lo slices stay resident in
// shared memory in the 128-byte-swizzled K-major layout the MMA reads, and a list of 128-row
// tiles of the stacked matrix.  The block runs TWO independent pipelines side by side, each on
// its own row tiles, with its own TMA ring, converter warps, MMA issuer, TMEM operand buffers and
// accumulator, so that one pipeline's waits are covered by the other's work.  Warp roles
// (p = pipeline 0 / 1):
//   warp p        TMA producer: 128 rows x 32 floats boxes of V (or x) into pipeline p's ring
//   warp 2+p      MMA issuer (tcgen05.mma, A operand from TMEM, B from shared); warp 2 owns TMEM
//   warps 4-7 / 8-11   converters of pipeline 0 / 1: thread t owns row t of the tile; reads its
//                 128 bytes from the stage, accumulates v^2, splits into hi/lo and stores both
//                 to TMEM (tcgen05.st) where the MMA picks them up
//   warps 12-15   epilogue: drain finished accumulators (tcgen05.ld) into the split-K partial
//                 output while both pipelines keep going; stream_combine_kernel adds the partials
//                 in k-range order.
// Producer and issuer warps stay converged and issue from one elected lane.  Every mbarrier wait
// is bounded; a wait that gives up raises a status word and the block leaves through the common
// teardown (pending bulk copies awaited, TMEM freed).
#include <cuda.h>

#include "zeno_internal.h"
#include "zeno_tc.cuh"

namespace zeno {

namespace {

constexpr int kTileRows = 128;          // rows of the stacked matrix per tile = TMEM lanes
constexpr int kBlockK = 32;             // floats per k-block = one 128-byte swizzle row
constexpr int kPipes = 2;               // independent pipelines per block
constexpr int kMaxStages = 6;           // TMA ring depth per pipeline
constexpr int kStageBytes = kTileRows * kBlockK * 4;
constexpr int kMaxABufs = 2;            // TMEM A buffers per pipeline (hi 32 + lo 32 columns each)
constexpr int kThreads = 32 * 16;
constexpr int kTmemCols = 512;          // one accumulator set per pipeline, then the A buffers (see TmemLayout)
constexpr int kSmemBudget = 226 * 1024;      // dynamic; the static barriers and flags fit below the 227 KB limit

// TMEM columns.  Pipeline p's accumulator set holds D1 = a_hi [x_hi; x_lo]^T (2 n_pad columns)
// and D2 = a_lo x_hi^T (n_pad columns); the A buffers (64 columns each) follow the two sets,
// n_abufs per pipeline.
struct TmemLayout {
    int set_stride, d2_off, a_base, n_abufs;
    __host__ __device__ explicit TmemLayout(int n_pad) {
        set_stride = n_pad <= 32 ? 128 : 192;
        d2_off = n_pad <= 32 ? 64 : 128;
        a_base = kPipes * set_stride;
        n_abufs = (kTmemCols - a_base) / (64 * kPipes);
    }
};

struct StreamArgs {
    const float *X;        // [n_r x K] the server batch
    const float *V;        // for the bias entries' v^2
    int64_t ldv;
    int64_t offB;          // element offset of this layer's bias inside a row of V, -1 if none
    float *part;           // [R][m+1][n_r][out] split-K partial products
    float *normpart;       // [m][np_slots]
    int np_slots, np_base;
    int K, out, n_r, n_pad, m;
    int KR;                // floats of K per k-range (multiple of 32)
    int tiles_per_model;   // ceil(out / 128)
    int stages;            // depth of each pipeline's TMA ring (<= kMaxStages)
    int *status;           // device status word (raised on a wait that gave up)
    uint32_t spin_limit;   // polls a bounded wait may take
};

// B = the shared batch, A = raw rows of [x; V] (the layer is linear in its weights, the combine
// kernel forms X W^T - gamma X V^T); a block's items are row tiles blockIdx.y, blockIdx.y +
// gridDim.y, .. of the stacked matrix.
__global__ void __launch_bounds__(kThreads, 1)
stream_tf32x3_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_v,
                     StreamArgs a) {
    constexpr int kStage = kStageBytes;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // per pipeline: full[kMaxStages], empty[kMaxStages], a_full[kMaxABufs], a_empty[kMaxABufs], d_full, d_empty
    constexpr int kBarsPerPipe = 2 * kMaxStages + 2 * kMaxABufs + 2;
    __shared__ __align__(8) uint64_t bars[kPipes * kBarsPerPipe];
    __shared__ __align__(8) uint64_t drain_bar[kPipes];   // teardown after an abort: each issuer's last commit
    __shared__ __align__(8) uint64_t never_bar;           // nothing arrives here (test hook, see wait_for_nothing)
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_state[kAbortWords];
    int &abort_flag = abort_state[0];
    __shared__ int issued[kPipes][kMaxStages];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // the descriptors are on their way while the barriers and TMEM are set up
    if (tid == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
    if (tid == 32) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    const int r = blockIdx.x;                         // k-range
    const int k0 = r * a.KR;
    const int k_len = min(a.KR, a.K - k0);
    const int nkb = (k_len + kBlockK - 1) / kBlockK;   // k-blocks in this range
    const int n_items_total = (a.m + 1) * a.tiles_per_model;
    // item li of this block -> (model, tile); false when the block has no such item
    auto get_item = [&](int li, int &model, int &tile) {
        const int item = blockIdx.y + li * gridDim.y;
        model = item / a.tiles_per_model;
        tile = item % a.tiles_per_model;
        return item < n_items_total;
    };
    const float *Xsrc = a.X;
    const int n_stages = a.stages;
    constexpr int pipes = kPipes;

    // shared memory carve-up (dynamic part is 1024-byte aligned)
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int nkb_max = a.KR / kBlockK;
    const uint32_t xkb_bytes = 2u * a.n_pad * 128;     // one k-block of [X_hi; X_lo]: a multiple of 1024
    uint8_t *xs = base;
    uint8_t *stage_base = base + (uint32_t)nkb_max * xkb_bytes;   // pipeline p's ring at p * n_stages * kStage
    const TmemLayout tl(a.n_pad);
    const int n_abufs = tl.n_abufs;
    const float inv_stages = 1.0f / (float)n_stages, inv_abufs = 1.0f / (float)n_abufs;

    auto bar_full = [&](int p, int s) { return smem_u32(&bars[p * kBarsPerPipe + s]); };
    auto bar_empty = [&](int p, int s) { return smem_u32(&bars[p * kBarsPerPipe + kMaxStages + s]); };
    auto bar_afull = [&](int p, int b) { return smem_u32(&bars[p * kBarsPerPipe + 2 * kMaxStages + b]); };
    auto bar_aempty = [&](int p, int b) { return smem_u32(&bars[p * kBarsPerPipe + 2 * kMaxStages + kMaxABufs + b]); };
    auto bar_dfull = [&](int p) { return smem_u32(&bars[p * kBarsPerPipe + 2 * kMaxStages + 2 * kMaxABufs]); };
    auto bar_dempty = [&](int p) { return smem_u32(&bars[p * kBarsPerPipe + 2 * kMaxStages + 2 * kMaxABufs + 1]); };

    if (tid == 0) {
        abort_flag = 0;
        abort_state[1] = (int)a.spin_limit;
        for (int p = 0; p < kPipes; ++p) {
            for (int s = 0; s < kMaxStages; ++s) {
                mbar_init(bar_full(p, s), 1);
                mbar_init(bar_empty(p, s), 4);
                issued[p][s] = 0;
            }
            for (int b = 0; b < kMaxABufs; ++b) {
                mbar_init(bar_afull(p, b), 4);
                mbar_init(bar_aempty(p, b), 1);
            }
            mbar_init(bar_dfull(p), 1);
            mbar_init(bar_dempty(p), 4);
            mbar_init(smem_u32(&drain_bar[p]), 1);
        }
        mbar_init(smem_u32(&never_bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {   // TMEM allocation by one full warp
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();                                   // barriers and the TMEM base are visible
    tc_fence_after();
    pdl_wait();                                        // on-chip set-up done; global memory from here on
    pdl_launch_dependents();
    const uint32_t tmem = tmem_base_slot;
    volatile int *abortp = &abort_flag;

    // [X_hi; X_lo] of this k-range in the swizzled K-major layout: k-block kb at kb * xkb_bytes,
    // row j of X_hi at j * 128, of X_lo at (n_pad + j) * 128, 16-byte chunk c at c ^ (row & 7).
    // Everyone but the producer warps fills it while the first tiles are in flight.
    if (warp >= kPipes) {
        constexpr int kFillers = kThreads - 32 * kPipes;
        const int fid = tid - 32 * kPipes;
        const int n_chunks = nkb_max * a.n_pad * 8;
        const float inv_n_pad = 1.0f / (float)a.n_pad;   // row index / n_pad without an integer division
        // 16-byte chunk t of the slice: k-block, row and column chunk; where it lives; whether it exists
        auto chunk = [&](int t, uint32_t &off, const float *&src) {
            const int c = t & 7, kb = __float2int_rd(((t >> 3) + 0.5f) * inv_n_pad), j = (t >> 3) - kb * a.n_pad;
            const int k = k0 + kb * kBlockK + c * 4;
            off = (uint32_t)kb * xkb_bytes + j * 128 + ((c ^ (j & 7)) << 4);
            src = Xsrc + (int64_t)j * a.K + k;
            return j < a.n_r && k < a.K && kb < nkb;
        };
        // asynchronous copies of the raw values (zero fill where there is nothing), all in flight at
        // once; then every thread splits the chunks it copied, in place
        constexpr int kIlp = 4;                          // independent chunks per loop trip
        for (int t0 = fid; t0 < n_chunks; t0 += kIlp * kFillers) {
#pragma unroll
            for (int u = 0; u < kIlp; ++u) {
                const int t = t0 + u * kFillers;
                uint32_t off;
                const float *src;
                const bool live = chunk(t, off, src);
                if (t < n_chunks)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;"
                                 ::"r"(smem_u32(xs + off)), "l"(live ? src : Xsrc), "r"(live ? 16 : 0) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
        for (int t0 = fid; t0 < n_chunks; t0 += kIlp * kFillers) {
            uint32_t off[kIlp];
            float4 v[kIlp];
#pragma unroll
            for (int u = 0; u < kIlp; ++u) {
                const float *src;
                chunk(min(t0 + u * kFillers, n_chunks - 1), off[u], src);
                v[u] = *reinterpret_cast<const float4 *>(xs + off[u]);
            }
#pragma unroll
            for (int u = 0; u < kIlp; ++u) {
                if (t0 + u * kFillers >= n_chunks) break;
                const float4 hi = make_float4(tf32_hi(v[u].x), tf32_hi(v[u].y), tf32_hi(v[u].z), tf32_hi(v[u].w));
                const float4 lo = make_float4(v[u].x - hi.x, v[u].y - hi.y, v[u].z - hi.z, v[u].w - hi.w);
                *reinterpret_cast<float4 *>(xs + off[u]) = hi;
                *reinterpret_cast<float4 *>(xs + off[u] + a.n_pad * 128) = lo;   // n_pad % 8 == 0: same swizzle phase
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
        asm volatile("bar.sync 1, %0;" ::"n"(kFillers) : "memory");      // named barrier of the filling warps
    }

    // Item li of this block (li = 0, 1, ..) is row tile blockIdx.y + li * gridDim.y of the stacked
    // matrix; pipeline p takes the items with li % kPipes == p.
    if (warp < kPipes) {
        // ------------------------------------------------------------------ TMA producers
        // The warp stays converged (every lane takes the waits); one elected lane arms the barrier
        // and issues the stage's copies, at ONE issue site.
        const int p = warp;
        if (p == 0) wait_for_nothing(smem_u32(&never_bar), abortp);
        uint8_t *ring = stage_base + (size_t)p * n_stages * kStage;
        int s = 0;                                 // stage, and how often the ring has wrapped
        uint32_t round = 0;
        int model, tile;
        for (int li = p;; li += pipes) {
            if (!__all_sync(0xffffffffu, get_item(li, model, tile) && !*abortp)) break;
            // x is a one-model stack, so both operands take the same path
            const CUtensorMap *map = model > 0 ? &map_v : &map_x;
            const int c2 = max(model - 1, 0);
            bool ok = true;
            for (int kb = 0; kb < nkb; ++kb) {
                ok = __all_sync(0xffffffffu, mbar_wait(bar_empty(p, s), (round & 1) ^ 1, abortp));
                if (!ok) break;
                if (elect_one()) {
                    mbar_expect_tx(bar_full(p, s), kStageBytes);
                    issued[p][s] = (int)round + 1;
                    tma_load_3d(smem_u32(ring + s * kStage), map, k0 + kb * kBlockK, tile * kTileRows, c2,
                                bar_full(p, s));
                }
                __syncwarp();
                if (++s == n_stages) {
                    s = 0;
                    ++round;
                }
            }
            if (!ok) break;
        }
    } else if (warp < 2 * kPipes) {
        // ------------------------------------------------------------------ MMA issuers
        // The warp stays converged; one elected lane issues the MMAs and their commits.
        const int p = warp - kPipes;
        // instruction descriptors: D fp32, A and B tf32, both K-major, M = 128, N = n_pad / 2 n_pad
        const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(a.n_pad >> 3) << 17) |
                               ((uint32_t)(kTileRows >> 4) << 24);
        const uint32_t idesc2 = (idesc & ~(0x3fu << 17)) | ((uint32_t)((2 * a.n_pad) >> 3) << 17);
        const uint32_t d1 = tmem + p * tl.set_stride, d2 = d1 + tl.d2_off;
        uint32_t it = 0, q = 0;
        int model, tile;
        for (int li = p;; li += pipes, ++q) {
            if (!__all_sync(0xffffffffu, get_item(li, model, tile) && !*abortp)) break;
            if (!__all_sync(0xffffffffu, mbar_wait(bar_dempty(p), (q & 1) ^ 1, abortp))) break;   // accumulator drained
            tc_fence_after();
            bool ok = true;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const uint32_t around = small_div(it, inv_abufs);          // uses of this A buffer so far
                const int ab = (int)(it - around * n_abufs);
                ok = __all_sync(0xffffffffu, mbar_wait(bar_afull(p, ab), around & 1, abortp));
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
                    const uint32_t a_tmem = tmem + tl.a_base + (p * n_abufs + ab) * 64;
                    const uint32_t bx = smem_u32(xs) + (uint32_t)kb * xkb_bytes;
#pragma unroll
                    for (int ks = 0; ks < kBlockK / 8; ++ks) {
                        const uint64_t db = smem_desc_sw128(bx + ks * 32);
                        tc_mma_tf32_ts(d1, a_tmem + ks * 8, db, idesc2, (uint32_t)(kb | ks));        // a_hi [x_hi; x_lo]
                        tc_mma_tf32_ts(d2, a_tmem + 32 + ks * 8, db, idesc, (uint32_t)(kb | ks));    // a_lo x_hi
                    }
                    tc_commit(bar_aempty(p, ab));          // the A buffer may be overwritten once these finish
                    if (kb + 1 == nkb) tc_commit(bar_dfull(p));   // accumulators complete
                }
                __syncwarp();
            }
            if (!ok) break;
        }
    } else if (warp < 2 * kPipes + 4 * kPipes) {
        // ------------------------------------------------------------------ converters
        const int p = (warp - 2 * kPipes) >> 2;
        const int quad = warp & 3;                    // TMEM lane quadrant this warp may access
        const int row = quad * 32 + lane;             // row of the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const uint8_t *ring = stage_base + (size_t)p * n_stages * kStage;
        const uint32_t a_bufs = tmem + lane_addr + tl.a_base + p * n_abufs * 64;
        uint32_t it = 0;
        int model, tile;
        for (int li = p; get_item(li, model, tile) && !*abortp; li += pipes) {
            float nrm4[4] = {0.f, 0.f, 0.f, 0.f};
            bool ok = true;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const uint32_t sround = small_div(it, inv_stages);
                const int s = (int)(it - sround * n_stages);
                if (!mbar_wait(bar_full(p, s), sround & 1, abortp)) { ok = false; break; }
                const uint8_t *src = ring + s * kStage + row * 128;
                float4 v[8];
                uint32_t hi[32], lo[32];
#pragma unroll
                for (int c = 0; c < 8; ++c) v[c] = *reinterpret_cast<const float4 *>(src + ((c ^ (row & 7)) << 4));
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_empty(p, s));    // the stage may be refilled
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const float e[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        nrm4[u] = fmaf(e[u], e[u], nrm4[u]);
                        const float h = tf32_hi(e[u]);
                        hi[4 * c + u] = __float_as_uint(h);
                        lo[4 * c + u] = __float_as_uint(e[u] - h);
                    }
                }
                const uint32_t around = small_div(it, inv_abufs);
                const int ab = (int)(it - around * n_abufs);
                if (!mbar_wait(bar_aempty(p, ab), (around & 1) ^ 1, abortp)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_tmem = a_bufs + ab * 64;
                tc_st32(a_tmem, hi);                  // 32 columns of a_hi, then 32 of a_lo
                tc_st32(a_tmem + 32, lo);
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_afull(p, ab));
            }
            if (!ok) break;

            // partial sum of squares of this tile's rows (model 0 is x itself: not a candidate)
            if (model > 0) {
                float nrm = (nrm4[0] + nrm4[1]) + (nrm4[2] + nrm4[3]);
                const int o = tile * kTileRows + row;
                if (r == 0 && a.offB >= 0 && o < a.out) {
                    const float bv = __ldg(a.V + (int64_t)(model - 1) * a.ldv + a.offB + o);
                    nrm = fmaf(bv, bv, nrm);
                }
#pragma unroll
                for (int sft = 16; sft >= 1; sft >>= 1) nrm += __shfl_xor_sync(0xffffffffu, nrm, sft);
                if (lane == 0)
                    a.normpart[(int64_t)(model - 1) * a.np_slots + a.np_base +
                               (r * a.tiles_per_model + tile) * 4 + quad] = nrm;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        int model, tile;
        for (uint32_t li = 0; get_item((int)li, model, tile) && !*abortp; ++li) {
            const int p = li % pipes;
            const uint32_t q = li / pipes;                // how many accumulators pipeline p has finished before
            // thread = output row o, column = sample j
            const int o = tile * kTileRows + row;
            if (!mbar_wait(bar_dfull(p), q & 1, abortp)) break;
            tc_fence_after();
            float *dst = a.part + (((int64_t)r * (a.m + 1) + model) * a.n_r) * a.out + o;
            const uint32_t dset = tmem + lane_addr + p * tl.set_stride;
            for (int j0 = 0; j0 < a.n_pad; j0 += 16) {
                uint32_t big[16], s1[16], s2[16];
                tc_ld16(dset + j0, big);                       // a_hi x_hi
                tc_ld16(dset + a.n_pad + j0, s1);              // a_hi x_lo
                tc_ld16(dset + tl.d2_off + j0, s2);            // a_lo x_hi
                tc_wait_ld();
                if (j0 + 16 >= a.n_pad) {                      // everything is in registers: release the accumulator
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_dempty(p));
                }
                if (o < a.out) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (j0 + j < a.n_r)
                            dst[(int64_t)(j0 + j) * a.out] =
                                __uint_as_float(big[j]) + (__uint_as_float(s1[j]) + __uint_as_float(s2[j]));
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (abort_flag && warp >= kPipes && warp < 2 * kPipes) drain_mmas(smem_u32(&drain_bar[warp - kPipes]));
    if (tid == 0) {
        // bulk copies still in flight (only after an aborted run) must land before the block exits
        if (abort_flag) {
            for (int p = 0; p < kPipes; ++p)
                for (int s = 0; s < n_stages; ++s)
                    if (issued[p][s] > 0) {
                        for (uint32_t i = 0; i < kSpinLimit; ++i) {
                            if (mbar_try_wait(bar_full(p, s), (uint32_t)(issued[p][s] - 1) & 1)) break;
                            __nanosleep(64);
                        }
                    }
            atomicCAS(a.status, 0, wait_code(1, abort_flag, smem_u32(bars)));   // the first block to give up is kept
        }
    }
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// Split-K reduction and activation after a first layer whose products were taken against raw rows:
//   z_0 = sum_r P[r][0] + b(x),   z_c = z_0 - gamma (sum_r P[r][c] + b(v_c)),   h = ReLU(z)
// Block row blockIdx.y = model c; one thread per (sample, four outputs).  The partials are added in
// k-range order, four k-ranges' loads in flight at a time (few registers: several blocks per SM hide
// the latency instead).
// H: plain activations [m+1][n_r][out]; Hsplit: the same values as the two-term stacked operand
// [m+1][2 n_pad][out] of a following tensor-core layer (tf32 value, then remainder; zero rows for the
// padded samples).  Either may be NULL.
template <bool VEC4>
__global__ void __launch_bounds__(256) stream_combine_kernel(const float *part, int R, int m, int n_r, int out,
                                                             const float *x, const float *V, int64_t ldv,
                                                             int64_t offB, float gamma, int relu,
                                                             float *H, float *Hsplit, int n_pad) {
    constexpr int E = VEC4 ? 4 : 1;
    pdl_wait();
    pdl_launch_dependents();
    const int og = (out + E - 1) / E;                       // output groups per row
    const int n_rows = Hsplit ? n_pad : n_r;
    const int c = blockIdx.y;
    const int64_t per_r = (int64_t)(m + 1) * n_r * out;
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < n_rows * og; t += gridDim.x * blockDim.x) {
        const int j = t / og, o = (t - j * og) * E;
        float *hs = Hsplit ? Hsplit + ((int64_t)c * 2 * n_pad + j) * out + o : nullptr;
        if (j >= n_r) {                                          // padded sample of the stacked operand
            if (VEC4) {
                *reinterpret_cast<float4 *>(hs) = make_float4(0.f, 0.f, 0.f, 0.f);
                *reinterpret_cast<float4 *>(hs + (int64_t)n_pad * out) = make_float4(0.f, 0.f, 0.f, 0.f);
            } else {
                hs[0] = hs[(int64_t)n_pad * out] = 0.f;
            }
            continue;
        }
        const int64_t ic = ((int64_t)c * n_r + j) * out + o;
        const int64_t i0 = (int64_t)j * out + o;                 // the same entry of model 0
        const bool two = c > 0;                                  // a candidate: a second set of partials to add
        float z0[E], pc[E], xb[E], vb[E];
#pragma unroll
        for (int e = 0; e < E; ++e) {
            z0[e] = pc[e] = 0.f;
            // the bias entries come from HBM: ask for them before the partials, not after
            const bool ok = offB >= 0 && o + e < out;
            xb[e] = ok ? __ldg(x + offB + o + e) : 0.f;
            vb[e] = ok && two ? __ldg(V + (int64_t)(c - 1) * ldv + offB + o + e) : 0.f;
        }
        for (int r0 = 0; r0 < R; r0 += 4) {
            if (VEC4) {
                float4 a4[4], b4[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const bool ok = r0 + u < R;
                    a4[u] = ok ? __ldcg(reinterpret_cast<const float4 *>(part + (r0 + u) * per_r + i0))
                               : make_float4(0.f, 0.f, 0.f, 0.f);
                    b4[u] = ok && two ? __ldcg(reinterpret_cast<const float4 *>(part + (r0 + u) * per_r + ic))
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    z0[0] += a4[u].x; z0[1] += a4[u].y; z0[2] += a4[u].z; z0[3] += a4[u].w;
                    pc[0] += b4[u].x; pc[1] += b4[u].y; pc[2] += b4[u].z; pc[3] += b4[u].w;
                }
            } else {
                for (int r = r0; r < min(r0 + 4, R); ++r) {
                    z0[0] += __ldcg(part + r * per_r + i0);
                    if (two) pc[0] += __ldcg(part + r * per_r + ic);
                }
            }
        }
#pragma unroll
        for (int e = 0; e < E; ++e) {
            float z = two ? fmaf(-gamma, pc[e] + vb[e], z0[e] + xb[e]) : z0[e] + xb[e];
            if (relu) z = (z > 0.f || z != z) ? z : 0.f;
            z0[e] = z;                                           // the activation
            pc[e] = tf32_hi(z);                                  // its leading term
        }
        if (VEC4) {                                              // out % 4 == 0: whole 16-byte groups
            if (H) *reinterpret_cast<float4 *>(H + ic) = make_float4(z0[0], z0[1], z0[2], z0[3]);
            if (hs) {
                *reinterpret_cast<float4 *>(hs) = make_float4(pc[0], pc[1], pc[2], pc[3]);
                *reinterpret_cast<float4 *>(hs + (int64_t)n_pad * out) =
                    make_float4(z0[0] - pc[0], z0[1] - pc[1], z0[2] - pc[2], z0[3] - pc[3]);
            }
        } else {
            if (H) H[ic] = z0[0];
            if (hs) {
                hs[0] = pc[0];
                hs[(int64_t)n_pad * out] = z0[0] - pc[0];
            }
        }
    }
}

// ---- host side ----------------------------------------------------------------------------

}  // namespace

// Shape of the launch for a layer of `out` rows and K inputs over m+1 models on `sms` SMs.
// Picks the k-range length that keeps all SMs busy with an even share of row tiles.
// Cost model, in units of the time one k-block takes: the block that finishes last runs
// ceil(items / 2) row tiles on its busier pipeline, nkb k-blocks each, plus a fixed start-up
// and drain; every extra k-range adds split-K partials that have to be written and summed.
bool stream_tc_plan(int sms, int K, int out, int n_r, int m, StreamTcPlan *p) {
    if (n_r < 1 || n_r > 64 || K < 256 || K % 4 != 0 || out < 64) return false;
    const int n_pad = (n_r + 15) / 16 * 16;
    const int tiles = (out + kTileRows - 1) / kTileRows;
    const int items_all = (m + 1) * tiles;
    double best = 1e30;
    for (int kr = kStreamTcMinKR; kr <= 1024; kr += kBlockK) {
        const int xs = 2 * (kr / kBlockK) * n_pad * 128;            // [X_hi; X_lo]
        if (xs + kPipes * 2 * kStageBytes + 1024 > kSmemBudget) break;
        int stages = (kSmemBudget - 1024 - xs) / (kPipes * kStageBytes);   // per pipeline
        if (stages > kMaxStages) stages = kMaxStages;
        const int R = (K + kr - 1) / kr;
        if (R > sms) continue;
        if (R > 1 && (R - 1) * kr >= K) continue;                    // same R as a shorter range
        const int nkb = kr / kBlockK;
        const int g_hi = sms / R < items_all ? sms / R : items_all;
        for (int g = 1; g <= g_hi; ++g) {                            // g = blocks along y: one wave
            const int items = (items_all + g - 1) / g;
            // split-K partials are written and read back: 2 R n_r / K of the streamed bytes,
            // cheap while they stay in L2
            const double part_bytes = (double)R * (m + 1) * n_r * out * 4.0;
            const double part_cost = 2.0 * R * n_r / K * (part_bytes > 64e6 ? 1.0 : 0.35);
            double est = (items + 1) / 2 * nkb * (1.0 + part_cost) + 6.0 + 0.2 * R;
            if (stages < 3) est *= 1.1;                             // a shallow ring hides less latency
            if (est < best) {
                best = est;
                p->KR = kr; p->R = R; p->stages = stages; p->G = g;
            }
        }
    }
    if (best > 1e29) return false;
    p->n_pad = n_pad;
    p->tiles_per_model = tiles;
    p->smem_bytes = 2 * (p->KR / kBlockK) * n_pad * 128 + kPipes * p->stages * kStageBytes + 1024;
    return true;
}

// one slot per (k-range, tile, converter warp)
int stream_tc_norm_slots(const StreamTcPlan &p) { return p.R * p.tiles_per_model * 4; }

cudaError_t launch_stream_tc(Context &c, const StreamTcPlan &p, const float *x, const float *V, int64_t ldv,
                             int64_t offW, int64_t offB, int K, int out, const float *X, int n_r, int m,
                             float *part, int np_base, cudaStream_t s, int *launches) {
    if (!encode_tiled_fn()) return cudaErrorNotSupported;
    CUtensorMap map_x, map_v;
    {   // x as a one-model stack, so that both operands go through the same 3-D path
        cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)out, 1};
        cuuint64_t strides[2] = {(cuuint64_t)K * 4, (cuuint64_t)K * 4 * (cuuint64_t)out};
        cuuint32_t box[3] = {kBlockK, kTileRows, 1};
        CUresult r = encode_cached(c, &map_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, x + offW, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)out, (cuuint64_t)m};
        cuuint64_t strides[2] = {(cuuint64_t)K * 4, (cuuint64_t)ldv * 4};
        cuuint32_t box[3] = {kBlockK, kTileRows, 1};
        CUresult r = encode_cached(c, &map_v, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, V + offW, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    StreamArgs a;
    a.X = X;
    a.V = V;
    a.ldv = ldv;
    a.offB = offB;
    a.part = part;
    a.normpart = c.normpart;
    a.np_slots = c.np_slots;
    a.np_base = np_base;
    a.K = K;
    a.out = out;
    a.n_r = n_r;
    a.n_pad = p.n_pad;
    a.m = m;
    a.KR = p.KR;
    a.tiles_per_model = p.tiles_per_model;
    a.stages = p.stages;
    a.status = c.dev_status;
    a.spin_limit = c.spin_limit;
    static PerDeviceOnce attr_set;
    if (attr_set.need(c.device)) {
        cudaError_t e = cudaFuncSetAttribute(stream_tf32x3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kSmemBudget);
        if (e != cudaSuccess) return e;
        attr_set.mark(c.device);
    }
    ++*launches;
    profile_mark(c, "stream_tf32x3", s);
    return launch_chained(stream_tf32x3_kernel, dim3(p.R, p.G), dim3(kThreads), p.smem_bytes, s, chain_launches(c),
                          map_x, map_v, a);
}

cudaError_t launch_stream_combine(Context &c, const StreamTcPlan &p, const float *part, const float *x,
                                  const float *V, int64_t ldv, int64_t offB, int out, int n_r, int m,
                                  float gamma, int relu, float *H, float *Hsplit, cudaStream_t s, int *launches) {
    ++*launches;
    profile_mark(c, "stream_combine", s);
    const bool vec = out % 4 == 0;
    const int n_pad = layer_tc_n_pad(n_r);
    const int per_model = (Hsplit ? n_pad : n_r) * (vec ? out / 4 : out);
    int bx = (per_model + 255) / 256;
    const int cap = ((c.sm_count > 0 ? c.sm_count : 148) * 16 + m) / (m + 1);   // about 16 blocks per SM in all
    if (bx > cap) bx = cap > 0 ? cap : 1;
    const dim3 grid(bx, m + 1);
    if (vec)
        return launch_chained(stream_combine_kernel<true>, grid, dim3(256), 0, s, chain_launches(c), part, p.R, m,
                              n_r, out, x, V, ldv, offB, gamma, relu, H, Hsplit, n_pad);
    return launch_chained(stream_combine_kernel<false>, grid, dim3(256), 0, s, chain_launches(c), part, p.R, m, n_r,
                          out, x, V, ldv, offB, gamma, relu, H, Hsplit, n_pad);
}

}  // namespace zeno
