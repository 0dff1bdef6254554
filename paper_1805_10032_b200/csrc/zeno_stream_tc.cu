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
// (the dropped a_lo b_lo term is below 2^-22 relative).
//
// Per block (one SM): a k-range of the input index, whose X_hi / X_lo slices stay resident in
// shared memory in the 128-byte-swizzled K-major layout the MMA reads, and a list of 128-row
// tiles of the stacked matrix.  Warp roles:
//   warp 0      TMA producer: 128 rows x 32 floats boxes of V (or x) into a 4-stage ring
//   warp 1      TMEM owner and MMA issuer (tcgen05.mma, A operand from TMEM, B from shared)
//   warps 2-5   converters: thread t owns row t of the tile; reads its 128 bytes from the stage,
//               accumulates v^2, splits into hi/lo and stores both to TMEM (tcgen05.st) where
//               the MMA picks them up; after the last k-block they drain the accumulator
//               (tcgen05.ld) into the split-K partial output.
// Every mbarrier wait is bounded; a wait that gives up raises a status word and the block leaves
// through the common teardown (pending bulk copies awaited, TMEM freed).
#include <cuda.h>

#include "zeno_internal.h"

namespace zeno {

namespace {

constexpr int kTileRows = 128;          // rows of the stacked matrix per tile = TMEM lanes
constexpr int kBlockK = 32;             // floats per k-block = one 128-byte swizzle row
constexpr int kStages = 4;
constexpr int kStageBytes = kTileRows * kBlockK * 4;
constexpr int kThreads = 192;
constexpr int kTmemCols = 256;          // D0 @0, D1 @64, A0 @128 (hi 32 + lo 32), A1 @192
constexpr uint32_t kSpinLimit = 1u << 22;

// ---- PTX wrappers -------------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if it gave up (and raises *abort_flag) or if another thread did.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 32) __nanosleep(40);
        if ((i & 127u) == 127u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]^T, tf32 inputs, fp32 accumulate
__device__ __forceinline__ void tc_mma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// value rounded to tf32 (10 explicit mantissa bits), ties away from zero in magnitude
__device__ __forceinline__ float tf32_hi(float a) {
    return __uint_as_float((__float_as_uint(a) + 0x1000u) & 0xffffe000u);
}

// K-major operand in the 128-byte swizzled layout: rows of 128 bytes, groups of 8 rows 1024
// bytes apart (stride-dimension offset), descriptor version 1, swizzle mode 2 (128 B).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)1 << 16;                 // leading-dimension offset: unused for swizzled K-major
    d |= (uint64_t)(1024 >> 4) << 32;       // stride-dimension offset
    d |= (uint64_t)1 << 46;                 // descriptor version
    d |= (uint64_t)2 << 61;                 // 128-byte swizzle
    return d;
}

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
    int *status;           // device status word (raised on a wait that gave up)
};

__global__ void __launch_bounds__(kThreads, 1)
stream_tf32x3_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_v,
                     StreamArgs a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[kStages * 2 + 8];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int issued[kStages];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int r = blockIdx.x;                         // k-range
    const int k0 = r * a.KR;
    const int k_len = min(a.KR, a.K - k0);
    const int nkb = (k_len + kBlockK - 1) / kBlockK;   // k-blocks in this range
    const int n_items_total = (a.m + 1) * a.tiles_per_model;

    // shared memory carve-up (dynamic part is 1024-byte aligned)
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int nkb_max = a.KR / kBlockK;
    const uint32_t xs_bytes = (uint32_t)nkb_max * a.n_pad * 128;
    uint8_t *xs_hi = base;
    uint8_t *xs_lo = base + xs_bytes;
    uint8_t *stages = base + 2 * xs_bytes;            // xs_bytes is a multiple of 1024 (n_pad % 16 == 0)

    const uint32_t bar_full = smem_u32(&bars[0]);               // + 8 * stage
    const uint32_t bar_empty = smem_u32(&bars[kStages]);
    const uint32_t bar_afull = smem_u32(&bars[2 * kStages]);     // 2 TMEM A buffers
    const uint32_t bar_aempty = smem_u32(&bars[2 * kStages + 2]);
    const uint32_t bar_dfull = smem_u32(&bars[2 * kStages + 4]);  // 2 accumulators
    const uint32_t bar_dempty = smem_u32(&bars[2 * kStages + 6]);

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 4);
            issued[s] = 0;
        }
        for (int q = 0; q < 2; ++q) {
            mbar_init(bar_afull + 8 * q, 4);
            mbar_init(bar_aempty + 8 * q, 1);
            mbar_init(bar_dfull + 8 * q, 1);
            mbar_init(bar_dempty + 8 * q, 4);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // TMEM allocation by one full warp
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }

    // X_hi / X_lo of this k-range in the swizzled K-major layout: row j of k-block kb at
    // kb * n_pad * 128 + j * 128, its 16-byte chunk c at position c ^ (j & 7).
    for (int t = tid; t < nkb_max * a.n_pad * 8; t += kThreads) {
        const int c = t & 7, j = (t >> 3) % a.n_pad, kb = (t >> 3) / a.n_pad;
        const int k = k0 + kb * kBlockK + c * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (j < a.n_r && k < a.K && kb < nkb) v = __ldg(reinterpret_cast<const float4 *>(a.X + (int64_t)j * a.K + k));
        float4 hi = make_float4(tf32_hi(v.x), tf32_hi(v.y), tf32_hi(v.z), tf32_hi(v.w));
        float4 lo = make_float4(v.x - hi.x, v.y - hi.y, v.z - hi.z, v.w - hi.w);
        const uint32_t off = (uint32_t)kb * a.n_pad * 128 + j * 128 + ((c ^ (j & 7)) << 4);
        *reinterpret_cast<float4 *>(xs_hi + off) = hi;
        *reinterpret_cast<float4 *>(xs_lo + off) = lo;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    volatile int *abortp = &abort_flag;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            for (int item = blockIdx.y; item < n_items_total && !*abortp; item += gridDim.y) {
                const int model = item / a.tiles_per_model, tile = item % a.tiles_per_model;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % kStages;
                    if (!mbar_wait(bar_empty + 8 * s, ((it / kStages) & 1) ^ 1, abortp)) break;
                    mbar_expect_tx(bar_full + 8 * s, kStageBytes);
                    const uint32_t dst = smem_u32(stages + s * kStageBytes);
                    // one issue site for both operands: x is a one-model stack
                    const CUtensorMap *map = model == 0 ? &map_x : &map_v;
                    tma_load_3d(dst, map, k0 + kb * kBlockK, tile * kTileRows, max(model - 1, 0), bar_full + 8 * s);
                    issued[s] = (int)(it / kStages) + 1;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // instruction descriptor: D fp32, A and B tf32, both K-major, N = n_pad, M = 128
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(a.n_pad >> 3) << 17) |
                                   ((uint32_t)(kTileRows >> 4) << 24);
            uint32_t it = 0, q = 0;
            for (int item = blockIdx.y; item < n_items_total && !*abortp; item += gridDim.y, ++q) {
                const uint32_t d_tmem = tmem + (q & 1) * 64;
                if (!mbar_wait(bar_dempty + 8 * (q & 1), ((q >> 1) & 1) ^ 1, abortp)) break;
                tc_fence_after();
                bool ok = true;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const uint32_t ab = it & 1;
                    if (!mbar_wait(bar_afull + 8 * ab, (it >> 1) & 1, abortp)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_tmem = tmem + 128 + ab * 64;
                    const uint32_t bh = smem_u32(xs_hi) + (uint32_t)kb * a.n_pad * 128;
                    const uint32_t bl = smem_u32(xs_lo) + (uint32_t)kb * a.n_pad * 128;
#pragma unroll
                    for (int ks = 0; ks < kBlockK / 8; ++ks) {
                        const uint64_t dh = smem_desc_sw128(bh + ks * 32);
                        const uint64_t dl = smem_desc_sw128(bl + ks * 32);
                        tc_mma_tf32_ts(d_tmem, a_tmem + ks * 8, dh, idesc, (kb | ks) != 0);        // a_hi x_hi
                        tc_mma_tf32_ts(d_tmem, a_tmem + 32 + ks * 8, dh, idesc, 1);                // a_lo x_hi
                        tc_mma_tf32_ts(d_tmem, a_tmem + ks * 8, dl, idesc, 1);                     // a_hi x_lo
                    }
                    tc_commit(bar_aempty + 8 * ab);    // the A buffer may be overwritten once these finish
                }
                if (!ok) break;
                tc_commit(bar_dfull + 8 * (q & 1));    // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------------------------ converters + epilogue
        const int quad = warp & 3;                    // TMEM lane quadrant this warp may access
        const int row = quad * 32 + lane;             // row of the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        uint32_t it = 0, q = 0;
        for (int item = blockIdx.y; item < n_items_total && !*abortp; item += gridDim.y, ++q) {
            const int model = item / a.tiles_per_model, tile = item % a.tiles_per_model;
            float nrm = 0.f;
            bool ok = true;
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const int s = it % kStages;
                if (!mbar_wait(bar_full + 8 * s, (it / kStages) & 1, abortp)) { ok = false; break; }
                const uint8_t *src = stages + s * kStageBytes + row * 128;
                float4 v[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) v[c] = *reinterpret_cast<const float4 *>(src + ((c ^ (row & 7)) << 4));
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_empty + 8 * s);      // the stage may be refilled
                uint32_t hi[32], lo[32];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const float e[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        nrm = fmaf(e[u], e[u], nrm);
                        const float h = tf32_hi(e[u]);
                        hi[4 * c + u] = __float_as_uint(h);
                        lo[4 * c + u] = __float_as_uint(e[u] - h);
                    }
                }
                const uint32_t ab = it & 1;
                if (!mbar_wait(bar_aempty + 8 * ab, ((it >> 1) & 1) ^ 1, abortp)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_tmem = tmem + lane_addr + 128 + ab * 64;
                tc_st16(a_tmem, reinterpret_cast<const uint32_t(&)[16]>(hi[0]));
                tc_st16(a_tmem + 16, reinterpret_cast<const uint32_t(&)[16]>(hi[16]));
                tc_st16(a_tmem + 32, reinterpret_cast<const uint32_t(&)[16]>(lo[0]));
                tc_st16(a_tmem + 48, reinterpret_cast<const uint32_t(&)[16]>(lo[16]));
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_afull + 8 * ab);
            }
            if (!ok) break;

            // partial sum of squares of this tile's rows (model 0 is x itself: not a candidate)
            if (model > 0) {
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

            // drain the accumulator: thread = output row o, column = sample j
            if (!mbar_wait(bar_dfull + 8 * (q & 1), (q >> 1) & 1, abortp)) break;
            tc_fence_after();
            const int o = tile * kTileRows + row;
            float *dst = a.part + (((int64_t)r * (a.m + 1) + model) * a.n_r) * a.out + o;
            for (int j0 = 0; j0 < a.n_pad; j0 += 16) {
                uint32_t acc[16];
                tc_ld16(tmem + lane_addr + (q & 1) * 64 + j0, acc);
                tc_wait_ld();
                if (o < a.out) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (j0 + j < a.n_r) dst[(int64_t)(j0 + j) * a.out] = __uint_as_float(acc[j]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_dempty + 8 * (q & 1));
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (tid == 0) {
        // bulk copies still in flight (only after an aborted run) must land before the block exits
        if (abort_flag) {
            for (int s = 0; s < kStages; ++s)
                if (issued[s] > 0) {
                    for (uint32_t i = 0; i < kSpinLimit; ++i) {
                        if (mbar_try_wait(bar_full + 8 * s, (uint32_t)(issued[s] - 1) & 1)) break;
                        __nanosleep(64);
                    }
                }
            atomicMax(a.status, 1);
        }
    }
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// Split-K reduction and activation after the streamed first layer:
//   z_0 = sum_r P[r][0] + b(x),   z_c = z_0 - gamma (sum_r P[r][c] + b(v_c)),   h = ReLU(z)
// One thread per (model, sample, output); partials are added in k-range order.
__global__ void __launch_bounds__(256) stream_combine_kernel(const float *part, int R, int m, int n_r, int out,
                                                             const float *x, const float *V, int64_t ldv,
                                                             int64_t offB, float gamma, int relu, float *H) {
    const int64_t total = (int64_t)(m + 1) * n_r * out;
    const int64_t per_r = total;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int o = (int)(t % out);
        const int64_t cj = t / out;
        const int c = (int)(cj / n_r), j = (int)(cj % n_r);
        const int64_t base_idx = (int64_t)j * out + o;          // model 0
        float z0 = 0.f, pc = 0.f;
        for (int r = 0; r < R; ++r) {
            z0 += part[r * per_r + base_idx];
            if (c > 0) pc += part[r * per_r + t];
        }
        if (offB >= 0) {
            z0 += __ldg(x + offB + o);
            if (c > 0) pc += __ldg(V + (int64_t)(c - 1) * ldv + offB + o);
        }
        float z = c > 0 ? fmaf(-gamma, pc, z0) : z0;
        if (relu) z = (z > 0.f || z != z) ? z : 0.f;
        H[t] = z;
    }
}

// ---- host side ----------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

// Shape of the launch for a layer of `out` rows and K inputs over m+1 models on `sms` SMs.
// Picks the k-range length that keeps all SMs busy with an even share of row tiles.
bool stream_tc_plan(int sms, int K, int out, int n_r, int m, StreamTcPlan *p) {
    if (n_r < 1 || n_r > 64 || K < 256 || K % 4 != 0 || out < 64) return false;
    const int n_pad = (n_r + 15) / 16 * 16;
    const int tiles = (out + kTileRows - 1) / kTileRows;
    const int items = (m + 1) * tiles;
    const int kr_cap = n_pad <= 32 ? 512 : 256;      // X_hi + X_lo <= 128 KB of shared memory
    double best = -1.0;
    for (int kr = kStreamTcMinKR; kr <= kr_cap; kr *= 2) {
        const int R = (K + kr - 1) / kr;
        if (R > sms) continue;
        int G = sms / R;
        if (G > items) G = items;
        if (G < 1) G = 1;
        const int per = (items + G - 1) / G;
        double eff = (double)items / ((double)G * per) * ((double)(R * G) / sms);
        eff -= 0.01 * R;                               // split-K partial traffic grows with R
        if (eff > best) {
            best = eff;
            p->KR = kr; p->R = R; p->G = G;
        }
    }
    if (best < 0) return false;
    p->n_pad = n_pad;
    p->tiles_per_model = tiles;
    p->smem_bytes = 2 * (p->KR / kBlockK) * n_pad * 128 + kStages * kStageBytes + 1024;
    return true;
}

int stream_tc_norm_slots(const StreamTcPlan &p) { return p.R * p.tiles_per_model * 4; }

cudaError_t launch_stream_tc(Context &c, const StreamTcPlan &p, const float *x, const float *V, int64_t ldv,
                             int64_t offW, int64_t offB, int K, int out, const float *X, int n_r, int m,
                             float *part, int np_base, cudaStream_t s, int *launches) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return cudaErrorNotSupported;
    CUtensorMap map_x, map_v;
    {   // x as a one-model stack, so that both operands go through the same 3-D path
        cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)out, 1};
        cuuint64_t strides[2] = {(cuuint64_t)K * 4, (cuuint64_t)K * 4 * (cuuint64_t)out};
        cuuint32_t box[3] = {kBlockK, kTileRows, 1};
        cuuint32_t es[3] = {1, 1, 1};
        CUresult r = enc(&map_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(x + offW), dims, strides,
                         box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)out, (cuuint64_t)m};
        cuuint64_t strides[2] = {(cuuint64_t)K * 4, (cuuint64_t)ldv * 4};
        cuuint32_t box[3] = {kBlockK, kTileRows, 1};
        cuuint32_t es[3] = {1, 1, 1};
        CUresult r = enc(&map_v, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(V + offW), dims, strides,
                         box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
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
    a.status = c.dev_status;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(stream_tf32x3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             200 * 1024);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    ++*launches;
    profile_mark(c, "stream_tf32x3", s);
    dim3 grid(p.R, p.G);
    stream_tf32x3_kernel<<<grid, kThreads, p.smem_bytes, s>>>(map_x, map_v, a);
    return cudaGetLastError();
}

cudaError_t launch_stream_combine(Context &c, const StreamTcPlan &p, const float *part, const float *x,
                                  const float *V, int64_t ldv, int64_t offB, int out, int n_r, int m,
                                  float gamma, int relu, float *H, cudaStream_t s, int *launches) {
    ++*launches;
    profile_mark(c, "stream_combine", s);
    const int64_t total = (int64_t)(m + 1) * n_r * out;
    int blocks = (int)((total + 255) / 256);
    const int cap = (c.sm_count > 0 ? c.sm_count : 148) * 8;
    if (blocks > cap) blocks = cap;
    stream_combine_kernel<<<blocks, 256, 0, s>>>(part, p.R, m, n_r, out, x, V, ldv, offB, gamma, relu, H);
    return cudaGetLastError();
}

}  // namespace zeno
