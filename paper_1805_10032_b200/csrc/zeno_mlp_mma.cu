// Dense layers whose input activations differ per model (every layer after the first, and the
// first layer of bfloat16 models), on warp-level tensor-core MMAs.
//
// Same contract as mlp_layer_kernel: one launch evaluates the layer for all m+1 models; the
// candidate's weights w = x - gamma v are formed in registers from the loads of x and V and go
// straight into the A fragments (the perturbed model is never written anywhere); ||v||^2 is
// accumulated from the same registers.  The n_r dot products per row, which bound the FMA
// version, become m16n8k8 (tf32) or m16n8k16 (bf16) MMAs against the model's activations
// staged in shared memory.
//
// Precision.  fp32 models: both operands are split into a tf32 value and its remainder and
// three products are accumulated (hi hi into one accumulator, lo hi + hi lo into another, so
// that the tensor core's truncating adds act on the small terms separately).  bfloat16 models:
// the weights are exact in bf16; the fp32 activations are split into two bf16 terms.
//
// The activations are split once per stage, by the whole block, while they are written to shared
// memory, in the order the B fragments want them: 16 bytes per (sample, k-pair) holding
// {hi(k), hi(k+1), lo(k), lo(k+1)} for tf32, per (sample, k-quad) holding the packed bf16 pairs
// {h0(k,k+1), h0(k+2,k+3), h1(k,k+1), h1(k+2,k+3)} for bf16.  One 16-byte shared load then feeds
// all the MMAs of an (n-tile, k-step); slots are swizzled so that these loads are conflict free.
//
// A warp owns 16 output rows; lane (g, t) = (lane / 4, lane % 4) loads, for rows g and g + 8,
// the eight consecutive k-values 8t .. 8t+7 of each 32-wide k-block (one or two 16-byte loads),
// so every row is read in full 128-byte (64-byte for bf16) segments.  The MMA's k index is a
// permutation of the memory order; the B fragments read the activations with the same
// permutation, which leaves the dot products unchanged.
#include "zeno_internal.h"

namespace zeno {

namespace {

constexpr int kMmaWarps = 4;                 // warps per block, 16 rows each
constexpr int kMmaRows = 16 * kMmaWarps;     // rows per block
constexpr int kHS = 64;                      // k-extent of one shared-memory stage of activations

// 16-byte slots per staged sample row (one spare slot staggers consecutive rows over the banks)
template <bool BF16> struct StageShape {
    static constexpr int kSlots = BF16 ? kHS / 4 : kHS / 2;
    static constexpr int kPitch = kSlots + 1;
};
// tf32 slots 8..15 of each 16 are rotated by two so that lanes t and t+2 of a row do not collide
template <bool BF16> __device__ __forceinline__ int swizzle_slot(int slot) {
    return BF16 ? slot : slot ^ (((slot >> 3) & 1) << 1);
}

__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);      // .x (low half) = lo
    return *reinterpret_cast<uint32_t *>(&p);
}
__device__ __forceinline__ float bf16_round(float a) { return __bfloat162float(__float2bfloat16_rn(a)); }
__device__ __forceinline__ float relu_keep_nan(float z) { return (z > 0.f || z != z) ? z : 0.f; }

// eight consecutive parameters starting at p (16-byte aligned for bf16, 32-byte span for fp32)
__device__ __forceinline__ void load8(const float *p, float (&o)[8]) {
    float4 a = __ldg(reinterpret_cast<const float4 *>(p));
    float4 b = __ldg(reinterpret_cast<const float4 *>(p) + 1);
    o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&o)[8]) {
    uint4 q = __ldg(reinterpret_cast<const uint4 *>(p));
    const unsigned w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        o[2 * i] = __uint_as_float(w[i] << 16);
        o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

template <typename T, int NRT>
__global__ void __launch_bounds__(kMmaWarps * 32) mlp_layer_mma_kernel(LayerArgs a) {
    constexpr bool kBf16 = is_bf16<T>::value;
    constexpr int NT = NRT / 8;                 // n-tiles of 8 samples
    constexpr int kPitch = StageShape<kBf16>::kPitch;
    constexpr int kChunks = NRT * (kHS / 4) / (kMmaWarps * 32);   // float4 chunks of a stage per thread
    extern __shared__ __align__(16) uint4 hs_dyn[];                 // [2][NRT][kPitch]

    pdl_wait();
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int c = blockIdx.y;
    // sample tiles of the same rows sit in neighbouring blocks, so that V is read from HBM once
    const int n_ztiles = (a.n_r + NRT - 1) / NRT;
    const int ztile = blockIdx.x % n_ztiles, rowblk = blockIdx.x / n_ztiles;
    const int j0 = ztile * NRT;
    const int row0 = (rowblk * kMmaWarps + warp) * 16;
    const int K = a.in;
    const bool has_v = c > 0;
    const int n_valid = min(NRT, a.n_r - j0);

    const int ra = min(row0 + g, a.out - 1), rb = min(row0 + g + 8, a.out - 1);   // clamped rows
    const bool live_a = row0 + g < a.out, live_b = row0 + g + 8 < a.out;
    const T *xw = static_cast<const T *>(a.x) + a.offW;
    const T *vbase = static_cast<const T *>(a.V) + (has_v ? (int64_t)(c - 1) * a.ldv : 0);
    const T *vw = vbase + a.offW;
    const T *xa = xw + (int64_t)ra * K, *xb = xw + (int64_t)rb * K;
    const T *va = vw + (int64_t)ra * K, *vb = vw + (int64_t)rb * K;
    const float *hin = a.Hin + (int64_t)c * a.hin_cand_stride + (int64_t)j0 * K;

    float big[NT][4], small[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int q = 0; q < 4; ++q) big[n][q] = small[n][q] = 0.f;
    float nrm = 0.f;

    const int n_stages = (K + kHS - 1) / kHS;
    const int n_blocks = (K + 31) / 32;

    // activations of stage s: loaded into registers one stage ahead, split and stored in
    // fragment order when the buffer is free
    float4 hreg[kChunks];
    auto load_stage = [&](int s) {
        const int kb = s * kHS;
#pragma unroll
        for (int u = 0; u < kChunks; ++u) {
            const int i = threadIdx.x + u * (kMmaWarps * 32);
            const int j = i / (kHS / 4), kk = (i % (kHS / 4)) * 4;
            hreg[u] = (j < n_valid && kb + kk < K) ? __ldg(reinterpret_cast<const float4 *>(hin + (int64_t)j * K + kb + kk))
                                                    : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    auto store_stage = [&](int s) {
        uint4 *dst = hs_dyn + (size_t)(s & 1) * NRT * kPitch;
#pragma unroll
        for (int u = 0; u < kChunks; ++u) {
            const int i = threadIdx.x + u * (kMmaWarps * 32);
            const int j = i / (kHS / 4), q = i % (kHS / 4);      // q: index of the 4-wide k chunk
            const float4 h = hreg[u];
            if (kBf16) {
                const float f0 = bf16_round(h.x), f1 = bf16_round(h.y), f2 = bf16_round(h.z), f3 = bf16_round(h.w);
                dst[j * kPitch + q] = make_uint4(pack_bf16(f0, f1), pack_bf16(f2, f3), pack_bf16(h.x - f0, h.y - f1),
                                                 pack_bf16(h.z - f2, h.w - f3));
            } else {
                const float a0 = tf32_hi(h.x), a1 = tf32_hi(h.y), a2 = tf32_hi(h.z), a3 = tf32_hi(h.w);
                dst[j * kPitch + swizzle_slot<false>(2 * q)] =
                    make_uint4(__float_as_uint(a0), __float_as_uint(a1), __float_as_uint(h.x - a0), __float_as_uint(h.y - a1));
                dst[j * kPitch + swizzle_slot<false>(2 * q + 1)] =
                    make_uint4(__float_as_uint(a2), __float_as_uint(a3), __float_as_uint(h.z - a2), __float_as_uint(h.w - a3));
            }
        }
    };
    // eight x and v values of rows g and g+8 for k-block kb (zero past K; K % 8 == 0 on this path)
    auto load_block = [&](int kblk, float (&xA)[8], float (&vA)[8], float (&xB)[8], float (&vB)[8]) {
        const int k = kblk * 32 + 8 * t;
        if (k < K) {
            load8(xa + k, xA);
            load8(xb + k, xB);
            if (has_v) {
                load8(va + k, vA);
                load8(vb + k, vB);
            }
        }
        if (k >= K || !has_v) {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if (k >= K) xA[e] = xB[e] = 0.f;
                vA[e] = vB[e] = 0.f;
            }
        }
    };

    float xA[8], vA[8], xB[8], vB[8];
    load_stage(0);
    load_block(0, xA, vA, xB, vB);
    store_stage(0);
    for (int s = 0; s < n_stages; ++s) {
        __syncthreads();                                   // stage s is complete, buffer (s+1)&1 is free
        if (s + 1 < n_stages) load_stage(s + 1);
        const uint4 *h = hs_dyn + (size_t)(s & 1) * NRT * kPitch;
#pragma unroll
        for (int half = 0; half < kHS / 32; ++half) {
            const int kblk = s * (kHS / 32) + half;
            if (kblk < n_blocks) {
                float xA2[8], vA2[8], xB2[8], vB2[8];
                if (kblk + 1 < n_blocks) load_block(kblk + 1, xA2, vA2, xB2, vB2);
                // candidate weights of this lane's 2 x 8 entries, and v^2
                float wA[8], wB[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    wA[e] = candidate_param<T>(xA[e], vA[e], a.gamma);
                    wB[e] = candidate_param<T>(xB[e], vB[e], a.gamma);
                    if (live_a) nrm = fmaf(vA[e], vA[e], nrm);
                    if (live_b) nrm = fmaf(vB[e], vB[e], nrm);
                }
                if (!kBf16) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        // MMA k index t <-> memory column 8t + 2ks, t + 4 <-> 8t + 2ks + 1
                        const float e[4] = {wA[2 * ks], wB[2 * ks], wA[2 * ks + 1], wB[2 * ks + 1]};
                        uint32_t ah[4], al[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float hi = tf32_hi(e[q]);
                            ah[q] = __float_as_uint(hi);
                            al[q] = __float_as_uint(e[q] - hi);
                        }
                        const int slot = swizzle_slot<false>(half * 16 + 4 * t + ks);
#pragma unroll
                        for (int n = 0; n < NT; ++n) {
                            const uint4 b = h[(n * 8 + g) * kPitch + slot];   // {hi k, hi k+1, lo k, lo k+1}
                            mma_tf32(big[n], ah, b.x, b.y);
                            mma_tf32(small[n], al, b.x, b.y);
                            mma_tf32(small[n], ah, b.z, b.w);
                        }
                    }
                } else {
#pragma unroll
                    for (int ks = 0; ks < 2; ++ks) {
                        // MMA k pairs (2t,2t+1) <-> columns 8t+4ks, +1 ; (2t+8,2t+9) <-> 8t+4ks+2, +3
                        uint32_t aw[4];
                        aw[0] = pack_bf16(wA[4 * ks], wA[4 * ks + 1]);
                        aw[1] = pack_bf16(wB[4 * ks], wB[4 * ks + 1]);
                        aw[2] = pack_bf16(wA[4 * ks + 2], wA[4 * ks + 3]);
                        aw[3] = pack_bf16(wB[4 * ks + 2], wB[4 * ks + 3]);
                        const int slot = half * 8 + 2 * t + ks;
#pragma unroll
                        for (int n = 0; n < NT; ++n) {
                            const uint4 b = h[(n * 8 + g) * kPitch + slot];   // {h0 pair, h0 pair, h1 pair, h1 pair}
                            mma_bf16(big[n], aw, b.x, b.y);
                            mma_bf16(small[n], aw, b.z, b.w);
                        }
                    }
                }
                if (kblk + 1 < n_blocks) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        xA[e] = xA2[e]; vA[e] = vA2[e]; xB[e] = xB2[e]; vB[e] = vB2[e];
                    }
                }
            }
        }
        if (s + 1 < n_stages) store_stage(s + 1);          // buffer (s+1)&1 was last read in stage s-1
    }

    // accumulator fragment: rows g / g+8, samples 8n + 2t, 8n + 2t + 1
    float bias_a = 0.f, bias_b = 0.f;
    if (a.offB >= 0) {
        const T *xbias = static_cast<const T *>(a.x) + a.offB;
        const float va0 = has_v ? load_elem(vbase + a.offB + ra) : 0.f;
        const float vb0 = has_v ? load_elem(vbase + a.offB + rb) : 0.f;
        bias_a = candidate_param<T>(load_elem(xbias + ra), va0, a.gamma);
        bias_b = candidate_param<T>(load_elem(xbias + rb), vb0, a.gamma);
        if (has_v && t == 0 && ztile == 0) {            // each bias entry counted once
            if (live_a) nrm = fmaf(va0, va0, nrm);
            if (live_b) nrm = fmaf(vb0, vb0, nrm);
        }
    }
#pragma unroll
    for (int n = 0; n < NT; ++n) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int j = n * 8 + 2 * t + (q & 1);
            const bool second = q >= 2;
            if (j < n_valid && (second ? live_b : live_a)) {
                float z = big[n][q] + small[n][q] + (second ? bias_b : bias_a);
                if (a.relu) z = relu_keep_nan(z);
                a.Hout[((int64_t)c * a.n_r + j0 + j) * a.out + (second ? row0 + g + 8 : row0 + g)] = z;
            }
        }
    }
    if (has_v && ztile == 0) {
#pragma unroll
        for (int sft = 16; sft >= 1; sft >>= 1) nrm += __shfl_xor_sync(0xffffffffu, nrm, sft);
        if (lane == 0)
            a.normpart[(int64_t)(c - 1) * a.np_slots + a.np_base + rowblk * kMmaWarps + warp] = nrm;
    }
}

template <typename T>
cudaError_t launch_mma_typed(const LayerArgs &a, cudaStream_t s, bool overlap) {
    auto go = [&](auto kernel, int nrt) {
        dim3 grid((a.out + kMmaRows - 1) / kMmaRows * ((a.n_r + nrt - 1) / nrt), a.m + 1);
        const size_t smem = (size_t)2 * nrt * StageShape<is_bf16<T>::value>::kPitch * 16;
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        return launch_chained(kernel, grid, dim3(kMmaWarps * 32), smem, s, overlap, a);
    };
    if (a.n_r <= 16) return go(mlp_layer_mma_kernel<T, 16>, 16);
    if (a.n_r <= 32) return go(mlp_layer_mma_kernel<T, 32>, 32);
    return go(mlp_layer_mma_kernel<T, 64>, 64);
}

}  // namespace

int mlp_mma_norm_slots(int out) { return (out + kMmaRows - 1) / kMmaRows * kMmaWarps; }

// Rows must be 16-byte aligned and every row a multiple of eight parameters long.
bool mlp_mma_usable(int in, int out) { return in % 8 == 0 && in >= 64 && out >= 16; }

cudaError_t launch_mlp_layer_mma(Context &c, const LayerArgs &a, cudaStream_t s, int *launches) {
    ++*launches;
    profile_mark(c, "mlp_layer_mma", s);
    if (c.desc.param_dtype == ZENO_BF16) return launch_mma_typed<__nv_bfloat16>(a, s, chain_launches(c));
    return launch_mma_typed<float>(a, s, chain_launches(c));
}

}  // namespace zeno
