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
constexpr int kHPitch = kHS + 4;             // floats per staged row (keeps 16-byte alignment)

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem, bool valid) {
    unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem));
    int bytes = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ float tf32_hi(float a) {
    return __uint_as_float((__float_as_uint(a) + 0x1000u) & 0xffffe000u);
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
    __shared__ __align__(16) float hs[2][NRT][kHPitch];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int c = blockIdx.y;
    const int j0 = blockIdx.z * NRT;
    const int row0 = (blockIdx.x * kMmaWarps + warp) * 16;
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

    auto issue_stage = [&](int s) {
        const int kb = s * kHS;
        for (int i = threadIdx.x; i < NRT * (kHS / 4); i += kMmaWarps * 32) {
            const int j = i / (kHS / 4), kk = (i % (kHS / 4)) * 4;
            const bool ok = j < n_valid && kb + kk < K;
            cp_async16(&hs[s & 1][j][kk], ok ? hin + (int64_t)j * K + kb + kk : a.Hin, ok);
        }
        cp_async_commit();
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
    issue_stage(0);
    load_block(0, xA, vA, xB, vB);
    for (int s = 0; s < n_stages; ++s) {
        if (s + 1 < n_stages) {
            issue_stage(s + 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
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
                const float(*h)[kHPitch] = hs[s & 1];
                const int kofs = half * 32 + 8 * t;
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
#pragma unroll
                        for (int n = 0; n < NT; ++n) {
                            const float2 hv = *reinterpret_cast<const float2 *>(&h[n * 8 + g][kofs + 2 * ks]);
                            const float h0 = tf32_hi(hv.x), h1 = tf32_hi(hv.y);
                            const uint32_t bh0 = __float_as_uint(h0), bh1 = __float_as_uint(h1);
                            const uint32_t bl0 = __float_as_uint(hv.x - h0), bl1 = __float_as_uint(hv.y - h1);
                            mma_tf32(big[n], ah, bh0, bh1);
                            mma_tf32(small[n], al, bh0, bh1);
                            mma_tf32(small[n], ah, bl0, bl1);
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
#pragma unroll
                        for (int n = 0; n < NT; ++n) {
                            const float4 hv = *reinterpret_cast<const float4 *>(&h[n * 8 + g][kofs + 4 * ks]);
                            const float f0 = bf16_round(hv.x), f1 = bf16_round(hv.y);
                            const float f2 = bf16_round(hv.z), f3 = bf16_round(hv.w);
                            const uint32_t bh0 = pack_bf16(f0, f1), bh1 = pack_bf16(f2, f3);
                            const uint32_t bl0 = pack_bf16(hv.x - f0, hv.y - f1), bl1 = pack_bf16(hv.z - f2, hv.w - f3);
                            mma_bf16(big[n], aw, bh0, bh1);
                            mma_bf16(small[n], aw, bl0, bl1);
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
        __syncthreads();
    }

    // accumulator fragment: rows g / g+8, samples 8n + 2t, 8n + 2t + 1
    float bias_a = 0.f, bias_b = 0.f;
    if (a.offB >= 0) {
        const T *xbias = static_cast<const T *>(a.x) + a.offB;
        const float va0 = has_v ? load_elem(vbase + a.offB + ra) : 0.f;
        const float vb0 = has_v ? load_elem(vbase + a.offB + rb) : 0.f;
        bias_a = candidate_param<T>(load_elem(xbias + ra), va0, a.gamma);
        bias_b = candidate_param<T>(load_elem(xbias + rb), vb0, a.gamma);
        if (has_v && t == 0 && blockIdx.z == 0) {       // each bias entry counted once
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
    if (has_v && blockIdx.z == 0) {
#pragma unroll
        for (int sft = 16; sft >= 1; sft >>= 1) nrm += __shfl_xor_sync(0xffffffffu, nrm, sft);
        if (lane == 0)
            a.normpart[(int64_t)(c - 1) * a.np_slots + a.np_base + blockIdx.x * kMmaWarps + warp] = nrm;
    }
}

template <typename T>
cudaError_t launch_mma_typed(const LayerArgs &a, cudaStream_t s) {
    auto go = [&](auto kernel, int nrt) {
        dim3 grid((a.out + kMmaRows - 1) / kMmaRows, a.m + 1, (a.n_r + nrt - 1) / nrt);
        kernel<<<grid, kMmaWarps * 32, 0, s>>>(a);
        return cudaGetLastError();
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
    if (c.desc.param_dtype == ZENO_BF16) return launch_mma_typed<__nv_bfloat16>(a, s);
    return launch_mma_typed<float>(a, s);
}

}  // namespace zeno
