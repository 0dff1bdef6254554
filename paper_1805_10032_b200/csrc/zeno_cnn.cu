// Convolutional layers of the candidates' models (loss kind ZENO_LOSS_SOFTMAX_CNN): one layer of all m + 1
// models per launch, 3 x 3 windows, stride 1, zero padding 1, bias, ReLU, and -- after every second layer --
// the 2 x 2 max pooling folded into the same kernel.  Every model has its own weights w = x - gamma v_c, formed
// while they are staged; the sums of v^2 come from the same loads.
//
// A block takes one model, sixteen output planes and as many samples as fill its 256 threads; a thread owns a
// 2 x 2 square of output pixels in all sixteen planes (64 accumulators), so that the pooling needs no exchange.
// The input planes go through shared memory eight at a time, with a zero border (the padding), next to that
// chunk's weights stored [input plane][tap][output plane]: a thread reads its 4 x 4 input patch once per input
// plane and, per tap, the sixteen planes' weights as four broadcast loads.  This is an fp32 FMA kernel: the
// models here are small (the paper's CNN has about 1e5 parameters), the work is in the activations, and each
// of the m + 1 models has other weights, so there is no shared operand to stream.
#include <math.h>

#include "zeno_internal.h"

namespace zeno {

namespace {

constexpr int kCnnThreads = 256;
constexpr int kCnnCo = 16;                   // output planes per block
constexpr int kCnnCi = 8;                    // input planes staged at a time
constexpr int kCnnMaxSpb = 16;               // most samples a block takes

__host__ __device__ inline int cnn_threads_per_plane(int side) { return (side / 2) * (side / 2); }
__host__ __device__ inline int cnn_samples_per_block(int side) {
    const int spb = kCnnThreads / cnn_threads_per_plane(side);
    return spb > kCnnMaxSpb ? kCnnMaxSpb : spb;
}
// padded plane: side + 2 rows of an even number of floats (a thread's patch starts at an even column)
__host__ __device__ inline int cnn_pitch(int side) { return side + 2; }
inline size_t cnn_smem_bytes(int side) {
    const size_t planes = (size_t)cnn_samples_per_block(side) * kCnnCi * (side + 2) * cnn_pitch(side);
    return (planes + (size_t)kCnnCi * 9 * kCnnCo) * sizeof(float);
}

__device__ __forceinline__ float max_nan(float a, float b) { return (a != a) ? a : ((b != b) ? b : fmaxf(a, b)); }
// a / b for small a (well below 2^20) with inv_b = 1.0f / b
__device__ __forceinline__ int div_small(int a, float inv_b) { return __float2int_rd(((float)a + 0.5f) * inv_b); }

template <typename T>
__global__ void __launch_bounds__(kCnnThreads) cnn_conv3x3_kernel(CnnLayerArgs a) {
    extern __shared__ __align__(16) float cnn_smem[];
    const int side = a.side, pitch = cnn_pitch(side), plane = (side + 2) * pitch;
    const int tpp = cnn_threads_per_plane(side), spb = cnn_samples_per_block(side);
    float *in_s = cnn_smem;                                          // [spb][kCnnCi][side + 2][pitch]
    float *w_s = cnn_smem + (size_t)spb * kCnnCi * plane;            // [kCnnCi][9][kCnnCo]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int c = blockIdx.z;                                        // model: 0 is x itself
    const int co0 = blockIdx.x * kCnnCo;
    const int j0 = blockIdx.y * spb;                                 // first sample of this block
    const bool has_v = c > 0;
    const T *xw = static_cast<const T *>(a.x) + a.offW;
    const T *vrow = static_cast<const T *>(a.V) + (has_v ? (int64_t)(c - 1) * a.ldv : 0);
    const T *vw = vrow + a.offW;

    // this thread's sample and 2 x 2 square
    const int ls = tid / tpp, tp = tid - ls * tpp;                   // local sample, square within the plane
    const int half = side / 2;
    const int qy = tp / half, qx = tp - qy * half;
    const bool live = ls < spb && j0 + ls < a.n_r;

    // zero the staged planes once: the border stays zero, the inside is overwritten by every chunk
    for (int t = tid; t < spb * kCnnCi * plane; t += kCnnThreads) in_s[t] = 0.f;

    pdl_wait();
    pdl_launch_dependents();

    float acc[kCnnCo][4];
#pragma unroll
    for (int o = 0; o < kCnnCo; ++o)
#pragma unroll
        for (int p = 0; p < 4; ++p) acc[o][p] = 0.f;
    float nrm = 0.f;
    const int pixels = side * side;
    const float inv_pixels = 1.0f / (float)pixels, inv_side = 1.0f / (float)side;
    const float *hin = a.Hin + (int64_t)c * a.hin_cand_stride;
    const bool count_norm = has_v && blockIdx.y == 0;                // one block per (model, plane group) adds up v^2

    for (int ci0 = 0; ci0 < a.cin; ci0 += kCnnCi) {
        __syncthreads();                                             // the previous chunk has been used
        // input planes ci0 .. ci0 + 7 of the block's samples (zero past cin and past the last sample)
#pragma unroll 4
        for (int t = tid; t < spb * kCnnCi * pixels; t += kCnnThreads) {
            const int sc = div_small(t, inv_pixels), pix = t - sc * pixels;      // (sample, plane) and pixel
            const int yy = div_small(pix, inv_side), xx = pix - yy * side;
            const int sm = sc / kCnnCi, ci = sc % kCnnCi;
            float v = 0.f;
            if (ci0 + ci < a.cin && j0 + sm < a.n_r)
                v = hin[((int64_t)(j0 + sm) * a.cin + ci0 + ci) * pixels + pix];
            in_s[sc * plane + (yy + 1) * pitch + xx + 1] = v;
        }
        // weights of the chunk: w = x - gamma v, zero past cin / cout
        for (int t = tid; t < kCnnCo * kCnnCi * 9; t += kCnnThreads) {
            const int o = t / (kCnnCi * 9), r = t - o * (kCnnCi * 9), ci = r / 9, tap = r - ci * 9;
            float w = 0.f;
            if (co0 + o < a.cout && ci0 + ci < a.cin) {
                const int64_t e = ((int64_t)(co0 + o) * a.cin + ci0 + ci) * 9 + tap;
                const float xv = load_elem(xw + e);
                const float vv = has_v ? load_elem(vw + e) : 0.f;
                w = candidate_param<T>(xv, vv, a.gamma);
                if (count_norm) nrm = fmaf(vv, vv, nrm);
            }
            w_s[(ci * 9 + tap) * kCnnCo + o] = w;
        }
        __syncthreads();
        if (live) {
            const float *base = in_s + (size_t)ls * kCnnCi * plane + (2 * qy) * pitch + 2 * qx;
#pragma unroll 1
            for (int ci = 0; ci < kCnnCi; ++ci) {
                float patch[4][4];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const float2 lo = *reinterpret_cast<const float2 *>(base + ci * plane + r * pitch);
                    const float2 hi = *reinterpret_cast<const float2 *>(base + ci * plane + r * pitch + 2);
                    patch[r][0] = lo.x; patch[r][1] = lo.y; patch[r][2] = hi.x; patch[r][3] = hi.y;
                }
#pragma unroll
                for (int tap = 0; tap < 9; ++tap) {
                    const int dy = tap / 3, dx = tap - dy * 3;
                    const float4 *wp = reinterpret_cast<const float4 *>(w_s + (ci * 9 + tap) * kCnnCo);
#pragma unroll
                    for (int g = 0; g < kCnnCo / 4; ++g) {
                        const float4 w4 = wp[g];
                        const float wv[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                        for (int u = 0; u < 4; ++u)
#pragma unroll
                            for (int p = 0; p < 4; ++p)
                                acc[4 * g + u][p] = fmaf(wv[u], patch[(p >> 1) + dy][(p & 1) + dx], acc[4 * g + u][p]);
                    }
                }
            }
        }
    }

    // bias, ReLU, pooling, store
    if (live) {
        const int so = a.pool ? half : side;
        float *out = a.Hout + ((int64_t)c * a.n_r + j0 + ls) * a.cout * so * so;
#pragma unroll
        for (int o = 0; o < kCnnCo; ++o) {
            if (co0 + o >= a.cout) break;
            float bias = 0.f;
            if (a.offB >= 0) {
                const float bx = load_elem(static_cast<const T *>(a.x) + a.offB + co0 + o);
                const float bv = has_v ? load_elem(vrow + a.offB + co0 + o) : 0.f;
                bias = candidate_param<T>(bx, bv, a.gamma);
            }
            float z[4];
#pragma unroll
            for (int p = 0; p < 4; ++p) z[p] = relu_keep_nan(acc[o][p] + bias);
            float *op = out + (int64_t)(co0 + o) * so * so;
            if (a.pool) {
                op[qy * so + qx] = max_nan(max_nan(z[0], z[1]), max_nan(z[2], z[3]));
            } else {
                *reinterpret_cast<float2 *>(op + (2 * qy) * so + 2 * qx) = make_float2(z[0], z[1]);
                *reinterpret_cast<float2 *>(op + (2 * qy + 1) * so + 2 * qx) = make_float2(z[2], z[3]);
            }
        }
    }
    // ||v||^2 of this block's planes' weights and biases: one slot per warp
    if (count_norm) {
        if (a.offB >= 0 && tid < kCnnCo && co0 + tid < a.cout) {
            const float bv = load_elem(vrow + a.offB + co0 + tid);
            nrm = fmaf(bv, bv, nrm);
        }
#pragma unroll
        for (int sft = 16; sft >= 1; sft >>= 1) nrm += __shfl_xor_sync(0xffffffffu, nrm, sft);
        if (lane == 0)
            a.normpart[(int64_t)(c - 1) * a.np_slots + a.np_base + blockIdx.x * (kCnnThreads / 32) + warp] = nrm;
    }
}

}  // namespace

// planes of up to 32 x 32 with an even side
bool cnn_side_ok(int side) { return side >= 2 && side <= 32 && (side & 1) == 0; }
int cnn_norm_slots(int cout) { return ((cout + kCnnCo - 1) / kCnnCo) * (kCnnThreads / 32); }

cudaError_t launch_cnn_conv(Context &c, const CnnLayerArgs &a, cudaStream_t s, int *launches) {
    ++*launches;
    profile_mark(c, "cnn_conv3x3", s);
    const size_t smem = cnn_smem_bytes(a.side);
    const int spb = cnn_samples_per_block(a.side);
    const dim3 grid((a.cout + kCnnCo - 1) / kCnnCo, (a.n_r + spb - 1) / spb, a.m + 1);
    static PerDeviceOnce attr_set;
    if (attr_set.need(c.device)) {
        size_t most = 0;
        for (int side = 2; side <= 32; side += 2)
            if (cnn_smem_bytes(side) > most) most = cnn_smem_bytes(side);
        cudaError_t e = cudaFuncSetAttribute(cnn_conv3x3_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(cnn_conv3x3_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)most);
        if (e != cudaSuccess) return e;
        attr_set.mark(c.device);
    }
    if (c.desc.param_dtype == ZENO_BF16)
        return launch_chained(cnn_conv3x3_kernel<__nv_bfloat16>, grid, dim3(kCnnThreads), smem, s, chain_launches(c), a);
    return launch_chained(cnn_conv3x3_kernel<float>, grid, dim3(kCnnThreads), smem, s, chain_launches(c), a);
}

}  // namespace zeno
