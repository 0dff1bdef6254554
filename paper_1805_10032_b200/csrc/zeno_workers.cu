// The workers' side of Algorithm 1 on the device, so that a whole synchronous iteration (workers' gradients,
// failures, Zeno_b, update) can run on one GPU without a host round trip:
//   worker_grad_softmax_kernel / worker_grad_lsq_kernel   v_i = grad F_i(x) on worker i's own samples,
//                                                         for softmax regression and for least squares;
//                                                         a worker's labels may be flipped (the
//                                                         experiments' label-flipping failure);
//   inject_faults_kernel                                  the bit-flipping failure (negated gradient, the
//                                                         first faulty row copied over the others) and the
//                                                         failure model's scaled gradient eps * v.
// These kernels build the step's INPUT (the candidate matrix V); they are not on the scoring path.  One
// block per worker; the sizes they are meant for are the paper's (a hundred samples per worker, a model of
// a few thousand parameters).
#include <math.h>

#include "zeno_internal.h"

namespace zeno {

namespace {

constexpr int kWThreads = 256;
constexpr int kWMaxClasses = 32;

__device__ __forceinline__ float block_sum(float v, float *scratch) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < kWThreads / 32; ++w) t += scratch[w];
    return t;
}

template <typename T> __device__ __forceinline__ void store_elem(T *p, float v);
template <> __device__ __forceinline__ void store_elem<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void store_elem<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// Softmax regression, worker w = blockIdx.x: samples feats[w][n][in], labels[w][n].
//   delta[j][c] = (softmax(W a_j + b)[c] - [c == label_j]) / n;  dW[c][k] = sum_j delta[j][c] a_j[k];  db[c] = sum_j delta[j][c]
// dynamic shared memory: delta [n][classes].
template <typename T>
__global__ void __launch_bounds__(kWThreads) worker_grad_softmax_kernel(const T *x, int in, int classes, int has_bias,
                                                                         const float *feats, const int32_t *labels, int n,
                                                                         const int32_t *flip, T *V, int64_t ldv) {
    extern __shared__ float delta[];
    const int w = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float *a = feats + (int64_t)w * n * in;
    const int32_t *lab = labels + (int64_t)w * n;
    const bool flipped = flip != nullptr && flip[w] != 0;
    T *out = V + (int64_t)w * ldv;
    // logits: one warp per sample, lanes stride the input index
    for (int j = warp; j < n; j += kWThreads / 32) {
        float z[kWMaxClasses];
#pragma unroll
        for (int c = 0; c < kWMaxClasses; ++c) z[c] = 0.f;
        for (int k = lane; k < in; k += 32) {
            const float av = a[(int64_t)j * in + k];
#pragma unroll
            for (int c = 0; c < kWMaxClasses; ++c)
                if (c < classes) z[c] = fmaf(load_elem(x + (int64_t)c * in + k), av, z[c]);
        }
        float zmax = -INFINITY;
#pragma unroll
        for (int c = 0; c < kWMaxClasses; ++c) {
            if (c < classes) {
#pragma unroll
                for (int s = 16; s >= 1; s >>= 1) z[c] += __shfl_xor_sync(0xffffffffu, z[c], s);
                if (has_bias) z[c] += load_elem(x + (int64_t)classes * in + c);
                zmax = fmaxf(zmax, z[c]);
            }
        }
        float se = 0.f;
#pragma unroll
        for (int c = 0; c < kWMaxClasses; ++c)
            if (c < classes) se += expf(z[c] - zmax);
        int label = lab[j];
        if (flipped) label = classes - 1 - label;
        if (lane == 0) {
#pragma unroll
            for (int c = 0; c < kWMaxClasses; ++c)
                if (c < classes) delta[j * classes + c] = (expf(z[c] - zmax) / se - (c == label ? 1.f : 0.f)) / (float)n;
        }
    }
    __syncthreads();
    // dW: a thread per input index k, all classes in registers; samples in order
    for (int k = threadIdx.x; k < in; k += kWThreads) {
        float g[kWMaxClasses];
#pragma unroll
        for (int c = 0; c < kWMaxClasses; ++c) g[c] = 0.f;
        for (int j = 0; j < n; ++j) {
            const float av = a[(int64_t)j * in + k];
#pragma unroll
            for (int c = 0; c < kWMaxClasses; ++c)
                if (c < classes) g[c] = fmaf(delta[j * classes + c], av, g[c]);
        }
#pragma unroll
        for (int c = 0; c < kWMaxClasses; ++c)
            if (c < classes) store_elem(out + (int64_t)c * in + k, g[c]);
    }
    if (has_bias && threadIdx.x < classes) {
        float g = 0.f;
        for (int j = 0; j < n; ++j) g += delta[j * classes + threadIdx.x];
        store_elem(out + (int64_t)classes * in + threadIdx.x, g);
    }
}

// Least squares, worker w = blockIdx.x: A[w][n][d], y[w][n]:  r_j = a_j . x - y_j;  grad[k] = sum_j a_j[k] r_j / n.
// dynamic shared memory: r [n].
__global__ void __launch_bounds__(kWThreads) worker_grad_lsq_kernel(const float *x, int64_t d, const float *A, const float *y,
                                                                     int n, float *V, int64_t ldv) {
    extern __shared__ float r[];
    __shared__ float scratch[kWThreads / 32];
    const int w = blockIdx.x;
    const float *a = A + (int64_t)w * n * d;
    for (int j = 0; j < n; ++j) {
        float s = 0.f;
        for (int64_t k = threadIdx.x; k < d; k += kWThreads) s = fmaf(a[(int64_t)j * d + k], x[k], s);
        s = block_sum(s, scratch);
        if (threadIdx.x == 0) r[j] = s - y[(int64_t)w * n + j];
    }
    __syncthreads();
    float *out = V + (int64_t)w * ldv;
    for (int64_t k = threadIdx.x; k < d; k += kWThreads) {
        float g = 0.f;
        for (int j = 0; j < n; ++j) g = fmaf(a[(int64_t)j * d + k], r[j], g);
        out[k] = g / (float)n;
    }
}

// mode 0: V[faulty[f]] = -V[faulty[0]] for every f (the first faulty row is negated in place, after the
// others have copied it: blocks of columns are independent, a thread owns a column); mode 1: V[faulty[f]] *= eps.
template <typename T>
__global__ void __launch_bounds__(256) inject_faults_kernel(T *V, int64_t ldv, int64_t d, const int32_t *faulty, int n_faulty,
                                                            int m, int mode, float eps) {
    for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < d; k += (int64_t)gridDim.x * blockDim.x) {
        if (mode == 0) {
            const int f0 = faulty[0];
            if (f0 < 0 || f0 >= m) continue;
            const float v = -load_elem(V + (int64_t)f0 * ldv + k);
            for (int f = 0; f < n_faulty; ++f) {
                const int row = faulty[f];
                if (row >= 0 && row < m) store_elem(V + (int64_t)row * ldv + k, v);
            }
        } else {
            for (int f = 0; f < n_faulty; ++f) {
                const int row = faulty[f];
                if (row >= 0 && row < m) store_elem(V + (int64_t)row * ldv + k, eps * load_elem(V + (int64_t)row * ldv + k));
            }
        }
    }
}

}  // namespace

bool worker_gradients_supported(const Context &c, int n) {
    if (n < 1) return false;
    if (c.desc.kind == ZENO_LOSS_LEAST_SQUARES) return c.desc.param_dtype == ZENO_F32 && n <= 4096;
    if (c.desc.kind != ZENO_LOSS_SOFTMAX_MLP) return false;
    return c.desc.n_layers == 1 && c.desc.dims[1] <= kWMaxClasses && (int64_t)n * c.desc.dims[1] * 4 <= 48 * 1024;
}

cudaError_t launch_worker_gradients(Context &c, const void *x, const float *features, const void *targets, int n, int m,
                                    const int32_t *flip, void *V, int64_t ldv, cudaStream_t s, int *launches) {
    ++*launches;
    profile_mark(c, "worker_gradients", s);
    if (c.desc.kind == ZENO_LOSS_LEAST_SQUARES) {
        worker_grad_lsq_kernel<<<m, kWThreads, (size_t)n * sizeof(float), s>>>(static_cast<const float *>(x), c.d, features,
                                                                              static_cast<const float *>(targets), n,
                                                                              static_cast<float *>(V), ldv);
        return cudaGetLastError();
    }
    const int in = (int)c.desc.dims[0], classes = (int)c.desc.dims[1];
    const size_t smem = (size_t)n * classes * sizeof(float);
    if (c.desc.param_dtype == ZENO_BF16)
        worker_grad_softmax_kernel<__nv_bfloat16><<<m, kWThreads, smem, s>>>(static_cast<const __nv_bfloat16 *>(x), in, classes,
                                                                            c.desc.has_bias, features,
                                                                            static_cast<const int32_t *>(targets), n, flip,
                                                                            static_cast<__nv_bfloat16 *>(V), ldv);
    else
        worker_grad_softmax_kernel<float><<<m, kWThreads, smem, s>>>(static_cast<const float *>(x), in, classes, c.desc.has_bias,
                                                                    features, static_cast<const int32_t *>(targets), n, flip,
                                                                    static_cast<float *>(V), ldv);
    return cudaGetLastError();
}

cudaError_t launch_inject_faults(Context &c, void *V, int64_t ldv, int m, const int32_t *faulty, int n_faulty, int mode,
                                 float eps, cudaStream_t s, int *launches) {
    ++*launches;
    profile_mark(c, "inject_faults", s);
    const int sms = c.sm_count > 0 ? c.sm_count : 148;
    int64_t want = (c.d + 255) / 256;
    const int blocks = (int)(want < (int64_t)sms * 8 ? (want < 1 ? 1 : want) : (int64_t)sms * 8);
    if (c.desc.param_dtype == ZENO_BF16)
        inject_faults_kernel<<<blocks, 256, 0, s>>>(static_cast<__nv_bfloat16 *>(V), ldv, c.d, faulty, n_faulty, m, mode, eps);
    else
        inject_faults_kernel<<<blocks, 256, 0, s>>>(static_cast<float *>(V), ldv, c.d, faulty, n_faulty, m, mode, eps);
    return cudaGetLastError();
}

}  // namespace zeno
