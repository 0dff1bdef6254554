// Scores for the least-squares loss f_r(x) = ||A x - y||^2 / (2 n_r) (Definition 2).
//
// The residual is linear in the parameters, A (x - gamma v_i) - y = (A x - y) - gamma A v_i,
// so one streaming pass computes the n_r-by-(m+1) products A [x, v_1 .. v_m] together with the
// squared norms of the rows of V.  Every element of A, x and V is read from HBM exactly once:
// a block owns a contiguous slab of the index k, stages the A-chunk of that slab in shared
// memory (cp.async, double buffered) and lets each warp stream kRowsPerWarp rows of [x; V]
// against it with per-lane register accumulators.  Per-slab partial sums are written out and
// combined in a fixed order (in double) by a one-block finishing kernel, which also forms the
// losses and the scores.
#include <mutex>

#include "zeno_internal.h"

namespace zeno {

namespace {

constexpr int kStageFloats = 8192;   // floats of A per shared-memory stage (32 KB)
constexpr int kIterK = 128;

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem, bool valid) {
    unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem));
    int bytes = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

template <int N>
__device__ __forceinline__ float warp_transpose_reduce(float (&v)[N], int lane) {
#pragma unroll
    for (int s = N / 2; s >= 1; s >>= 1) {
        const bool upper = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < s; ++i) {
            float send = upper ? v[i] : v[i + s];
            float keep = upper ? v[i + s] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
        }
    }
    float r = v[0];
#pragma unroll
    for (int s = N; s < 32; s <<= 1) r += __shfl_xor_sync(0xffffffffu, r, s);
    return r;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
    return v;
}

template <bool VEC>
__device__ __forceinline__ void load_row4(const float *row, int64_t kbase, int lane, int64_t K,
                                          float (&o)[4]) {
    if (VEC) {
        int64_t k = kbase + 4 * lane;
        if (k < K) {
            // streamed once: keep it out of L1
            float4 t = __ldcs(reinterpret_cast<const float4 *>(row + k));
            o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w;
        } else {
            o[0] = o[1] = o[2] = o[3] = 0.f;
        }
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int64_t k = kbase + 32 * e + lane;
            o[e] = k < K ? __ldcs(row + k) : 0.f;
        }
    }
}

// Warps per block: bounded by the register file (RB * NRT accumulators per lane; the
// register budget per thread is 65536 / threads with threads rounded up to 128).
template <int NRT, int RB> struct LsqShape {
    static constexpr int kMaxWarps = RB * NRT >= 128 ? 8 : (RB * NRT >= 96 ? 12 : 16);
};

// grid.x = slabs of k, grid.y = sets of rows (blockDim.x/32 warps x RB rows each),
// grid.z = tiles of NRT samples.  Row 0 is x, row 1+i is v_i.
template <int NRT, int RB, bool VEC>
__global__ void __launch_bounds__(LsqShape<NRT, RB>::kMaxWarps * 32, 1) lsq_stream_kernel(LsqArgs a) {
    constexpr int kStageK = kStageFloats / NRT;
    extern __shared__ __align__(16) float smem_dyn[];
    float(*as)[NRT][kStageK] = reinterpret_cast<float(*)[NRT][kStageK]>(smem_dyn);

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    const int rows = a.m + 1;
    const int row0 = (blockIdx.y * nwarps + warp) * RB;
    const int j0 = blockIdx.z * NRT;
    const int n_valid = min(NRT, a.n_r - j0);
    const int64_t K = a.d;

    const float *rowp[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        int rr = min(row0 + r, rows - 1);
        rowp[r] = rr == 0 ? a.x : a.V + (int64_t)(rr - 1) * a.ldv;
    }

    // this block's stages: [s_begin, s_end) of ceil(d / kStageK)
    const int64_t total = (K + kStageK - 1) / kStageK;
    const int64_t s_begin = total * blockIdx.x / gridDim.x;
    const int64_t s_end = total * (blockIdx.x + 1) / gridDim.x;

    float acc[RB][NRT];
    float nrm[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        nrm[r] = 0.f;
#pragma unroll
        for (int j = 0; j < NRT; ++j) acc[r][j] = 0.f;
    }

    auto issue_stage = [&](int64_t s, int buf) {
        float(*dst)[kStageK] = as[buf];
        const int64_t kb = s * kStageK;
        if (VEC) {
            constexpr int kVecPerRow = kStageK / 4;
            for (int t = threadIdx.x; t < NRT * kVecPerRow; t += blockDim.x) {
                int j = t / kVecPerRow, kk = (t % kVecPerRow) * 4;
                bool ok = j < n_valid && kb + kk < K;
                const float *src = ok ? a.A + (int64_t)(j0 + j) * K + kb + kk : a.A;
                cp_async16(&dst[j][kk], src, ok);
            }
        } else {
            for (int t = threadIdx.x; t < NRT * kStageK; t += blockDim.x) {
                int j = t / kStageK, kk = t % kStageK;
                bool ok = j < n_valid && kb + kk < K;
                dst[j][kk] = ok ? __ldg(a.A + (int64_t)(j0 + j) * K + kb + kk) : 0.f;
            }
        }
        cp_async_commit();
    };

    if (s_begin < s_end) issue_stage(s_begin, 0);
    for (int64_t s = s_begin; s < s_end; ++s) {
        const int buf = (int)((s - s_begin) & 1);
        if (s + 1 < s_end) {
            issue_stage(s + 1, buf ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const float(*h)[kStageK] = as[buf];
        if (row0 < rows) {
#pragma unroll 1
            for (int it = 0; it < kStageK / kIterK; ++it) {
                const int64_t kbase = s * kStageK + it * kIterK;
                if (kbase >= K) break;
                float w[RB][4];
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    load_row4<VEC>(rowp[r], kbase, lane, K, w[r]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) nrm[r] = fmaf(w[r][e], w[r][e], nrm[r]);
                }
#pragma unroll
                for (int j = 0; j < NRT; ++j) {
                    float hv[4];
                    if (VEC) {
                        float4 t = *reinterpret_cast<const float4 *>(&h[j][it * kIterK + 4 * lane]);
                        hv[0] = t.x; hv[1] = t.y; hv[2] = t.z; hv[3] = t.w;
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e) hv[e] = h[j][it * kIterK + 32 * e + lane];
                    }
#pragma unroll
                    for (int r = 0; r < RB; ++r)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[r][j] = fmaf(w[r][e], hv[e], acc[r][j]);
                }
            }
        }
        __syncthreads();
    }

    // part[slab][row][0..n_r) = partial A.row ; part[slab][row][n_r] = partial sum of squares
    const int stride = a.n_r + 1;
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        float z = warp_transpose_reduce<NRT>(acc[r], lane);
        float q = warp_sum(nrm[r]);
        const int rr = row0 + r;
        if (rr < rows) {
            float *dst = a.part + ((int64_t)blockIdx.x * rows + rr) * stride;
            if (lane < n_valid) dst[j0 + lane] = z;
            if (lane == 0 && blockIdx.z == 0) dst[a.n_r] = q;
        }
    }
}

// One block.  Sums the slab partials in slab order (double), then
//   residual r_j = (A x)_j - y_j,  f_0 = sum r_j^2 / (2 n_r),
//   f_i = sum (r_j - gamma (A v_i)_j)^2 / (2 n_r),  score_i = f_0 - f_i - rho ||v_i||^2.
__global__ void __launch_bounds__(1024) lsq_finish_kernel(const float *part, int slabs, int m,
                                                           int n_r, const float *y, float gamma,
                                                           float rho, float *losses, float *norms,
                                                           float *scores, float *sums /*[m+1][n_r+1]*/) {
    const int rows = m + 1, stride = n_r + 1;
    for (int t = threadIdx.x; t < rows * stride; t += blockDim.x) {
        double acc = 0.0;
        for (int s = 0; s < slabs; ++s) acc += (double)part[(int64_t)s * rows * stride + t];
        sums[t] = (float)acc;
    }
    __syncthreads();
    // the losses stay in double until the score is formed: f_0 - f_i cancels many digits
    __shared__ double f_s[ZENO_MAX_CANDIDATES + 1];
    for (int r = threadIdx.x; r < rows; r += blockDim.x) {
        double f = 0.0;
        for (int j = 0; j < n_r; ++j) {
            double res = (double)sums[j] - (double)y[j];
            if (r > 0) res -= (double)gamma * (double)sums[r * stride + j];
            f += res * res;
        }
        f_s[r] = f / (2.0 * n_r);
        losses[r] = (float)f_s[r];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < m; i += blockDim.x) {
        float nv = sums[(i + 1) * stride + n_r];
        if (norms) norms[i] = nv;
        scores[i] = (float)(f_s[0] - f_s[1 + i] - (double)rho * (double)nv);
    }
}

// The two halves of the finish for a parameter vector that is sharded over several GPUs by column slice:
// the sums are additive over slices (the residual is linear in the parameters), so every GPU adds up its
// own slab partials (in double, slab order), the sums of all GPUs are added by a collective in between,
// and the losses and scores follow from the total.
__global__ void __launch_bounds__(256) lsq_reduce_kernel(const float *part, int slabs, int n, double *sums) {
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < n; t += gridDim.x * blockDim.x) {
        double acc = 0.0;
        for (int s = 0; s < slabs; ++s) acc += (double)part[(int64_t)s * n + t];
        sums[t] = acc;
    }
}

__global__ void __launch_bounds__(1024) lsq_from_sums_kernel(const double *sums /*[m+1][n_r+1]*/, int m, int n_r,
                                                              const float *y, float gamma, float rho, float *losses,
                                                              float *norms, float *scores) {
    const int rows = m + 1, stride = n_r + 1;
    __shared__ double f_s[ZENO_MAX_CANDIDATES + 1];
    for (int r = threadIdx.x; r < rows; r += blockDim.x) {
        double f = 0.0;
        for (int j = 0; j < n_r; ++j) {
            double res = sums[j] - (double)y[j];
            if (r > 0) res -= (double)gamma * sums[r * stride + j];
            f += res * res;
        }
        f_s[r] = f / (2.0 * n_r);
        if (losses) losses[r] = (float)f_s[r];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < m; i += blockDim.x) {
        const double nv = sums[(i + 1) * stride + n_r];
        if (norms) norms[i] = (float)nv;
        scores[i] = (float)(f_s[0] - f_s[1 + i] - (double)rho * nv);
    }
}

template <int NRT, int RB, bool VEC>
cudaError_t launch_stream(const LsqArgs &a, cudaStream_t s) {
    const size_t smem = sizeof(float) * 2 * kStageFloats;
    auto kernel = lsq_stream_kernel<NRT, RB, VEC>;
    // the row groups are spread evenly over as few row sets as the warp limit allows
    const int groups = (a.m + 1 + RB - 1) / RB;
    const int row_sets = (groups + LsqShape<NRT, RB>::kMaxWarps - 1) / LsqShape<NRT, RB>::kMaxWarps;
    const int warps = (groups + row_sets - 1) / row_sets;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid(a.slabs, row_sets, (a.n_r + NRT - 1) / NRT);
    kernel<<<grid, warps * 32, smem, s>>>(a);
    return cudaGetLastError();
}

}  // namespace

int lsq_slab_count(const Context &c) {
    int s = c.sm_count > 0 ? c.sm_count : 148;
    return s < kMaxSlabs ? s : kMaxSlabs;
}

// The streaming pass over this handle's parameters: slab partials into a.part; *slabs_out slabs written.
static cudaError_t launch_lsq_pass(Context &c, const LsqArgs &a_in, bool aligned, int *slabs_out, cudaStream_t s,
                                   int *launches) {
    LsqArgs a = a_in;
    const int nrt = a.n_r <= 8 ? 8 : (a.n_r <= 16 ? 16 : 32);
    // small problems: no more slabs than there are stages of A
    const int64_t stages = (a.d + (kStageFloats / nrt) - 1) / (kStageFloats / nrt);
    int slabs = lsq_slab_count(c);
    if ((int64_t)slabs > stages) slabs = (int)stages;
    a.slabs = slabs;
    cudaError_t e;
    ++*launches;
    if (lsq_tc_usable(a, aligned) && c.use_tc) {
        // up to 64 candidates on aligned rows: the tensor-core stream (one slab per block)
        profile_mark(c, "lsq_tc", s);
        e = launch_lsq_tc(c, a, lsq_slab_count(c), &slabs, s);
    } else {
        profile_mark(c, "lsq_stream", s);
        if (nrt == 8)
            e = aligned ? launch_stream<8, 8, true>(a, s) : launch_stream<8, 8, false>(a, s);
        else if (nrt == 16)
            e = aligned ? launch_stream<16, 6, true>(a, s) : launch_stream<16, 6, false>(a, s);
        else
            e = aligned ? launch_stream<32, 4, true>(a, s) : launch_stream<32, 4, false>(a, s);
    }
    *slabs_out = slabs;
    return e;
}

cudaError_t launch_lsq_score(Context &c, const LsqArgs &a, const float *y, float gamma,
                             float rho, bool aligned, float *losses, float *norms, float *scores,
                             cudaStream_t s, int *launches) {
    int slabs = 0;
    cudaError_t e = launch_lsq_pass(c, a, aligned, &slabs, s, launches);
    if (e != cudaSuccess) return e;
    ++*launches;
    profile_mark(c, "lsq_finish", s);
    // the combined sums live behind the slab partials in the same workspace region
    const int rows = a.m + 1;
    float *sums = a.part + (int64_t)slabs * rows * (a.n_r + 1);
    lsq_finish_kernel<<<1, 1024, 0, s>>>(a.part, slabs, a.m, a.n_r, y, gamma, rho, losses, norms,
                                         scores, sums);
    return cudaGetLastError();
}

// This handle's slice of the sums: [m+1][n_r+1] doubles (row 0: A x, row 1 + c: A v_c; last column: ||v_c||^2).
cudaError_t launch_lsq_partial(Context &c, const LsqArgs &a, bool aligned, double *sums, cudaStream_t s,
                               int *launches) {
    int slabs = 0;
    cudaError_t e = launch_lsq_pass(c, a, aligned, &slabs, s, launches);
    if (e != cudaSuccess) return e;
    ++*launches;
    profile_mark(c, "lsq_reduce", s);
    const int n = (a.m + 1) * (a.n_r + 1);
    lsq_reduce_kernel<<<(n + 255) / 256, 256, 0, s>>>(a.part, slabs, n, sums);
    return cudaGetLastError();
}

cudaError_t launch_lsq_from_sums(Context &c, const double *sums, int m, int n_r, const float *y, float gamma,
                                 float rho, float *losses, float *norms, float *scores, cudaStream_t s,
                                 int *launches) {
    ++*launches;
    profile_mark(c, "lsq_from_sums", s);
    lsq_from_sums_kernel<<<1, 1024, 0, s>>>(sums, m, n_r, y, gamma, rho, losses, norms, scores);
    return cudaGetLastError();
}

}  // namespace zeno

// ---- scoring without any allocation -------------------------------------------------------
//
// The slab partials, the combined sums and the losses of zeno_score_lsq_static live in this
// array.  It is part of the library image: every GPU that loads the library carries it until
// the process exits.  Size: (slabs + 1) (m + 1) (n_r + 1) + (m + 1) floats with slabs <= 160,
// m <= ZENO_STATIC_MAX_M, n_r <= ZENO_STATIC_MAX_N_R -- about 1.4 MB.
namespace {

constexpr int kStaticMaxSlabs = 160;
constexpr size_t kStaticScratchFloats =
    (size_t)(kStaticMaxSlabs + 1) * (ZENO_STATIC_MAX_M + 1) * (ZENO_STATIC_MAX_N_R + 1) + (ZENO_STATIC_MAX_M + 1);

static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

using zeno::kMaxDevices;
float *g_static_scratch_ptr[kMaxDevices];      // device address of the array, per device
int g_static_sms[kMaxDevices];
bool g_static_ready[kMaxDevices];
std::mutex g_static_mutex;                     // host threads may make their first calls at the same time

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel can
// use: the device address is asked for once per device, with that device current.
cudaError_t static_scratch_setup(int device) {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_ready[device]) return cudaSuccess;
    float *ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_scratch);
    if (e != cudaSuccess) return e;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) return e;
    g_static_scratch_ptr[device] = ptr;
    g_static_sms[device] = sms;
    g_static_ready[device] = true;
    return cudaSuccess;
}

}  // namespace

extern "C" zeno_status zeno_score_lsq_static(int32_t device, const float *x, const float *V, int64_t ldv,
                                             int64_t d, int32_t m, const float *A, const float *y,
                                             int32_t n_r, float gamma, float rho, float *scores,
                                             float *losses, float *norms, void *stream) {
    if (device < 0 || device >= kMaxDevices) return ZENO_ERR_INVALID_ARG;
    if (!x || !V || !A || !y || !scores) return ZENO_ERR_INVALID_ARG;
    if (d < 1 || ldv < d || m < 1 || n_r < 1) return ZENO_ERR_INVALID_ARG;
    if (!isfinite(gamma) || !isfinite(rho) || rho < 0.f) return ZENO_ERR_INVALID_ARG;
    if (m > ZENO_STATIC_MAX_M || n_r > ZENO_STATIC_MAX_N_R) return ZENO_ERR_WORKSPACE;   // beyond the fixed scratch

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return ZENO_ERR_CUDA;
    if (prev != device && cudaSetDevice(device) != cudaSuccess) return ZENO_ERR_CUDA;
    zeno_status st = ZENO_OK;
    cudaError_t e = static_scratch_setup(device);
    if (e == cudaSuccess) {
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        zeno::LsqArgs a;
        a.x = x;
        a.V = V;
        a.ldv = ldv;
        a.d = d;
        a.A = A;
        a.n_r = n_r;
        a.m = m;
        a.part = g_static_scratch_ptr[device];
        const int rows = m + 1;
        const int nrt = n_r <= 8 ? 8 : (n_r <= 16 ? 16 : 32);
        const int64_t stages = (d + (zeno::kStageFloats / nrt) - 1) / (zeno::kStageFloats / nrt);
        int slabs = g_static_sms[device] > 0 ? g_static_sms[device] : 148;
        if (slabs > kStaticMaxSlabs) slabs = kStaticMaxSlabs;
        if ((int64_t)slabs > stages) slabs = (int)stages;
        a.slabs = slabs;
        const bool aligned = reinterpret_cast<uintptr_t>(x) % 16 == 0 && reinterpret_cast<uintptr_t>(V) % 16 == 0 &&
                             reinterpret_cast<uintptr_t>(A) % 16 == 0 && ldv % 4 == 0 && d % 4 == 0;
        if (nrt == 8)
            e = aligned ? zeno::launch_stream<8, 8, true>(a, s) : zeno::launch_stream<8, 8, false>(a, s);
        else if (nrt == 16)
            e = aligned ? zeno::launch_stream<16, 6, true>(a, s) : zeno::launch_stream<16, 6, false>(a, s);
        else
            e = aligned ? zeno::launch_stream<32, 4, true>(a, s) : zeno::launch_stream<32, 4, false>(a, s);
        if (e == cudaSuccess) {
            // Every partial the finishing kernel reads is rewritten by the stream kernel of the same
            // call, so nothing left over from an earlier call has to be cleared.
            float *sums = a.part + (int64_t)slabs * rows * (n_r + 1);
            float *loss_buf = losses ? losses : sums + (int64_t)rows * (n_r + 1);
            zeno::lsq_finish_kernel<<<1, 1024, 0, s>>>(a.part, slabs, m, n_r, y, gamma, rho, loss_buf, norms, scores,
                                                       sums);
            e = cudaGetLastError();
        }
    }
    if (e != cudaSuccess) st = ZENO_ERR_CUDA;
    if (prev != device) cudaSetDevice(prev);
    return st;
}

