// Candidate-model forward for the softmax-cross-entropy MLP (Definition 2: f_r(x) and
// f_r(x - gamma v_i) on the same n_r samples), CUDA-core path.
//
// One launch per dense layer evaluates that layer for all m+1 models at once (model 0 is x
// itself).  A warp owns kRowsPerWarp output rows of one model: its lanes stride the input
// index k, form w = x - gamma v in registers straight from the loads of x and V (the
// perturbed model never exists in memory), accumulate the n_r dot products and, in the same
// pass, the sum of squares of the V entries they touched (the rho ||v||^2 term).  The loads of
// the next 128 columns are issued before the current ones are consumed; the layer's input
// activations are staged through shared memory, double buffered.
//
// A small last layer (mlp_head_kernel) runs as one block per model and also evaluates the
// cross-entropy; the block that finishes last (a ticket, no waiting) then forms the scores and the
// ranking, so the whole tail of the scoring pass costs no extra launch.
#include "zeno_internal.h"
#include "zeno_tail.cuh"

namespace zeno {

namespace {

constexpr int kStageK = 256;   // k-extent of one shared-memory stage of the activations
constexpr int kIterK = 128;    // k-extent one warp consumes per inner iteration (32 lanes x 4)

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem, bool valid) {
    unsigned s = static_cast<unsigned>(__cvta_generic_to_shared(smem));
    int bytes = valid ? 16 : 0;  // 0 source bytes: the destination is zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

// Sum, over the 32 lanes, of each of N per-lane values; lane j (< N) ends up holding the total
// of value j.  Recursive halving: 31 shuffles for N = 32 instead of 160.
template <int N>
__device__ __forceinline__ float warp_transpose_reduce(float (&v)[N], int lane) {
    static_assert(N == 1 || N == 2 || N == 4 || N == 8 || N == 16 || N == 32, "N must be 2^k");
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
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
    return v;
}


// A lane's four k-indices inside a 128-wide block: vector path 4*lane + e (one 16-byte / 8-byte
// load); scalar path 32*e + lane (coalesced).
template <typename T, bool VEC>
__device__ __forceinline__ void load_row4(const T *row, int kbase, int lane, int K, float (&o)[4]) {
    if (VEC) {
        int k = kbase + 4 * lane;
        if (k < K) {  // K is a multiple of 4 on this path
            load_vec4(row + k, o);
        } else {
            o[0] = o[1] = o[2] = o[3] = 0.f;
        }
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int k = kbase + 32 * e + lane;
            o[e] = k < K ? load_elem(row + k) : 0.f;
        }
    }
}

template <typename T, int NRT, bool VEC>
__global__ void __launch_bounds__(kLayerWarps * 32, 1) mlp_layer_kernel(LayerArgs a) {
    constexpr int RB = kRowsPerWarp;
    extern __shared__ __align__(16) float smem_dyn[];
    float(*hs)[NRT][kStageK] = reinterpret_cast<float(*)[NRT][kStageK]>(smem_dyn);

    pdl_wait();
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int c = blockIdx.y;                    // model: 0 = x, 1+i = x - gamma v_i
    const int j0 = blockIdx.z * NRT;             // first sample of this tile
    const int row0 = (blockIdx.x * kLayerWarps + warp) * RB;
    const int K = a.in;
    const bool has_v = c > 0;

    const T *xw = static_cast<const T *>(a.x) + a.offW;
    const T *vw = static_cast<const T *>(a.V) + (has_v ? (int64_t)(c - 1) * a.ldv : 0) + a.offW;
    int orow[RB];                                // rows past the end are computed on a clamp and dropped
#pragma unroll
    for (int r = 0; r < RB; ++r) orow[r] = min(row0 + r, a.out - 1);
    const int n_valid = min(NRT, a.n_r - j0);

    float acc[RB][NRT];
    float nrm = 0.f;
#pragma unroll
    for (int r = 0; r < RB; ++r)
#pragma unroll
        for (int j = 0; j < NRT; ++j) acc[r][j] = 0.f;

    const int stages = (K + kStageK - 1) / kStageK;
    const int iters = (K + kIterK - 1) / kIterK;

    // ---- staging of the input activations ------------------------------------------------
    auto issue_stage = [&](int s) {
        float(*dst)[kStageK] = hs[s & 1];
        const int kb = s * kStageK;
        const float *hin = a.Hin + (int64_t)c * a.hin_cand_stride + (int64_t)j0 * K;
        if (VEC) {
            constexpr int kVecPerRow = kStageK / 4;
            for (int t = threadIdx.x; t < NRT * kVecPerRow; t += blockDim.x) {
                int j = t / kVecPerRow, kk = (t % kVecPerRow) * 4;
                bool ok = j < n_valid && kb + kk < K;
                const float *src = ok ? hin + (int64_t)j * K + kb + kk : a.Hin;
                cp_async16(&dst[j][kk], src, ok);
            }
        } else {
            for (int t = threadIdx.x; t < NRT * kStageK; t += blockDim.x) {
                int j = t / kStageK, kk = t % kStageK;
                bool ok = j < n_valid && kb + kk < K;
                dst[j][kk] = ok ? __ldg(hin + (int64_t)j * K + kb + kk) : 0.f;
            }
        }
        cp_async_commit();
    };

    // ---- the streamed operands: this iteration's x / v values, the next ones in flight ------
    float xc[RB][4], vc[RB][4];
    auto load_iter = [&](int g, float (&xo)[RB][4], float (&vo)[RB][4]) {
        const int kbase = g * kIterK;
#pragma unroll
        for (int r = 0; r < RB; ++r) {
            load_row4<T, VEC>(xw + (int64_t)orow[r] * K, kbase, lane, K, xo[r]);
            if (has_v) {
                load_row4<T, VEC>(vw + (int64_t)orow[r] * K, kbase, lane, K, vo[r]);
            } else {
                vo[r][0] = vo[r][1] = vo[r][2] = vo[r][3] = 0.f;
            }
        }
    };

    issue_stage(0);
    load_iter(0, xc, vc);
    for (int s = 0; s < stages; ++s) {
        if (s + 1 < stages) {
            issue_stage(s + 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const float(*h)[kStageK] = hs[s & 1];
#pragma unroll
        for (int it = 0; it < kStageK / kIterK; ++it) {
            const int g = s * (kStageK / kIterK) + it;
            if (g < iters) {
                float xn[RB][4], vn[RB][4];
                if (g + 1 < iters) load_iter(g + 1, xn, vn);
                float w[RB][4];
#pragma unroll
                for (int r = 0; r < RB; ++r) {
                    const bool live = row0 + r < a.out;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        w[r][e] = candidate_param<T>(xc[r][e], vc[r][e], a.gamma);
                        if (live) nrm = fmaf(vc[r][e], vc[r][e], nrm);
                    }
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
                if (g + 1 < iters) {
#pragma unroll
                    for (int r = 0; r < RB; ++r)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            xc[r][e] = xn[r][e];
                            vc[r][e] = vn[r][e];
                        }
                }
            }
        }
        __syncthreads();
    }

    // ---- epilogue: lane j collects sample j0 + j of each row --------------------------------
    const T *vrow_base = static_cast<const T *>(a.V) + (has_v ? (int64_t)(c - 1) * a.ldv : 0);
#pragma unroll
    for (int r = 0; r < RB; ++r) {
        float z = warp_transpose_reduce<NRT>(acc[r], lane);
        const int o = row0 + r;
        if (o < a.out && lane < n_valid) {
            if (a.offB >= 0) {
                float bx = load_elem(static_cast<const T *>(a.x) + a.offB + o);
                float bv = has_v ? load_elem(vrow_base + a.offB + o) : 0.f;
                z += candidate_param<T>(bx, bv, a.gamma);
            }
            if (a.relu) z = relu_keep_nan(z);
            a.Hout[((int64_t)c * a.n_r + j0 + lane) * a.out + o] = z;
        }
    }

    // partial ||v||^2 of the rows (and bias entries) this warp touched; one slot per warp
    if (has_v && blockIdx.z == 0) {
        if (a.offB >= 0 && lane < RB && row0 + lane < a.out) {
            float bv = load_elem(vrow_base + a.offB + row0 + lane);
            nrm = fmaf(bv, bv, nrm);
        }
        nrm = warp_sum(nrm);
        if (lane == 0)
            a.normpart[(int64_t)(c - 1) * a.np_slots + a.np_base + blockIdx.x * kLayerWarps + warp] = nrm;
    }
}

// The last layer when it is small (out <= 32 classes and n_r <= 32 samples, or out <= 16 and
// n_r <= 64): one block per model
// computes all of the model's logits, its cross-entropy, and -- in the block that finishes last --
// the scores and the ranking.  The block first forms w = x - gamma v for the layer's rows in
// shared memory (coalesced loads, v^2 accumulated on the way) next to the model's input
// activations; then warp q multiplies samples SPW q .. SPW q + SPW - 1 against all rows, lanes
// striding k.
template <typename T, int OUT_T, int SPW, bool VEC>
__global__ void __launch_bounds__(256, 1) mlp_head_kernel(LayerArgs a) {
    constexpr int KC = 512;                      // k-extent staged per pass
    constexpr int NS = 8 * SPW;                  // samples a block can hold
    extern __shared__ __align__(16) float smem_dyn[];
    float(*ws)[KC] = reinterpret_cast<float(*)[KC]>(smem_dyn);                  // [OUT_T][KC]
    float(*hs)[KC] = reinterpret_cast<float(*)[KC]>(smem_dyn + OUT_T * KC);     // [NS][KC]
    __shared__ float zl[32][NS + 1];

    // The weights are inputs of the whole call: unless this is the call's first kernel (what precedes it
    // on the stream may then still be producing x or V), they are read while the kernel that produces the
    // activations is still running.
    if (a.first_in_call) pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c = blockIdx.x;
    const int K = a.in;
    const bool has_v = c > 0;
    const T *xw = static_cast<const T *>(a.x) + a.offW;
    const T *vbase = static_cast<const T *>(a.V) + (has_v ? (int64_t)(c - 1) * a.ldv : 0);
    const T *vw = vbase + a.offW;
    const float *hin = a.Hin + (int64_t)c * a.hin_cand_stride;

    float acc[OUT_T][SPW];
#pragma unroll
    for (int o = 0; o < OUT_T; ++o)
#pragma unroll
        for (int q = 0; q < SPW; ++q) acc[o][q] = 0.f;
    float nrm = 0.f;
    // bias of the rows this lane ends up with after the reduction: requested now, used at the end
    constexpr int kBatches = OUT_T * SPW / 32;
    float bias_x[kBatches], bias_v[kBatches];
#pragma unroll
    for (int bi = 0; bi < kBatches; ++bi) {
        const int o = bi * (32 / SPW) + lane / SPW;
        const bool ok = a.offB >= 0 && o < a.out;
        bias_x[bi] = ok ? load_elem(static_cast<const T *>(a.x) + a.offB + o) : 0.f;
        bias_v[bi] = ok && has_v ? load_elem(vbase + a.offB + o) : 0.f;
    }

    // w = x - gamma v of the layer's rows for the chunk starting at kb (zero beyond the rows / K)
    auto stage_weights = [&](int kb) {
        if (VEC) {
            // all of a thread's loads are issued before the first is used
            constexpr int kPerThread = OUT_T * (KC / 4) / 256;
            float xv[kPerThread][4], vv[kPerThread][4];
#pragma unroll
            for (int u = 0; u < kPerThread; ++u) {
                const int t = threadIdx.x + u * 256;
                const int o = t / (KC / 4), kk = (t % (KC / 4)) * 4;
#pragma unroll
                for (int e = 0; e < 4; ++e) xv[u][e] = vv[u][e] = 0.f;
                if (o < a.out && kb + kk < K) {
                    load_vec4(xw + (int64_t)o * K + kb + kk, xv[u]);
                    if (has_v) load_vec4(vw + (int64_t)o * K + kb + kk, vv[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < kPerThread; ++u) {
                const int t = threadIdx.x + u * 256;
                const int o = t / (KC / 4), kk = (t % (KC / 4)) * 4;
                float w4[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    w4[e] = candidate_param<T>(xv[u][e], vv[u][e], a.gamma);
                    nrm = fmaf(vv[u][e], vv[u][e], nrm);
                }
                *reinterpret_cast<float4 *>(&ws[o][kk]) = make_float4(w4[0], w4[1], w4[2], w4[3]);
            }
        } else {
            for (int t = threadIdx.x; t < OUT_T * KC; t += 256) {
                const int o = t / KC, kk = t % KC;
                float w = 0.f;
                if (o < a.out && kb + kk < K) {
                    const float xv = load_elem(xw + (int64_t)o * K + kb + kk);
                    const float vv = has_v ? load_elem(vw + (int64_t)o * K + kb + kk) : 0.f;
                    w = candidate_param<T>(xv, vv, a.gamma);
                    nrm = fmaf(vv, vv, nrm);
                }
                ws[o][kk] = w;
            }
        }
    };
    // the model's input activations for the chunk (asynchronous copies on the vector path)
    auto stage_acts = [&](int kb) {
        if (VEC) {
            for (int t = threadIdx.x; t < NS * (KC / 4); t += 256) {
                const int j = t / (KC / 4), kk = (t % (KC / 4)) * 4;
                const bool ok = j < a.n_r && kb + kk < K;
                cp_async16(&hs[j][kk], ok ? hin + (int64_t)j * K + kb + kk : a.Hin, ok);
            }
            cp_async_commit();
        } else {
            for (int t = threadIdx.x; t < NS * KC; t += 256) {
                const int j = t / KC, kk = t % KC;
                hs[j][kk] = (j < a.n_r && kb + kk < K) ? __ldg(hin + (int64_t)j * K + kb + kk) : 0.f;
            }
        }
    };

    stage_weights(0);
    pdl_wait();
    pdl_launch_dependents();
    for (int kb = 0; kb < K; kb += KC) {
        if (kb > 0) __syncthreads();
        stage_acts(kb);                 // in flight while the weights are formed
        if (kb > 0) stage_weights(kb);
        if (VEC) cp_async_wait<0>();
        __syncthreads();
        // warp q: its SPW samples against every row; lane l takes k = 4l + 128 i
#pragma unroll 1
        for (int i = 0; i < KC / 128; ++i) {
            if (kb + i * 128 >= K) break;
            const int kk = i * 128 + 4 * lane;
            float4 h4[SPW];
#pragma unroll
            for (int q = 0; q < SPW; ++q) h4[q] = *reinterpret_cast<const float4 *>(&hs[warp * SPW + q][kk]);
#pragma unroll
            for (int o = 0; o < OUT_T; ++o) {
                const float4 w4 = *reinterpret_cast<const float4 *>(&ws[o][kk]);
#pragma unroll
                for (int q = 0; q < SPW; ++q) {
                    acc[o][q] = fmaf(w4.x, h4[q].x, acc[o][q]);
                    acc[o][q] = fmaf(w4.y, h4[q].y, acc[o][q]);
                    acc[o][q] = fmaf(w4.z, h4[q].z, acc[o][q]);
                    acc[o][q] = fmaf(w4.w, h4[q].w, acc[o][q]);
                }
            }
        }
    }

    // lane totals: 32 (row, sample) pairs at a time; lane l receives pair l of the batch
    constexpr int kRowsPerBatch = 32 / SPW;
#pragma unroll
    for (int ob = 0; ob < OUT_T; ob += kRowsPerBatch) {
        float v[32];
#pragma unroll
        for (int o = 0; o < kRowsPerBatch; ++o)
#pragma unroll
            for (int q = 0; q < SPW; ++q) v[o * SPW + q] = acc[ob + o][q];
        float z = warp_transpose_reduce<32>(v, lane);
        const int o = ob + lane / SPW, j = warp * SPW + lane % SPW;
        if (o < a.out && j < a.n_r) {
            if (a.offB >= 0) z += candidate_param<T>(bias_x[ob / kRowsPerBatch], bias_v[ob / kRowsPerBatch], a.gamma);
            if (a.relu) z = relu_keep_nan(z);
            zl[o][j] = z;
        }
    }
    // ||v||^2 of this layer's rows and bias entries: one slot per warp
    if (has_v) {
        if (a.offB >= 0 && threadIdx.x < a.out) {
            const float bv = load_elem(vbase + a.offB + threadIdx.x);
            nrm = fmaf(bv, bv, nrm);
        }
        nrm = warp_sum(nrm);
        if (lane == 0) a.normpart[(int64_t)(c - 1) * a.np_slots + a.np_base + warp] = nrm;
    }
    __syncthreads();
    if (has_v) block_norm_total(a.tail, c - 1);          // all layers' partials of this candidate
    if (warp == 0) {
        double l = 0.0;
        for (int j = lane; j < a.n_r; j += 32) {
            float zmax = -INFINITY;
            for (int o = 0; o < a.out; ++o) zmax = fmaxf(zmax, zl[o][j]);
            float se = 0.f;
            for (int o = 0; o < a.out; ++o) se += expf(zl[o][j] - zmax);   // a NaN logit makes se NaN
            int lab = a.labels[j];
            if (lab < 0 || lab >= a.out) lab = 0;
            l += (double)((zmax - zl[lab][j]) + logf(se));
        }
        l = warp_sum(l);
        if (lane == 0) {
            a.tail.loss_sum[c] = l;
            a.losses[c] = (float)(l / (double)a.n_r);
        }
    }
    if (take_last_ticket(a.tail.ticket, gridDim.x)) finalize_and_select(a.tail);
}

// Per model: mean over the samples of log-sum-exp(z) - z[label].  G blocks per model (block g takes
// the samples j = g, g + G, ..), one warp per sample, fixed summation order: the blocks leave their
// sums in loss_part and the last block to finish adds them up, model by model, before it runs the
// tail.  G = 1 for small problems: the block writes the model's loss itself.
__global__ void __launch_bounds__(256) mlp_loss_kernel(const float *logits, const int32_t *labels,
                                                        int n_r, int classes, float *losses, double *loss_part,
                                                        int G, TailArgs tail) {
    __shared__ double per_warp[8];
    pdl_wait();
    pdl_launch_dependents();
    const int c = blockIdx.x / G, g = blockIdx.x - c * G;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double mine = 0.0;
    for (int j = g + warp * G; j < n_r; j += 8 * G) {
        const float *z = logits + ((int64_t)c * n_r + j) * classes;
        float zmax = -INFINITY;
        for (int q = lane; q < classes; q += 32) zmax = fmaxf(zmax, z[q]);
#pragma unroll
        for (int s = 16; s >= 1; s >>= 1) zmax = fmaxf(zmax, __shfl_xor_sync(0xffffffffu, zmax, s));
        float se = 0.f;
        for (int q = lane; q < classes; q += 32) se += expf(z[q] - zmax);   // a NaN logit makes se NaN
        se = warp_sum(se);
        int lab = labels[j];
        if (lab < 0 || lab >= classes) lab = 0;
        mine += (double)((zmax - z[lab]) + logf(se));   // identical in every lane of the warp
    }
    if (lane == 0) per_warp[warp] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += per_warp[w];
        if (G == 1) {
            tail.loss_sum[c] = t;
            losses[c] = (float)(t / (double)n_r);
        } else {
            loss_part[blockIdx.x] = t;
        }
    }
    if (c > 0 && g == 0) block_norm_total(tail, c - 1);
    if (take_last_ticket(tail.ticket, gridDim.x)) {
        if (G > 1) {
            for (int i = threadIdx.x; i <= tail.m; i += blockDim.x) {
                double t = 0.0;
                for (int q = 0; q < G; ++q) t += __ldcg(loss_part + i * G + q);
                tail.loss_sum[i] = t;
                losses[i] = (float)(t / (double)n_r);
            }
            __threadfence();
            __syncthreads();
        }
        finalize_and_select(tail);
    }
}

template <typename T, bool VEC>
cudaError_t launch_layer_nrt(const LayerArgs &a, cudaStream_t s, bool overlap) {
    const int rows_per_block = kRowsPerWarp * kLayerWarps;
    auto go = [&](auto kernel, int nrt) {
        dim3 grid((a.out + rows_per_block - 1) / rows_per_block, a.m + 1, (a.n_r + nrt - 1) / nrt);
        const size_t smem = sizeof(float) * 2 * nrt * kStageK;
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 (int)smem);
            if (e != cudaSuccess) return e;
        }
        return launch_chained(kernel, grid, dim3(kLayerWarps * 32), smem, s, overlap, a);
    };
    if (a.n_r <= 8) return go(mlp_layer_kernel<T, 8, VEC>, 8);
    if (a.n_r <= 16) return go(mlp_layer_kernel<T, 16, VEC>, 16);
    return go(mlp_layer_kernel<T, 32, VEC>, 32);
}

}  // namespace

int mlp_norm_slots(int out) {
    const int rows_per_block = kRowsPerWarp * kLayerWarps;
    return (out + rows_per_block - 1) / rows_per_block * kLayerWarps;
}

// The cross-entropy can ride on the last layer's launch when one block sees all of a model's
// logits: every output row in one block, every sample in one tile.
bool mlp_can_fuse_loss(int out, int n_r) { return (out <= 32 && n_r <= 32) || (out <= 16 && n_r <= 64); }

template <typename T, bool VEC>
cudaError_t launch_head(const LayerArgs &a, cudaStream_t s, bool overlap) {
    auto go = [&](auto kernel, int out_t, int ns) {
        const size_t smem = sizeof(float) * (size_t)(out_t + ns) * 512;
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        return launch_chained(kernel, dim3(a.m + 1), dim3(256), smem, s, overlap, a);
    };
    if (a.n_r > 32) return go(mlp_head_kernel<T, 16, 8, VEC>, 16, 64);
    if (a.out <= 16) return go(mlp_head_kernel<T, 16, 4, VEC>, 16, 32);
    return go(mlp_head_kernel<T, 32, 4, VEC>, 32, 32);
}

cudaError_t launch_mlp_layer(Context &c, const LayerArgs &a, bool aligned, cudaStream_t s,
                             int *launches) {
    ++*launches;
    profile_mark(c, a.fuse_loss ? "mlp_head_loss_tail" : "mlp_layer", s);
    if (a.fuse_loss) {
        if (c.desc.param_dtype == ZENO_BF16)
            return aligned ? launch_head<__nv_bfloat16, true>(a, s, chain_launches(c)) : launch_head<__nv_bfloat16, false>(a, s, chain_launches(c));
        return aligned ? launch_head<float, true>(a, s, chain_launches(c)) : launch_head<float, false>(a, s, chain_launches(c));
    }
    if (c.desc.param_dtype == ZENO_BF16)
        return aligned ? launch_layer_nrt<__nv_bfloat16, true>(a, s, chain_launches(c))
                       : launch_layer_nrt<__nv_bfloat16, false>(a, s, chain_launches(c));
    return aligned ? launch_layer_nrt<float, true>(a, s, chain_launches(c)) : launch_layer_nrt<float, false>(a, s, chain_launches(c));
}

cudaError_t launch_mlp_loss(Context &c, const float *logits, const int32_t *labels, int n_r,
                            int m, int classes, float *losses, const TailArgs &tail, cudaStream_t s,
                            int *launches) {
    ++*launches;
    profile_mark(c, "mlp_loss_tail", s);
    // enough blocks to spread a large batch of wide logits over the SMs
    int G = 1;
    if ((int64_t)n_r * classes >= 16384) G = n_r >= 64 ? 8 : n_r >= 32 ? 4 : 2;
    return launch_chained(mlp_loss_kernel, dim3((m + 1) * G), dim3(256), 0, s, chain_launches(c), logits, labels, n_r,
                          classes, losses, c.loss_part, G, tail);
}

}  // namespace zeno
