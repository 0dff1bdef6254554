// Definition 3, the average: out[j] = (1/k) sum_{r<k} V[idx[r]][j], binary32 output.
//
// Pure streaming: only the k selected rows of V are read, each element once, with 16-byte
// loads when the rows allow it.  A thread owns one 16-byte column group and walks the k rows in
// batches, so several independent loads are in flight per thread and consecutive threads read
// consecutive addresses of the same row.  Rows are added in rank order, in binary32.
//
// With xu != NULL the same pass applies Algorithm 1's server update, xu[j] <- xu[j] - gamma out[j]
// (one fused multiply-add in binary32, rounded to the storage type of x), so that the step costs no
// further pass over x; out may then be NULL.
#include "zeno_internal.h"

namespace zeno {

namespace {

// How a 16-byte group is loaded: streaming (evict-first) loads for inputs of a few L2 capacities, plain
// read-only loads for larger ones (measured: 8-10 % apart in either direction on the two size classes).
enum class Load { kStreaming, kPlain };

template <typename T> struct Group;           // one 16-byte group of columns
template <> struct Group<float> {
    static constexpr int kElems = 4;
    __device__ static void add(const uint4 &t, float (&acc)[4]) {
        acc[0] += __uint_as_float(t.x); acc[1] += __uint_as_float(t.y);
        acc[2] += __uint_as_float(t.z); acc[3] += __uint_as_float(t.w);
    }
    __device__ static void unpack(const uint4 &t, float (&o)[4]) {
        o[0] = __uint_as_float(t.x); o[1] = __uint_as_float(t.y); o[2] = __uint_as_float(t.z); o[3] = __uint_as_float(t.w);
    }
    __device__ static void store(float *p, const float (&v)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
};
template <> struct Group<__nv_bfloat16> {
    static constexpr int kElems = 8;
    __device__ static void add(const uint4 &t, float (&acc)[8]) {
        const unsigned w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            acc[2 * q] += __uint_as_float(w[q] << 16);
            acc[2 * q + 1] += __uint_as_float(w[q] & 0xffff0000u);
        }
    }
    __device__ static void unpack(const uint4 &t, float (&o)[8]) {
        const unsigned w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            o[2 * q] = __uint_as_float(w[q] << 16);
            o[2 * q + 1] = __uint_as_float(w[q] & 0xffff0000u);
        }
    }
    __device__ static void store(__nv_bfloat16 *p, const float (&v)[8]) {
        uint4 t;
        unsigned *w = &t.x;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const __nv_bfloat162 pk = __floats2bfloat162_rn(v[2 * q], v[2 * q + 1]);
            w[q] = *reinterpret_cast<const unsigned *>(&pk);
        }
        *reinterpret_cast<uint4 *>(p) = t;
    }
};

template <Load L> __device__ __forceinline__ uint4 load_group(const void *p) {
    return L == Load::kStreaming ? __ldcs(reinterpret_cast<const uint4 *>(p)) : __ldg(reinterpret_cast<const uint4 *>(p));
}

// rows_s[r] = element offset of selected row r, or -1 for an index outside [0, m)
__device__ __forceinline__ void stage_rows(const int32_t *idx, int k, int m, int64_t ldv,
                                           int64_t *rows_s) {
    for (int r = threadIdx.x; r < k; r += blockDim.x) {
        int i = idx[r];
        rows_s[r] = (i >= 0 && i < m) ? (int64_t)i * ldv : -1;
    }
    __syncthreads();
}

// x is read and written in this file, so it is read with ordinary loads (the read-only path is for data
// nobody writes while the kernel runs).
__device__ __forceinline__ float load_param(const float *p) { return *p; }
__device__ __forceinline__ float load_param(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ __forceinline__ void store_param(float *p, float v) { *p = v; }
__device__ __forceinline__ void store_param(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// B rows are in flight per thread: all B loads of a batch are issued, raw, before the first is
// converted and added (a conversion between the loads would make each wait for the one before).
// A row that is not to be added (beyond k, or an index outside [0, m)) is read from row 0 instead,
// so that the load needs no branch, and its value is dropped.
template <typename T, int B, Load L>
__global__ void __launch_bounds__(256) aggregate_vec_kernel(const T *V, int64_t ldv, int64_t d, int m,
                                                             const int32_t *idx, int k, float *out, T *xu,
                                                             float gamma) {
    constexpr int E = Group<T>::kElems;
    __shared__ int64_t rows_s[ZENO_MAX_CANDIDATES];
    pdl_wait();
    // With the in-place update the next kernel on the stream (the next step's first kernel, which reads x
    // through the read-only path) must not become resident before x is final: no early trigger then, the
    // dependents start when this grid has completed.
    if (!xu) pdl_launch_dependents();
    stage_rows(idx, k, m, ldv, rows_s);
    const int64_t groups = d / E;            // whole groups; the d % E tail columns follow below
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < groups;
         g += (int64_t)gridDim.x * blockDim.x) {
        float acc[E];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = 0.f;
        const T *col = V + g * E;
        for (int r = 0; r < k; r += B) {
            uint4 v[B];
            bool on[B];
#pragma unroll
            for (int q = 0; q < B; ++q) {
                const int64_t off = r + q < k ? rows_s[r + q] : -1;
                on[q] = off >= 0;
                v[q] = load_group<L>(col + (on[q] ? off : 0));
            }
#pragma unroll
            for (int q = 0; q < B; ++q)
                if (on[q]) Group<T>::add(v[q], acc);       // rank order, binary32
        }
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = acc[e] / (float)k;
        if (out) {
            float4 *o = reinterpret_cast<float4 *>(out + g * E);
#pragma unroll
            for (int q = 0; q < E / 4; ++q) o[q] = make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]);
        }
        if (xu) {                                // 16-byte aligned like the rows of V
            float xv[E];
            Group<T>::unpack(*reinterpret_cast<const uint4 *>(xu + g * E), xv);
#pragma unroll
            for (int e = 0; e < E; ++e) xv[e] = fmaf(-gamma, acc[e], xv[e]);
            Group<T>::store(xu + g * E, xv);
        }
    }
    // tail columns (fewer than one group), one per thread of block 0
    if (blockIdx.x == 0) {
        const int64_t j = groups * E + threadIdx.x;
        if (j < d) {
            float acc = 0.f;
            for (int r = 0; r < k; ++r) {
                int64_t off = rows_s[r];
                if (off >= 0) acc += load_elem(V + off + j);
            }
            acc = acc / (float)k;
            if (out) out[j] = acc;
            if (xu) store_param(xu + j, fmaf(-gamma, acc, load_param(xu + j)));
        }
    }
}

// Any ldv >= d, any d: one element per thread.
template <typename T>
__global__ void __launch_bounds__(256) aggregate_scalar_kernel(const T *V, int64_t ldv, int64_t d,
                                                                int m, const int32_t *idx, int k,
                                                                float *out, T *xu, float gamma) {
    __shared__ int64_t rows_s[ZENO_MAX_CANDIDATES];
    pdl_wait();
    // With the in-place update the next kernel on the stream (the next step's first kernel, which reads x
    // through the read-only path) must not become resident before x is final: no early trigger then, the
    // dependents start when this grid has completed.
    if (!xu) pdl_launch_dependents();
    stage_rows(idx, k, m, ldv, rows_s);
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < d;
         j += (int64_t)gridDim.x * blockDim.x) {
        float acc = 0.f;
        for (int r = 0; r < k; ++r) {
            int64_t off = rows_s[r];
            if (off >= 0) acc += load_elem(V + off + j);
        }
        acc = acc / (float)k;
        if (out) out[j] = acc;
        if (xu) store_param(xu + j, fmaf(-gamma, acc, load_param(xu + j)));
    }
}

template <typename T, int B>
cudaError_t launch_vec(const Context &c, int blocks, bool plain, const T *V, int64_t ldv, int m, const int32_t *idx,
                       int k, float *out, T *xu, float gamma, cudaStream_t s) {
    if (plain)
        return launch_chained(aggregate_vec_kernel<T, B, Load::kPlain>, dim3(blocks), dim3(256), 0, s, chain_launches(c),
                              V, ldv, c.d, m, idx, k, out, xu, gamma);
    return launch_chained(aggregate_vec_kernel<T, B, Load::kStreaming>, dim3(blocks), dim3(256), 0, s, chain_launches(c),
                          V, ldv, c.d, m, idx, k, out, xu, gamma);
}

template <typename T>
cudaError_t launch_typed(const Context &c, const T *V, int64_t ldv, int m, const int32_t *idx, int k,
                         float *out, T *xu, float gamma, bool aligned, cudaStream_t s) {
    const int sms = c.sm_count > 0 ? c.sm_count : 148;
    const int64_t d = c.d;
    constexpr int E = Group<T>::kElems;
    // two waves of resident blocks at most: small enough shares that the last wave ends evenly
    const int64_t cap = (int64_t)sms * 16;
    if (aligned) {
        const int64_t want = (d / E + 255) / 256;
        int blocks = (int)(want < cap ? want : cap);
        if (blocks < 1) blocks = 1;
        // selected rows of more than four L2 capacities: plain loads; below: streaming loads
        const bool plain = (double)k * (double)d * sizeof(T) > 4.0 * 126.0 * 1024 * 1024;
        // rows in flight per thread: the largest of 8, 6, 5, 4 that divides k (no ragged last batch), else 6
        if (k % 8 == 0) return launch_vec<T, 8>(c, blocks, plain, V, ldv, m, idx, k, out, xu, gamma, s);
        if (k % 6 == 0) return launch_vec<T, 6>(c, blocks, plain, V, ldv, m, idx, k, out, xu, gamma, s);
        if (k % 5 == 0) return launch_vec<T, 5>(c, blocks, plain, V, ldv, m, idx, k, out, xu, gamma, s);
        if (k % 4 == 0) return launch_vec<T, 4>(c, blocks, plain, V, ldv, m, idx, k, out, xu, gamma, s);
        return launch_vec<T, 6>(c, blocks, plain, V, ldv, m, idx, k, out, xu, gamma, s);
    }
    const int64_t want = (d + 255) / 256;
    int blocks = (int)(want < cap ? want : cap);
    if (blocks < 1) blocks = 1;
    return launch_chained(aggregate_scalar_kernel<T>, dim3(blocks), dim3(256), 0, s, chain_launches(c), V, ldv, d, m,
                          idx, k, out, xu, gamma);
}

}  // namespace

cudaError_t launch_aggregate(Context &c, const void *V, int64_t ldv, int m,
                             const int32_t *idx, int k, float *out, void *xu, float gamma, bool aligned,
                             cudaStream_t s, int *launches) {
    ++*launches;
    profile_mark(c, "aggregate", s);
    if (c.desc.param_dtype == ZENO_BF16)
        return launch_typed(c, static_cast<const __nv_bfloat16 *>(V), ldv, m, idx, k, out, static_cast<__nv_bfloat16 *>(xu),
                            gamma, aligned, s);
    return launch_typed(c, static_cast<const float *>(V), ldv, m, idx, k, out, static_cast<float *>(xu), gamma, aligned, s);
}

}  // namespace zeno
