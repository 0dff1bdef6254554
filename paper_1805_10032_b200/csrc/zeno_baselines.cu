// The paper's baseline aggregation rules on the same candidate matrix V (Experiments, "Baselines"):
// the marginal Median and Krum_b.  They share Zeno's inputs and storage types, so a caller can compare
// the three rules on the same step.
//
// Median: out[j] = the one-dimensional median of column j (the middle value of the m sorted entries, the
// mean of the two middle ones for even m; a NaN entry counts as plus infinity).  One pass over V.  Up to
// 64 candidates a thread keeps its column in registers and sorts it with a bitonic network (padded with
// plus infinity, which leaves the middle ranks where they are); beyond that the block keeps a tile of
// columns in shared memory and every thread sorts its own column there.
//
// Krum: the squared distances ||v_i - v_j||^2 of all pairs, taken as sums of squared differences (not
// from a Gram matrix: two honest candidates may differ by far less than their norms), then for every
// candidate the sum over its m - b - 2 nearest neighbours, the arg min of those sums, and a copy of the
// winning row.  The pair sums are accumulated per block and group of threads over their share of the
// columns and added up afterwards in a fixed order, so the result does not depend on scheduling.
#include <math.h>

#include "zeno_internal.h"

namespace zeno {

namespace {

__device__ __forceinline__ float nan_to_inf(float v) { return v != v ? INFINITY : v; }

template <int N>
__device__ __forceinline__ void bitonic_sort_regs(float (&a)[N]) {
#pragma unroll
    for (int k = 2; k <= N; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
#pragma unroll
            for (int i = 0; i < N; ++i) {
                const int l = i ^ j;
                if (l > i) {
                    const bool up = (i & k) == 0;
                    const float lo = fminf(a[i], a[l]), hi = fmaxf(a[i], a[l]);
                    a[i] = up ? lo : hi;
                    a[l] = up ? hi : lo;
                }
            }
        }
    }
}

// the median of the m smallest entries of an ascending array (entries m.. are padding)
template <int N>
__device__ __forceinline__ float middle_of(const float (&a)[N], int m) {
    float lo = 0.f, hi = 0.f;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        if (i == (m - 1) / 2) lo = a[i];
        if (i == m / 2) hi = a[i];
    }
    return (m & 1) ? lo : 0.5f * lo + 0.5f * hi;
}

// One column per thread, the column in registers (m <= N).
template <typename T, int N>
__global__ void __launch_bounds__(128) median_regs_kernel(const T *V, int64_t ldv, int64_t d, int m, float *out) {
    pdl_wait();
    pdl_launch_dependents();
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < d; j += (int64_t)gridDim.x * blockDim.x) {
        float a[N];
#pragma unroll
        for (int r = 0; r < N; ++r) a[r] = r < m ? nan_to_inf(load_elem(V + (int64_t)r * ldv + j)) : INFINITY;
        bitonic_sort_regs<N>(a);
        out[j] = middle_of<N>(a, m);
    }
}

// A tile of `cols` columns in shared memory, [np][cols] with np the power of two >= m; thread t sorts
// column t (its own: no synchronisation, and neighbouring threads touch neighbouring banks).
template <typename T>
__global__ void __launch_bounds__(128) median_smem_kernel(const T *V, int64_t ldv, int64_t d, int m, int np, int cols,
                                                          float *out) {
    extern __shared__ float tile[];
    pdl_wait();
    pdl_launch_dependents();
    const int t = threadIdx.x;
    for (int64_t j0 = (int64_t)blockIdx.x * cols; j0 < d; j0 += (int64_t)gridDim.x * cols) {
        const int64_t j = j0 + t;
        if (t < cols && j < d) {
            for (int r = 0; r < np; ++r) tile[r * cols + t] = r < m ? nan_to_inf(load_elem(V + (int64_t)r * ldv + j)) : INFINITY;
            for (int k = 2; k <= np; k <<= 1)
                for (int s = k >> 1; s > 0; s >>= 1)
                    for (int i = 0; i < np; ++i) {
                        const int l = i ^ s;
                        if (l > i) {
                            const bool up = (i & k) == 0;
                            const float x = tile[i * cols + t], y = tile[l * cols + t];
                            const float lo = fminf(x, y), hi = fmaxf(x, y);
                            tile[i * cols + t] = up ? lo : hi;
                            tile[l * cols + t] = up ? hi : lo;
                        }
                    }
            const float lo = tile[((m - 1) / 2) * cols + t], hi = tile[(m / 2) * cols + t];
            out[j] = (m & 1) ? lo : 0.5f * lo + 0.5f * hi;
        }
    }
}

// ---- Krum -----------------------------------------------------------------------------------

constexpr int kKrumThreads = 256;
constexpr int kKrumCols = 64;                 // columns staged per tile
constexpr int kKrumPitch = kKrumCols + 1;     // row pitch in floats: rows of a tile start in different banks

__host__ __device__ inline int krum_row_blocks(int m) { return (m + 3) / 4; }
__host__ __device__ inline int krum_tiles(int m) { const int mb = krum_row_blocks(m); return mb * (mb + 1) / 2; }
// groups of threads that share the pair tiles and split a tile's columns between them
__host__ __device__ inline int krum_groups(int m) { const int t = krum_tiles(m); return t >= kKrumThreads ? 1 : kKrumThreads / t; }

// part[block][group][tile][4][4]: sums of squared differences of the 4 x 4 pairs (i, j) of a tile over
// the columns this block and group took.  Tiles are the (ib <= jb) blocks of four rows.
template <typename T>
__global__ void __launch_bounds__(kKrumThreads) krum_pairs_kernel(const T *V, int64_t ldv, int64_t d, int m, float *part) {
    extern __shared__ float rows[];           // [m rounded up to 4][kKrumPitch]
    pdl_wait();
    pdl_launch_dependents();
    const int mb = krum_row_blocks(m), tiles = krum_tiles(m), groups = krum_groups(m);
    const int m4 = mb * 4;
    const int tid = threadIdx.x;
    const int group = tid / tiles < groups ? tid / tiles : -1;      // threads beyond groups * tiles idle (tiles < 256)
    // tile index -> (ib, jb) with ib <= jb, row by row of the upper triangle
    auto tile_of = [&](int t, int &ib, int &jb) {
        ib = 0;
        int left = t;
        while (left >= mb - ib) { left -= mb - ib; ++ib; }
        jb = ib + left;
    };
    const int n_mine = tiles >= kKrumThreads ? (tiles - tid + kKrumThreads - 1) / kKrumThreads : (group >= 0 ? 1 : 0);
    constexpr int kMaxMine = 3;               // tiles per thread: 528 tiles (m = 128) over 256 threads
    float acc[kMaxMine][16];
#pragma unroll
    for (int q = 0; q < kMaxMine; ++q)
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[q][e] = 0.f;
    for (int64_t j0 = (int64_t)blockIdx.x * kKrumCols; j0 < d; j0 += (int64_t)gridDim.x * kKrumCols) {
        __syncthreads();
        for (int t = tid; t < m4 * kKrumCols; t += kKrumThreads) {
            const int r = t / kKrumCols, c = t - r * kKrumCols;
            rows[r * kKrumPitch + c] = (r < m && j0 + c < d) ? load_elem(V + (int64_t)r * ldv + j0 + c) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kMaxMine; ++q) {
            if (q >= n_mine) break;
            const int tile = tiles >= kKrumThreads ? tid + q * kKrumThreads : tid - group * tiles;
            int ib, jb;
            tile_of(tile, ib, jb);
            const float *ri = rows + ib * 4 * kKrumPitch, *rj = rows + jb * 4 * kKrumPitch;
            const int c0 = tiles >= kKrumThreads ? 0 : group, cs = tiles >= kKrumThreads ? 1 : groups;
            for (int c = c0; c < kKrumCols; c += cs) {
                float a[4], b[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    a[u] = ri[u * kKrumPitch + c];
                    b[u] = rj[u * kKrumPitch + c];
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const float df = a[u] - b[w];
                        acc[q][u * 4 + w] = fmaf(df, df, acc[q][u * 4 + w]);
                    }
            }
        }
    }
#pragma unroll
    for (int q = 0; q < kMaxMine; ++q) {
        if (q >= n_mine) break;
        const int tile = tiles >= kKrumThreads ? tid + q * kKrumThreads : tid - group * tiles;
        const int g = tiles >= kKrumThreads ? 0 : group;
        float *dst = part + (((int64_t)blockIdx.x * groups + g) * tiles + tile) * 16;
#pragma unroll
        for (int e = 0; e < 16; e += 4) *reinterpret_cast<float4 *>(dst + e) = make_float4(acc[q][e], acc[q][e + 1], acc[q][e + 2], acc[q][e + 3]);
    }
}

// One block.  dist[i][j] from the partial sums (added in block, group order, in double); for every
// candidate the sum of its m - b - 2 smallest distances to the others (ascending, as a sorted sum);
// the arg min, lowest index first.  A NaN distance counts as plus infinity.
__global__ void __launch_bounds__(1024) krum_finish_kernel(const float *part, int slabs, int m, int b, float *sums_out,
                                                           int32_t *k_out, float *sums_ws) {
    extern __shared__ float dist[];           // [m][m + 1]
    const int mb = krum_row_blocks(m), tiles = krum_tiles(m);
    const int pitch = m + 1;
    for (int t = threadIdx.x; t < tiles * 16; t += blockDim.x) {
        const int tile = t >> 4, e = t & 15;
        int ib = 0, left = tile;
        while (left >= mb - ib) { left -= mb - ib; ++ib; }
        const int jb = ib + left;
        const int i = ib * 4 + (e >> 2), j = jb * 4 + (e & 3);
        if (i < m && j < m) {
            double s = 0.0;
            for (int q = 0; q < slabs; ++q) s += (double)part[((int64_t)q * tiles + tile) * 16 + e];
            const float v = nan_to_inf((float)s);
            dist[i * pitch + j] = v;
            if (ib != jb) dist[j * pitch + i] = v;      // a diagonal tile holds both (i, j) and (j, i) itself
        }
    }
    __syncthreads();
    const int nn = m - b - 2;
    for (int i = threadIdx.x; i < m; i += blockDim.x) {
        unsigned used[ZENO_KRUM_MAX_M / 32];
#pragma unroll
        for (int w = 0; w < ZENO_KRUM_MAX_M / 32; ++w) used[w] = 0u;
        used[i >> 5] |= 1u << (i & 31);
        float s = 0.f;
        for (int t = 0; t < nn; ++t) {
            int best = -1;
            float bv = INFINITY;
            for (int j = 0; j < m; ++j) {
                if (used[j >> 5] & (1u << (j & 31))) continue;
                const float v = dist[i * pitch + j];
                if (best < 0 || v < bv) { best = j; bv = v; }
            }
            used[best >> 5] |= 1u << (best & 31);
            s += bv;
        }
        sums_ws[i] = s;
        if (sums_out) sums_out[i] = s;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int best = 0;
        for (int i = 1; i < m; ++i)
            if (sums_ws[i] < sums_ws[best]) best = i;
        *k_out = best;
    }
}

template <typename T>
__global__ void __launch_bounds__(256) copy_row_kernel(const T *V, int64_t ldv, int64_t d, int m, const int32_t *k, float *out) {
    const int row = *k;
    if (row < 0 || row >= m) return;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < d; j += (int64_t)gridDim.x * blockDim.x)
        out[j] = load_elem(V + (int64_t)row * ldv + j);
}

template <typename T>
cudaError_t launch_median_typed(Context &c, const T *V, int64_t ldv, int m, float *out, cudaStream_t s) {
    const int sms = c.sm_count > 0 ? c.sm_count : 148;
    const int64_t d = c.d;
    if (m <= 64) {
        int64_t want = (d + 127) / 128;
        const int64_t cap = (int64_t)sms * 32;
        const int blocks = (int)(want < cap ? (want < 1 ? 1 : want) : cap);
        if (m <= 32)
            return launch_chained(median_regs_kernel<T, 32>, dim3(blocks), dim3(128), 0, s, chain_launches(c), V, ldv, d, m, out);
        return launch_chained(median_regs_kernel<T, 64>, dim3(blocks), dim3(128), 0, s, chain_launches(c), V, ldv, d, m, out);
    }
    int np = 128;
    while (np < m) np <<= 1;
    const int cols = np <= 256 ? 128 : 32768 / np;            // 64 KB to 128 KB of shared memory per block
    const size_t smem = (size_t)np * cols * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(median_smem_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int64_t want = (d + cols - 1) / cols;
    const int64_t cap = (int64_t)sms * 4;
    const int blocks = (int)(want < cap ? (want < 1 ? 1 : want) : cap);
    return launch_chained(median_smem_kernel<T>, dim3(blocks), dim3(128), smem, s, chain_launches(c), V, ldv, d, m, np, cols, out);
}

template <typename T>
cudaError_t launch_krum_typed(Context &c, const T *V, int64_t ldv, int m, int b, float *out, int32_t *k, float *sums,
                              cudaStream_t s) {
    const int64_t d = c.d;
    const int tiles = krum_tiles(m), groups = krum_groups(m);
    int64_t want = (d + kKrumCols - 1) / kKrumCols;
    int blocks = (int)(want < c.krum_blocks ? want : c.krum_blocks);
    if (blocks < 1) blocks = 1;
    const size_t smem = (size_t)krum_row_blocks(m) * 4 * kKrumPitch * sizeof(float);
    krum_pairs_kernel<T><<<blocks, kKrumThreads, smem, s>>>(V, ldv, d, m, c.krum_part);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t fsmem = (size_t)m * (m + 1) * sizeof(float);
    e = cudaFuncSetAttribute(krum_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)fsmem);
    if (e != cudaSuccess) return e;
    krum_finish_kernel<<<1, 1024, fsmem, s>>>(c.krum_part, blocks * groups, m, b, sums, k, c.krum_sums);
    e = cudaGetLastError();
    if (e != cudaSuccess || !out) return e;
    const int sms = c.sm_count > 0 ? c.sm_count : 148;
    int64_t cw = (d + 255) / 256;
    const int cblocks = (int)(cw < (int64_t)sms * 8 ? (cw < 1 ? 1 : cw) : (int64_t)sms * 8);
    copy_row_kernel<T><<<cblocks, 256, 0, s>>>(V, ldv, d, m, k, out);
    return cudaGetLastError();
}

}  // namespace

// floats of pair partials for up to m candidates and `blocks` blocks
size_t krum_part_floats(int m, int blocks) { return (size_t)blocks * krum_groups(m) * krum_tiles(m) * 16; }

cudaError_t launch_median(Context &c, const void *V, int64_t ldv, int m, float *out, cudaStream_t s, int *launches) {
    ++*launches;
    profile_mark(c, "median", s);
    if (c.desc.param_dtype == ZENO_BF16) return launch_median_typed(c, static_cast<const __nv_bfloat16 *>(V), ldv, m, out, s);
    return launch_median_typed(c, static_cast<const float *>(V), ldv, m, out, s);
}

cudaError_t launch_krum(Context &c, const void *V, int64_t ldv, int m, int b, float *out, int32_t *k, float *sums,
                        cudaStream_t s, int *launches) {
    *launches += out ? 3 : 2;
    profile_mark(c, "krum", s);
    if (c.desc.param_dtype == ZENO_BF16)
        return launch_krum_typed(c, static_cast<const __nv_bfloat16 *>(V), ldv, m, b, out, k, sums, s);
    return launch_krum_typed(c, static_cast<const float *>(V), ldv, m, b, out, k, sums, s);
}

}  // namespace zeno
