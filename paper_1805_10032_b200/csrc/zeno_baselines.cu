// The paper's baseline aggregation rules on the same candidate matrix V (Experiments, "Baselines"):
// the marginal Median and Krum_b.  They share Zeno's inputs and storage types, so a caller can compare
// the three rules on the same step.
//
// Median: out[j] = the one-dimensional median of column j (the middle value of the m sorted entries, the
// mean of the two middle ones for even m; a NaN entry counts as plus infinity).  One pass over V.  A
// column is sorted in registers by a bitonic network, 32 values a thread, padded with plus infinity
// (which leaves the middle ranks where they are); beyond 32 candidates 2, 4, .. 32 neighbouring lanes of
// a warp share a column and the network's long-range stages exchange values by shuffles.
//
// Krum: the squared distances ||v_i - v_j||^2 of all pairs, taken as sums of squared differences (not
// from a Gram matrix: two honest candidates may differ by far less than their norms), then for every
// candidate the sum over its m - b - 2 nearest neighbours, the arg min of those sums, and a copy of the
// winning row.  The pair sums are accumulated per block over its share of the columns and added up
// afterwards in a fixed order, so the result does not depend on scheduling.
#include <math.h>

#include "zeno_internal.h"

namespace zeno {

namespace {

__device__ __forceinline__ float nan_to_inf(float v) { return v != v ? INFINITY : v; }

constexpr int kMedianRegs = 32;               // values of a column one thread holds
constexpr int kMedianThreads = 128;

__host__ __device__ constexpr int ilog2(int v) { return v <= 1 ? 0 : 1 + ilog2(v >> 1); }

// Ascending sort of the R * TPC values that TPC neighbouring lanes hold, element e = t * R + i in
// register i of lane t, by the bitonic network in the form whose comparators all point the same way: a
// merge of blocks of k elements first compares every element with its mirror image in the block
// (e ^ (k - 1)), then halves the distance from k / 4 down.  Every index below is a constant once the
// loops are unrolled, so the values stay in registers; partners R or more elements away sit in another
// lane and come by shuffle.  With one lane a column, elements from NP on are padding (plus infinity at
// the top of an ascending network never moves), so comparators that touch them are left out.
template <int R, int TPC, int NP>
__device__ __forceinline__ void bitonic_sort_lanes(float (&a)[R], int t) {
    constexpr int kLogN = ilog2(R) + ilog2(TPC);
#pragma unroll
    for (int lk = 1; lk <= kLogN; ++lk) {
        const int k = 1 << lk;
        if (k > R) {                          // mirror partner: register R - 1 - i of lane t ^ (k / R - 1)
            const bool keep_min = (t & (k / (2 * R))) == 0;
            float o[R];
#pragma unroll
            for (int i = 0; i < R; ++i) o[i] = __shfl_xor_sync(0xffffffffu, a[R - 1 - i], k / R - 1);
#pragma unroll
            for (int i = 0; i < R; ++i) a[i] = keep_min ? fminf(a[i], o[i]) : fmaxf(a[i], o[i]);
        } else {
#pragma unroll
            for (int i = 0; i < R; ++i) {
                const int l = i ^ (k - 1);
                if (l > i && l < NP) {
                    const float lo = fminf(a[i], a[l]), hi = fmaxf(a[i], a[l]);
                    a[i] = lo;
                    a[l] = hi;
                }
            }
        }
#pragma unroll
        for (int lj = lk - 2; lj >= 0; --lj) {
            const int j = 1 << lj;
            if (j >= R) {
                const bool keep_min = (t & (j / R)) == 0;
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    const float o = __shfl_xor_sync(0xffffffffu, a[i], j / R);
                    a[i] = keep_min ? fminf(a[i], o) : fmaxf(a[i], o);
                }
            } else {
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    const int l = i ^ j;
                    if (l > i && l < NP) {
                        const float lo = fminf(a[i], a[l]), hi = fmaxf(a[i], a[l]);
                        a[i] = lo;
                        a[l] = hi;
                    }
                }
            }
        }
    }
}

// A warp takes 32 / TPC neighbouring columns at a time; lane = column * TPC + t holds rows t * R .. of it.
// With one lane a column the kernel is compiled for its number of candidates, NP = m: the padding, the
// row bounds and the ranks of the middle values are constants, and the comparators whose results the
// middle values do not depend on fall away with them.  With more lanes NP = R and m is an argument.
template <typename T, int TPC, int NP>
__global__ void __launch_bounds__(kMedianThreads, 4) median_kernel(const T *V, int64_t ldv, int64_t d, int m_arg, float *out) {
    constexpr int R = kMedianRegs, kCols = 32 / TPC;
    static_assert(TPC == 1 || NP == R, "padding is only left out when a lane holds the whole column");
    pdl_wait();
    pdl_launch_dependents();
    const int lane = threadIdx.x & 31, t = lane % TPC, c = lane / TPC;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int m = TPC == 1 ? NP : m_arg;
    const int p0 = (m - 1) / 2, p1 = m / 2;   // ranks of the middle values
    for (int64_t j0 = warp * kCols; j0 < d; j0 += warps * kCols) {
        const int64_t j = j0 + c;
        const bool live = j < d;
        float a[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const int row = t * R + i;
            a[i] = (i < NP && live && row < m) ? nan_to_inf(load_elem(V + (int64_t)row * ldv + j)) : INFINITY;
        }
        bitonic_sort_lanes<R, TPC, NP>(a, t);
        float lo = 0.f, hi = 0.f;
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            if (t * R + i == p0) lo = a[i];
            if (t * R + i == p1) hi = a[i];
        }
        if (TPC > 1) {
            lo = __shfl_sync(0xffffffffu, lo, (lane & ~(TPC - 1)) | (p0 / R));
            hi = __shfl_sync(0xffffffffu, hi, (lane & ~(TPC - 1)) | (p1 / R));
        }
        if (live && t == 0) out[j] = (m & 1) ? lo : 0.5f * lo + 0.5f * hi;
    }
}

// ---- Krum -----------------------------------------------------------------------------------

constexpr int kKrumThreads = 256;
constexpr int kKrumCols = 128;                // columns staged per tile
constexpr int kKrumPitch = kKrumCols + 1;     // row pitch in floats: rows of a tile start in different banks

__host__ __device__ inline int krum_row_blocks(int m) { return (m + 3) / 4; }
__host__ __device__ inline int krum_tiles(int m) { const int mb = krum_row_blocks(m); return mb * (mb + 1) / 2; }
// groups of threads that share the pair tiles and split a tile's columns between them
__host__ __device__ inline int krum_groups(int m) { const int t = krum_tiles(m); return t >= kKrumThreads ? 1 : kKrumThreads / t; }
// shared memory of the pair kernel: the staged rows, or the groups' sums when those need more
inline size_t krum_pairs_smem(int m) {
    const size_t rows = (size_t)krum_row_blocks(m) * 4 * kKrumPitch, red = (size_t)krum_groups(m) * krum_tiles(m) * 16;
    return (rows > red ? rows : red) * sizeof(float);
}

// tile index -> (ib, jb) with ib <= jb, row by row of the upper triangle of blocks of four rows
__device__ __forceinline__ void krum_tile_of(int tile, int mb, int &ib, int &jb) {
    ib = 0;
    int left = tile;
    while (left >= mb - ib) { left -= mb - ib; ++ib; }
    jb = ib + left;
}

// part[block][tile][4][4]: sums of squared differences of the 4 x 4 pairs (i, j) of a tile over the
// columns this block took.  With fewer tiles than threads, groups of threads split a staged tile's
// columns and their sums are added in group order before they are written.
// kMaxMine: pair tiles a thread may hold (1 while the tiles are fewer than the threads; 528 tiles at m = 128
// over 256 threads need 3).
template <typename T, int kMaxMine>
__global__ void __launch_bounds__(kKrumThreads, kMaxMine == 1 ? 4 : 3) krum_pairs_kernel(const T *V, int64_t ldv, int64_t d, int m, float *part) {
    extern __shared__ float rows[];           // [m rounded up to 4][kKrumPitch], then [groups][tiles][16]
    pdl_wait();
    pdl_launch_dependents();
    const int mb = krum_row_blocks(m), tiles = krum_tiles(m), groups = krum_groups(m);
    const int m4 = mb * 4;
    const int tid = threadIdx.x;
    const bool shared_tiles = tiles < kKrumThreads;                 // one tile a thread, groups of threads
    const int group = tid / tiles < groups ? tid / tiles : -1;      // threads beyond groups * tiles idle
    const int n_mine = shared_tiles ? (group >= 0 ? 1 : 0) : (tiles - tid + kKrumThreads - 1) / kKrumThreads;
    float acc[kMaxMine][16];
#pragma unroll
    for (int q = 0; q < kMaxMine; ++q)
#pragma unroll
        for (int e = 0; e < 16; ++e) acc[q][e] = 0.f;
    for (int64_t j0 = (int64_t)blockIdx.x * kKrumCols; j0 < d; j0 += (int64_t)gridDim.x * kKrumCols) {
        __syncthreads();
#pragma unroll 8
        for (int t = tid; t < m4 * kKrumCols; t += kKrumThreads) {
            const int r = t / kKrumCols, c = t - r * kKrumCols;
            rows[r * kKrumPitch + c] = (r < m && j0 + c < d) ? load_elem(V + (int64_t)r * ldv + j0 + c) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kMaxMine; ++q) {
            if (q >= n_mine) break;
            const int tile = shared_tiles ? tid - group * tiles : tid + q * kKrumThreads;
            int ib, jb;
            krum_tile_of(tile, mb, ib, jb);
            const float *ri = rows + ib * 4 * kKrumPitch, *rj = rows + jb * 4 * kKrumPitch;
            const int c0 = shared_tiles ? group : 0, cs = shared_tiles ? groups : 1;
#pragma unroll(kMaxMine == 1 ? 4 : 1)
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
    float *dst = part + (int64_t)blockIdx.x * tiles * 16;
    if (!shared_tiles) {
#pragma unroll
        for (int q = 0; q < kMaxMine; ++q) {
            if (q >= n_mine) break;
            float *o = dst + (tid + q * kKrumThreads) * 16;
#pragma unroll
            for (int e = 0; e < 16; e += 4) *reinterpret_cast<float4 *>(o + e) = make_float4(acc[q][e], acc[q][e + 1], acc[q][e + 2], acc[q][e + 3]);
        }
        return;
    }
    __syncthreads();                          // the staged rows are done with: the groups' sums take their place
    if (group >= 0) {
#pragma unroll
        for (int e = 0; e < 16; ++e) rows[tid * 16 + e] = acc[0][e];       // tid = group * tiles + tile
    }
    __syncthreads();
    for (int t = tid; t < tiles * 16; t += kKrumThreads) {
        float sum = 0.f;
        for (int g = 0; g < groups; ++g) sum += rows[g * tiles * 16 + t];
        dst[t] = sum;
    }
}

// dist[i][j] = the blocks' partial sums added in block order (in double), one warp an entry: lanes take
// every 32nd block and their sums meet in a fixed butterfly.  A NaN distance counts as plus infinity.
__global__ void __launch_bounds__(256) krum_reduce_kernel(const float *part, int slabs, int m, float *dist) {
    const int mb = krum_row_blocks(m), tiles = krum_tiles(m);
    const int lane = threadIdx.x & 31;
    const int entry = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    if (entry >= tiles * 16) return;
    const int tile = entry >> 4, e = entry & 15;
    int ib, jb;
    krum_tile_of(tile, mb, ib, jb);
    const int i = ib * 4 + (e >> 2), j = jb * 4 + (e & 3);
    if (i >= m || j >= m) return;
    double s = 0.0;
    for (int q = lane; q < slabs; q += 32) s += (double)part[(int64_t)q * tiles * 16 + entry];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
        const float v = nan_to_inf((float)s);
        dist[i * m + j] = v;
        if (ib != jb) dist[j * m + i] = v;    // a diagonal tile holds both (i, j) and (j, i) itself
    }
}

// One block.  For every candidate the sum of its m - b - 2 smallest distances to the others (ascending,
// as a sorted sum); the arg min, lowest index first.
__global__ void __launch_bounds__(128) krum_finish_kernel(const float *dist, int m, int b, float *sums_out, int32_t *k_out,
                                                          float *sums_ws) {
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
                const float v = dist[i * m + j];
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

template <typename T, int TPC, int NP>
cudaError_t launch_median_lanes(Context &c, const T *V, int64_t ldv, int m, float *out, cudaStream_t s) {
    const int sms = c.sm_count > 0 ? c.sm_count : 148;
    const int64_t d = c.d;
    const int per_block = (kMedianThreads / 32) * (32 / TPC);          // columns a block takes at a time
    const int64_t want = (d + per_block - 1) / per_block, cap = (int64_t)sms * 16;
    const int blocks = (int)(want < cap ? (want < 1 ? 1 : want) : cap);
    return launch_chained(median_kernel<T, TPC, NP>, dim3(blocks), dim3(kMedianThreads), 0, s, chain_launches(c), V, ldv, d, m, out);
}

// the one-lane kernel compiled for exactly m candidates, m = M, M - 1, .. 1
template <typename T, int M>
struct MedianOneLane {
    static cudaError_t launch(Context &c, const T *V, int64_t ldv, int m, float *out, cudaStream_t s) {
        if (m == M) return launch_median_lanes<T, 1, M>(c, V, ldv, m, out, s);
        return MedianOneLane<T, M - 1>::launch(c, V, ldv, m, out, s);
    }
};
template <typename T>
struct MedianOneLane<T, 0> {
    static cudaError_t launch(Context &, const T *, int64_t, int, float *, cudaStream_t) { return cudaErrorInvalidValue; }
};

template <typename T>
cudaError_t launch_median_typed(Context &c, const T *V, int64_t ldv, int m, float *out, cudaStream_t s) {
    constexpr int R = kMedianRegs;
    static_assert(R * 32 >= ZENO_MAX_CANDIDATES, "a warp holds the longest column");
    if (m <= R) return MedianOneLane<T, R>::launch(c, V, ldv, m, out, s);
    if (m <= R * 2) return launch_median_lanes<T, 2, R>(c, V, ldv, m, out, s);
    if (m <= R * 4) return launch_median_lanes<T, 4, R>(c, V, ldv, m, out, s);
    if (m <= R * 8) return launch_median_lanes<T, 8, R>(c, V, ldv, m, out, s);
    if (m <= R * 16) return launch_median_lanes<T, 16, R>(c, V, ldv, m, out, s);
    return launch_median_lanes<T, 32, R>(c, V, ldv, m, out, s);
}

template <typename T>
cudaError_t launch_krum_typed(Context &c, const T *V, int64_t ldv, int m, int b, float *out, int32_t *k, float *sums,
                              cudaStream_t s) {
    const int64_t d = c.d;
    const int sms = c.sm_count > 0 ? c.sm_count : 148;
    const int tiles = krum_tiles(m);
    const size_t smem = krum_pairs_smem(m);
    static PerDeviceOnce attr_set;
    if (attr_set.need(c.device)) {
        cudaError_t e = cudaFuncSetAttribute(krum_pairs_kernel<T, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)krum_pairs_smem(ZENO_KRUM_MAX_M));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(krum_pairs_kernel<T, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)krum_pairs_smem(ZENO_KRUM_MAX_M));
        if (e != cudaSuccess) return e;
        attr_set.mark(c.device);
    }
    // as many blocks as stay resident (shared memory, 2048 threads an SM), within what the partials were sized for
    int per_sm = (int)((200u << 10) / smem);
    per_sm = per_sm > 8 ? 8 : (per_sm < 1 ? 1 : per_sm);
    const int64_t want = (d + kKrumCols - 1) / kKrumCols;
    int blocks = per_sm * sms < c.krum_blocks ? per_sm * sms : c.krum_blocks;
    if (want < blocks) blocks = (int)(want < 1 ? 1 : want);
    if (tiles < kKrumThreads)
        krum_pairs_kernel<T, 1><<<blocks, kKrumThreads, smem, s>>>(V, ldv, d, m, c.krum_part);
    else
        krum_pairs_kernel<T, 3><<<blocks, kKrumThreads, smem, s>>>(V, ldv, d, m, c.krum_part);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    float *dist = c.krum_part + (size_t)c.krum_blocks * krum_tiles(c.m_max) * 16;     // m_max <= ZENO_KRUM_MAX_M here
    krum_reduce_kernel<<<(tiles * 16 + 7) / 8, 256, 0, s>>>(c.krum_part, blocks, m, dist);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    krum_finish_kernel<<<1, 128, 0, s>>>(dist, m, b, sums, k, c.krum_sums);
    e = cudaGetLastError();
    if (e != cudaSuccess || !out) return e;
    int64_t cw = (d + 255) / 256;
    const int cblocks = (int)(cw < (int64_t)sms * 8 ? (cw < 1 ? 1 : cw) : (int64_t)sms * 8);
    copy_row_kernel<T><<<cblocks, 256, 0, s>>>(V, ldv, d, m, k, out);
    return cudaGetLastError();
}

}  // namespace

// floats of Krum's workspace for up to m candidates and `blocks` blocks: the blocks' pair sums, then dist[m][m]
size_t krum_part_floats(int m, int blocks) { return (size_t)blocks * krum_tiles(m) * 16 + (size_t)m * m; }

cudaError_t launch_median(Context &c, const void *V, int64_t ldv, int m, float *out, cudaStream_t s, int *launches) {
    ++*launches;
    profile_mark(c, "median", s);
    if (c.desc.param_dtype == ZENO_BF16) return launch_median_typed(c, static_cast<const __nv_bfloat16 *>(V), ldv, m, out, s);
    return launch_median_typed(c, static_cast<const float *>(V), ldv, m, out, s);
}

cudaError_t launch_krum(Context &c, const void *V, int64_t ldv, int m, int b, float *out, int32_t *k, float *sums,
                        cudaStream_t s, int *launches) {
    *launches += out ? 4 : 3;
    profile_mark(c, "krum", s);
    if (c.desc.param_dtype == ZENO_BF16)
        return launch_krum_typed(c, static_cast<const __nv_bfloat16 *>(V), ldv, m, b, out, k, sums, s);
    return launch_krum_typed(c, static_cast<const float *>(V), ldv, m, b, out, k, sums, s);
}

}  // namespace zeno
