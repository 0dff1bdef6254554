// The end of the scoring pass, run by whichever block finishes last (a ticket, no waiting):
// norms from their partial sums, Definition 2's score, and optionally Definition 3's ranking.
#pragma once

#include "zeno_internal.h"

namespace zeno {

// Called by ALL threads of a block.  Returns true in the block that took the last ticket, after
// making the other blocks' global writes visible to it.
__device__ __forceinline__ bool take_last_ticket(unsigned *ticket, unsigned n_blocks) {
    __shared__ bool is_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned t = atomicAdd(ticket, 1u);
        is_last = t == n_blocks - 1;
        if (is_last) *ticket = 0;          // ready for the next launch
    }
    __syncthreads();
    if (is_last) __threadfence();
    return is_last;
}

// Called by ALL threads of a block of at most 1024 threads, after the block's own partial sums
// are in global memory and a __syncthreads().  Adds candidate i's partial sums of v^2 over all
// layers in a fixed order (each lane's loads are issued eight at a time before they are added)
// and leaves the total in norm_tot[i].
__device__ __forceinline__ void block_norm_total(const TailArgs &t, int i) {
    __shared__ float warp_part[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    float nv = 0.f;
    for (int l = 0; l < t.used.layers; ++l) {
        const float *src = t.normpart + (int64_t)i * t.np_slots + t.used.base[l];
        const int count = t.used.count[l];
        for (int s0 = warp * 256; s0 < count; s0 += n_warps * 256) {
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int s = s0 + u * 32 + lane;
                v[u] = s < count ? __ldcg(src + s) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) nv += v[u];
        }
    }
#pragma unroll
    for (int sft = 16; sft >= 1; sft >>= 1) nv += __shfl_xor_sync(0xffffffffu, nv, sft);
    if (lane == 0) warp_part[warp] = nv;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
        for (int w = 0; w < n_warps; ++w) tot += warp_part[w];
        t.norm_tot[i] = tot;
    }
}

// One block, any size.  norms[i] = the per-candidate totals left by block_norm_total;
// scores[i] = f_0 - f_i - rho norms[i]; if keep > 0, idx[0..keep) = the candidates with the
// highest scores in rank order (bitonic sort of the packed keys in shared memory).
// The loss difference is formed in double from the models' loss sums (t.loss_sum), so that the
// score of a candidate whose loss is close to f_0 is not rounded twice to binary32 before the
// terms cancel; only the finished score is rounded.
__device__ __forceinline__ void finalize_and_select(const TailArgs &t) {
    __shared__ unsigned long long keys[ZENO_MAX_CANDIDATES];
    int n = 32;
    while (n < t.m) n <<= 1;
    const double s0 = __ldcg(t.loss_sum);
    const double inv_n = 1.0 / (double)t.n_r;
    for (int i = threadIdx.x; i < n; i += blockDim.x)
        if (i >= t.m) keys[i] = 0ull;      // padding: below every real key
    for (int i = threadIdx.x; i < t.m; i += blockDim.x) {
        const float nv = __ldcg(t.norm_tot + i);
        const float sc = (float)((s0 - __ldcg(t.loss_sum + 1 + i)) * inv_n - (double)t.rho * (double)nv);
        if (t.norms_out) t.norms_out[i] = nv;
        t.scores[i] = sc;
        keys[i] = rank_key(sc, i);
    }
    if (t.keep <= 0) return;
    __syncthreads();
    for (int size = 2; size <= n; size <<= 1) {
        for (int stride = size >> 1; stride >= 1; stride >>= 1) {
            for (int i = threadIdx.x; i < n; i += blockDim.x) {
                const int partner = i ^ stride;
                if (partner > i) {
                    const unsigned long long a = keys[i], b = keys[partner];
                    const bool descending = (i & size) == 0;
                    if ((a < b) == descending) {
                        keys[i] = b;
                        keys[partner] = a;
                    }
                }
            }
            __syncthreads();
        }
    }
    for (int i = threadIdx.x; i < t.keep; i += blockDim.x)
        t.idx[i] = (int32_t)(0xffffffffu - (unsigned)(keys[i] & 0xffffffffull));
}

}  // namespace zeno
