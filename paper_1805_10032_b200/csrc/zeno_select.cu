// Definition 3, the ranking: the m - b candidates with the highest scores, in rank order.
//
// One thread block sorts m <= 1024 (score, index) pairs with a bitonic network.  Each pair is
// packed into one 64-bit key whose unsigned order is "higher score first, then lower index":
// the score's bit pattern is mapped to an order-preserving unsigned integer (NaN and minus
// infinity share the lowest real key, -0 is folded into +0) and the index is stored
// complemented in the low half.  Compare-exchange steps between lanes of a warp use shuffles;
// steps across warps go through shared memory.
#include "zeno_internal.h"

namespace zeno {

namespace {

__global__ void __launch_bounds__(1024) select_kernel(const float *scores, int m, int keep,
                                                       int32_t *idx) {
    __shared__ unsigned long long keys[ZENO_MAX_CANDIDATES];
    const int t = threadIdx.x;
    const int n = blockDim.x;            // power of two >= max(m, 32)
    // padding keys are 0: below every real key (a real key has a non-zero low half or high half)
    unsigned long long key = t < m ? rank_key(scores[t], t) : 0ull;

    // bitonic sort, descending
    for (int size = 2; size <= n; size <<= 1) {
        for (int stride = size >> 1; stride >= 1; stride >>= 1) {
            unsigned long long other;
            if (stride >= 32) {
                keys[t] = key;
                __syncthreads();
                other = keys[t ^ stride];
                __syncthreads();
            } else {
                other = __shfl_xor_sync(0xffffffffu, key, stride);
            }
            const bool descending_block = (t & size) == 0;
            const bool lower_lane = (t & stride) == 0;
            // in a descending block the lower lane keeps the larger key
            const bool keep_max = descending_block == lower_lane;
            key = keep_max ? (key > other ? key : other) : (key < other ? key : other);
        }
    }
    if (t < keep) idx[t] = (int32_t)(0xffffffffu - (unsigned)(key & 0xffffffffull));
}

}  // namespace

cudaError_t launch_select(Context &c, const float *scores, int m, int b, int32_t *idx,
                          cudaStream_t s, int *launches) {
    int n = 32;
    while (n < m) n <<= 1;
    ++*launches;
    profile_mark(c, "select", s);
    select_kernel<<<1, n, 0, s>>>(scores, m, m - b, idx);
    return cudaGetLastError();
}

}  // namespace zeno
