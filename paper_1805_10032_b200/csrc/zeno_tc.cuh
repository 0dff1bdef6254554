// Device-side wrappers of the sm_100a instructions the tensor-core kernels are built from
// (mbarrier, bulk tensor copies, tcgen05 MMA / TMEM access), and the host-side tensor-map encoder.
#pragma once

#include <cuda.h>
#include <stdlib.h>
#include <string.h>

#include "zeno_internal.h"

namespace zeno {

// A block's abort state in shared memory: word 0 is the flag (zero until a wait gives up), word 1 the
// number of polls a wait may take, copied from the launch arguments.  The bounded waits get a pointer
// to word 0.
constexpr int kAbortWords = 2;

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// The polling part of a bounded wait, kept out of line so that the common case below stays a single
// probe (with the loop inlined, a wait on the MMA-issuing warp cost about 190 cycles even when the
// barrier's phase had already completed; a bare probe costs 15 to 20).
static __device__ __noinline__ bool mbar_wait_poll(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    const uint32_t limit = (uint32_t)abort_flag[1];
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 32) __nanosleep(40);
        if ((i & 127u) == 127u && *abort_flag) return false;
    }
    *abort_flag = (int)(0x40000000u | ((parity & 1u) << 20) | (bar & 0xfffffu));
    return false;
}
// Bounded wait.  Returns false if it gave up or if another thread did.  The thread that gives up
// leaves in *abort_flag which wait it was: bit 30, the parity in bit 20, the barrier's shared-memory
// address in the low 20 bits (wait_code() turns that into the word the host reads).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_poll(bar, parity, abort_flag);
}
// After an aborted run the MMAs a warp issued before the abort may still be running (they read the
// ring and write TMEM).  Called by that whole warp, converged, before TMEM is freed: one more commit
// from the lane that issued them, then a bounded wait for it.  `bar` is a barrier of count 1 used
// for nothing else.
__device__ __forceinline__ void tc_commit(uint32_t bar);
__device__ __forceinline__ bool elect_one();
__device__ __forceinline__ void drain_mmas(uint32_t bar) {
    if (elect_one()) tc_commit(bar);
    __syncwarp();
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, 0)) break;
        __nanosleep(64);
    }
    __syncwarp();
}
// Test hook (a wait limit of zero): the calling warp waits, bounded, for an arrival on a barrier that
// nothing ever arrives at, so that the block is certain to take its give-up path -- on a small problem
// every real wait may well be satisfied at its first probe.  `bar` is a barrier used for nothing else.
__device__ __forceinline__ void wait_for_nothing(uint32_t bar, volatile int *abort_flag) {
    if (abort_flag[1] == 0) (void)__all_sync(0xffffffffu, mbar_wait(bar, 0, abort_flag));
}
// Status word of a block that gave up: kernel id (1 first-layer stream, 2 layer, 3 least squares) in
// bits 24-27, the index of the barrier within the block's barrier array in bits 1-16, the awaited
// parity in bit 0.  Never zero.
__device__ __forceinline__ int wait_code(int kernel_id, int flag, uint32_t bars_base) {
    const uint32_t index = (((uint32_t)flag & 0xfffffu) - (bars_base & 0xfffffu)) >> 3;
    return (kernel_id << 24) | (int)((index & 0xffffu) << 1) | ((flag >> 20) & 1);
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
// One lane of a fully converged warp.  Code under this predicate is known to run on a single
// thread with warp-uniform operands, which is what lets tcgen05.mma and the bulk copies be issued
// back to back; the same sequence under `if (lane == 0)` issues several times slower.
__device__ __forceinline__ bool elect_one() {
    uint32_t e;
    asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}\n" : "=r"(e));
    return e != 0;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]^T, tf32 inputs, fp32 accumulate
__device__ __forceinline__ void tc_mma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// a / b for small a (well below 2^20) with inv_b = 1.0f / b: no integer division in the pipelines' loops
__device__ __forceinline__ uint32_t small_div(uint32_t a, float inv_b) {
    return (uint32_t)__float2int_rd(((float)a + 0.5f) * inv_b);
}

// K-major operand in the 128-byte swizzled layout: rows of 128 bytes, groups of 8 rows 1024
// bytes apart (stride-dimension offset), descriptor version 1, swizzle mode 2 (128 B).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)1 << 16;                 // leading-dimension offset: unused for swizzled K-major
    d |= (uint64_t)(1024 >> 4) << 32;       // stride-dimension offset
    d |= (uint64_t)1 << 46;                 // descriptor version
    d |= (uint64_t)2 << 61;                 // 128-byte swizzle
    return d;
}


// ---- host side ----------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Tensor maps are descriptions of (pointer, shape, box): a handle sees the same few over and over, one step
// after the other, so the encoded maps are kept per handle and looked up by what they describe (a few
// dozen entries, replaced round robin).  All maps of this library have rank 3, element strides of one,
// no interleave, 256-byte L2 promotion and no out-of-bounds fill value.
struct TensorMapKey {
    const void *base;
    cuuint64_t dims[3];
    cuuint64_t strides[2];
    cuuint32_t box[3];
    int type, swizzle;
};
struct TensorMapCache {
    static constexpr int kEntries = 32;
    CUtensorMap map[kEntries];
    TensorMapKey key[kEntries];
    bool valid[kEntries];
    int next;
};

inline CUresult encode_cached(Context &c, CUtensorMap *out, CUtensorMapDataType type, const void *base,
                              const cuuint64_t (&dims)[3], const cuuint64_t (&strides)[2], const cuuint32_t (&box)[3],
                              CUtensorMapSwizzle swizzle) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return CUDA_ERROR_NOT_SUPPORTED;
    if (!c.tmap_cache) {
        const size_t bytes = (sizeof(TensorMapCache) + 63) / 64 * 64;
        c.tmap_cache = aligned_alloc(64, bytes);
        if (c.tmap_cache) memset(c.tmap_cache, 0, bytes);
    }
    TensorMapKey k;
    memset(&k, 0, sizeof(k));
    k.base = base;
    for (int i = 0; i < 3; ++i) { k.dims[i] = dims[i]; k.box[i] = box[i]; }
    k.strides[0] = strides[0];
    k.strides[1] = strides[1];
    k.type = (int)type;
    k.swizzle = (int)swizzle;
    TensorMapCache *cache = static_cast<TensorMapCache *>(c.tmap_cache);
    if (cache)
        for (int i = 0; i < TensorMapCache::kEntries; ++i)
            if (cache->valid[i] && memcmp(&cache->key[i], &k, sizeof(k)) == 0) {
                *out = cache->map[i];
                return CUDA_SUCCESS;
            }
    cuuint32_t ones[3] = {1, 1, 1};
    const CUresult r = enc(out, type, 3, const_cast<void *>(base), dims, strides, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r == CUDA_SUCCESS && cache) {
        const int i = cache->next;
        cache->next = (i + 1) % TensorMapCache::kEntries;
        cache->map[i] = *out;
        cache->key[i] = k;
        cache->valid[i] = true;
    }
    return r;
}

}  // namespace zeno
