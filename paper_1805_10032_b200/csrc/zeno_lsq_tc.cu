// Least-squares scoring pass on the 5th-generation tensor cores.
//
// The residual of candidate i is linear in the parameters, A (x - gamma v_i) - y = A x - gamma A v_i - y,
// so one pass over V, A and x yields everything: the products A v_i^T for all candidates (a skinny
// GEMM of the rows of V against the n_r rows of A over the parameter index k), A x, and the sums of
// squares of the rows of V.  All three operands are streamed from HBM exactly once; the k-blocks are dealt
// to the blocks round robin, and a block leaves its partial sums in a slab that lsq_finish_kernel adds up in
// double.
//
// A tile of the MMA has 128 rows but there are at most 64 candidates, so a block works on TWO neighbouring
// k-blocks at once (every row of V, A and x is then read 256 contiguous bytes at a time): TMEM lanes 0-63
// hold the candidates' entries of the even k-block, lanes 64-127 those of the odd one.  The rows of A of both
// k-blocks are stacked into ONE B operand, [a_hi(even); a_hi(odd); a_lo(even); a_lo(odd)], so a pair takes one
// group of MMAs: every lane gets the products against all four blocks, and a lane's meaningful columns are
// those of its own k-block (the others multiply entries of one k-block with rows of the other and are never read).
//
// fp32 accuracy on tf32 tensor cores as in the first-layer stream: both operands are split,
// a = a_hi + a_lo, and a_hi b_hi + a_hi b_lo + a_lo b_hi is accumulated, the small products in columns of
// their own.  The tensor core adds into its accumulator with truncation, so the accumulator is drained
// into fp32 registers every kFlush k-blocks (two sets alternate: one is drained while the other adds).
//
// Warp roles (every producer / issuer warp stays converged and issues from one elected lane):
//   warps 0, 16  TMA producers (warp 0 the even stages, warp 16 the odd ones: issuing a stage's copies takes one
//                lane about 800 cycles, more than a stage may take): per stage two 64-row boxes of V, two boxes
//                of A, two 128-byte pieces of x, or one copy of each when the rows allow
//   warp 1       MMA issuer, owner of TMEM
//   warps 2, 3, 18, 19   split the stage's rows of A (the first of a pair of warps the even k-block's, the
//                second the odd one's; warps 2, 3 on even stages, 18, 19 on odd ones) into hi and lo terms
//                (the MMA's B operand, 128-byte swizzled, in a ring of its own) and take A x from the same
//                registers
//   warps 4-11   two converter sets on alternate k-blocks: thread = TMEM lane; reads its 128 bytes of V,
//                accumulates v^2, stores v_hi / v_lo to TMEM as the A operand
//   warps 12-15  drain the accumulator sets into registers; at the end write the slab
// A stage of the load ring is free again as soon as the converters and the splitters have read it into
// registers; only the operand slots wait for the MMAs.  An operand slot is a TMEM buffer (A: the
// candidates' entries) and a shared-memory buffer (B: the split rows of A) with ONE pair of barriers:
// the issuing warp is the slowest link of the chain (cycle stamps: every barrier probe costs it 100 to
// 500 cycles of shared-memory latency even when the phase has long completed), so it waits for one barrier
// a k-block pair, probes the two pairs of a turn back to back, and commits once a pair.
// Every mbarrier wait is bounded; a wait that gives up raises a status word and the block leaves through
// the common teardown.
#include "zeno_internal.h"
#include "zeno_tc.cuh"

namespace zeno {

namespace {

constexpr int kHalfRows = 64;               // candidates per half tile
constexpr int kQBlockK = 32;                // floats per k-block = one 128-byte swizzle row
constexpr int kVHalfBytes = kHalfRows * 128;
constexpr int kQThreads = 32 * 20;
constexpr int kQMaxStages = 8;
constexpr int kQMaxABufs = 5;               // operand slots
constexpr int kQSmem = 217 * 1024;          // dynamic: the ring, reused for the result exchange at the end
constexpr int kQTmemCols = 512;
constexpr int kFlush = 32;                  // k-blocks accumulated in TMEM before a drain

struct LsqTcArgs {
    int m, n_r, n_pad;                      // n_pad: 16 or 32
    int nkb;                                // pairs of k-blocks in a block's k-range
    int stages, n_abufs;                    // stages of the load ring, operand slots
    int wide;                               // the tensor maps fetch both k-blocks of a pair in one copy (d % 32 == 0)
    float *part;                            // [blocks][m+1][n_r+1]
    int *status;
    uint32_t spin_limit;                    // polls a bounded wait may take
};

// bytes of a stage of the load ring: V halves | raw A halves | x pieces (padded to 1 KB)
__host__ __device__ inline int lsq_stage_bytes(int n_pad) { return 2 * kVHalfBytes + 2 * (n_pad * 128) + 1024; }
// bytes of a B operand: [a_hi; a_lo] of both halves
__host__ __device__ inline int lsq_b_bytes(int n_pad) { return 2 * (2 * n_pad * 128); }

__global__ void __launch_bounds__(kQThreads, 1)
lsq_tc_kernel(const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_a,
              const __grid_constant__ CUtensorMap map_x, LsqTcArgs a) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    // full, empty [stages]; ready, free [operand slots]; dfull, dempty [2 sets]
    constexpr int kBars = 2 * kQMaxStages + 2 * kQMaxABufs + 4;
    __shared__ __align__(8) uint64_t bars[kBars];
    __shared__ __align__(8) uint64_t drain_bar;   // teardown after an abort: the issuer's last commit
    __shared__ __align__(8) uint64_t never_bar;   // nothing arrives here (test hook, see wait_for_nothing)
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_state[kAbortWords];
    int &abort_flag = abort_state[0];
    __shared__ int issued[kQMaxStages];
    __shared__ float nrm_s[2][128];         // sums of squares per lane and converter set
    __shared__ float z0_s[4][32];           // A x, per splitter warp

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    if (tid == 32) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
    if (tid == 64) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");

    const int n_pad = a.n_pad, nkb = a.nkb, n_stages = a.stages, n_abufs = a.n_abufs;
    const int raw_bytes = n_pad * 128;
    const int stage_bytes = lsq_stage_bytes(n_pad), b_bytes = lsq_b_bytes(n_pad);
    const int off_raw = 2 * kVHalfBytes, off_x = off_raw + 2 * raw_bytes;
    const int set_cols = 6 * n_pad;                        // D1 (4 n_pad) and D2 (2 n_pad), both halves side by side
    const int a_base = 2 * set_cols;
    const int n_flush = (nkb + kFlush - 1) / kFlush;
    const float inv_stages = 1.0f / (float)n_stages, inv_abufs = 1.0f / (float)n_abufs;
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *bring = ring + (size_t)n_stages * stage_bytes;             // the B operands, 1 KB aligned like the stages
    // drained products per TMEM lane; written once the last accumulator set has been drained, when every
    // stage of the ring has been consumed
    float(*res)[33] = reinterpret_cast<float(*)[33]>(ring);

    auto bar_full = [&](int s) { return smem_u32(&bars[s]); };
    auto bar_empty = [&](int s) { return smem_u32(&bars[kQMaxStages + s]); };
    constexpr int kBarA = 2 * kQMaxStages, kBarD = kBarA + 2 * kQMaxABufs;
    auto bar_ready = [&](int g) { return smem_u32(&bars[kBarA + g]); };
    auto bar_free = [&](int g) { return smem_u32(&bars[kBarA + kQMaxABufs + g]); };
    auto bar_dfull = [&](int q) { return smem_u32(&bars[kBarD + q]); };
    auto bar_dempty = [&](int q) { return smem_u32(&bars[kBarD + 2 + q]); };

    if (tid == 0) {
        abort_flag = 0;
        abort_state[1] = (int)a.spin_limit;
        for (int s = 0; s < kQMaxStages; ++s) {
            mbar_init(bar_full(s), 1);
            mbar_init(bar_empty(s), 6);        // the four warps of a converter set and the two that split the rows of A
            issued[s] = 0;
        }
        for (int g = 0; g < kQMaxABufs; ++g) {
            mbar_init(bar_ready(g), 6);        // a converter set's four warps and the two that split the rows of A
            mbar_init(bar_free(g), 1);         // the MMAs' commit
        }
        for (int q = 0; q < 2; ++q) {
            mbar_init(bar_dfull(q), 1);
            mbar_init(bar_dempty(q), 4);
        }
        mbar_init(smem_u32(&drain_bar), 1);
        mbar_init(smem_u32(&never_bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_base_slot)), "r"(kQTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_wait();
    pdl_launch_dependents();
    const uint32_t tmem = tmem_base_slot;
    volatile int *abortp = &abort_flag;

    if (warp == 0 || warp == 16) {
        // ------------------------------------------------------------------ TMA producers
        if (warp == 0) wait_for_nothing(smem_u32(&never_bar), abortp);
        for (int kb = warp == 0 ? 0 : 1; kb < nkb; kb += 2) {
            const uint32_t round = small_div((uint32_t)kb, inv_stages);
            const int s = kb - (int)round * n_stages;
            if (!__all_sync(0xffffffffu, mbar_wait(bar_empty(s), (round & 1) ^ 1, abortp))) break;
            if (elect_one()) {
                const uint32_t dst = smem_u32(ring + (size_t)s * stage_bytes);
                mbar_expect_tx(bar_full(s), 2 * kVHalfBytes + 2 * raw_bytes + 2 * 128);
                issued[s] = (int)round + 1;
                // Pairs of neighbouring k-blocks (256 contiguous bytes of every row) are dealt round robin:
                // at any moment the blocks read neighbouring addresses of the same ~80 rows, a few hundred
                // pages in all; with one contiguous k-range per block it was ~12,000 pages of 2 MB at once
                const int64_t pair = (int64_t)blockIdx.x + (int64_t)kb * gridDim.x;
                // Issuing a copy costs this lane well over a hundred cycles, and with six per stage the producer
                // was what the ring waited for (cycle stamps: stages re-armed 1,400-2,200 cycles after they were
                // free).  When d and ldv are multiples of 32 the maps see V and A as [row][k-block][32] and one box
                // takes both k-blocks of the pair (a row's two 128-byte pieces then lie side by side in the stage),
                // x comes as one 256-byte piece: three copies per stage.  (A map ordered [k-block][row][32] gives
                // the stage layout of two separate boxes with one copy, but it fetches every row in two 128-byte
                // visits and the kernel ran 7 % slower.)
                const int n_loads = a.wide ? 3 : 6;
#pragma unroll 1
                for (int w = 0; w < n_loads; ++w) {    // V, A, x (of the two halves): ONE issue site
                    const int h = a.wide ? 0 : (w & 1), what = a.wide ? w : (w >> 1);
                    const CUtensorMap *map = what == 0 ? &map_v : what == 1 ? &map_a : &map_x;
                    const uint32_t off = what == 0 ? h * kVHalfBytes : what == 1 ? off_raw + h * raw_bytes : off_x + h * 128;
                    const int64_t k = (2 * pair + h) * kQBlockK;
                    const bool blocked = a.wide && what < 2;          // coordinates (0, k-block, row 0)
                    tma_load_3d(dst + off, map, blocked ? 0 : (int)k, blocked ? (int)(2 * pair) : 0, 0, bar_full(s));
                }
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc_base = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(128 >> 4) << 24);
        const uint32_t idesc_2n = idesc_base | ((uint32_t)((2 * n_pad) >> 3) << 17);
        const uint32_t idesc_4n = idesc_base | ((uint32_t)((4 * n_pad) >> 3) << 17);
        int ag = 0;                                      // operand slot of the next k-block pair
        uint32_t aph = 0;                                // and the phase its barrier is awaited in
        // Two k-block pairs per turn of the loop (the operands are in place well ahead of this warp, and its
        // waits, vote, fence and election cost as much as the MMAs it issues).  kFlush is even, so the two
        // pairs of a turn always add into the same accumulator set.
        for (int kb = 0; kb < nkb; kb += 2) {
            const bool two = kb + 1 < nkb;
            const int fl = kb / kFlush, in_fl = kb - fl * kFlush;
            const int set = fl & 1;
            if (in_fl == 0) {                          // a fresh accumulator set: wait until it was drained
                if (!__all_sync(0xffffffffu, mbar_wait(bar_dempty(set), (((uint32_t)fl >> 1) & 1) ^ 1, abortp))) break;
                tc_fence_after();
            }
            int g1 = ag + 1;
            uint32_t aph1 = aph;
            if (g1 == n_abufs) { g1 = 0; aph1 ^= 1; }
            // both probes are issued before either result is looked at
            bool r0 = mbar_try_wait(bar_ready(ag), aph);
            bool r1 = !two || mbar_try_wait(bar_ready(g1), aph1);
            if (!r0) r0 = mbar_wait_poll(bar_ready(ag), aph, abortp);
            if (!r1) r1 = mbar_wait_poll(bar_ready(g1), aph1, abortp);
            if (!__all_sync(0xffffffffu, r0 && r1)) break;
            tc_fence_after();
            if (elect_one()) {
                // D1 = v_hi [a_hi(even); a_hi(odd); a_lo(even); a_lo(odd)]^T, D2 = v_lo [a_hi(even); a_hi(odd)]^T:
                // lanes 0-63 use the even k-block's columns, lanes 64-127 the odd one's
                const uint32_t d1 = tmem + set * set_cols, d2 = d1 + 4 * n_pad;
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    if (q == 1 && !two) break;
                    const int g = q ? g1 : ag;
                    const uint32_t a_tmem = tmem + a_base + g * 64;
                    const uint32_t bx = smem_u32(bring + (size_t)g * b_bytes);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint64_t db = smem_desc_sw128(bx + ks * 32);
                        const uint32_t acc = (uint32_t)(in_fl | q | ks);
                        tc_mma_tf32_ts(d1, a_tmem + ks * 8, db, idesc_4n, acc);
                        tc_mma_tf32_ts(d2, a_tmem + 32 + ks * 8, db, idesc_2n, acc);
                    }
                    tc_commit(bar_free(g));
                }
                const int last = two ? kb + 1 : kb;
                if (last - fl * kFlush == kFlush - 1 || last + 1 == nkb) tc_commit(bar_dfull(set));
            }
            __syncwarp();
            ag = two ? g1 + 1 : g1;
            aph = aph1;
            if (two && ag == n_abufs) { ag = 0; aph ^= 1; }
        }
    } else if (warp == 2 || warp == 3 || warp == 18 || warp == 19) {
        // ------------------------------------------------------------------ rows of A: split for the MMA, and A x
        // Warp 2 takes the even k-block's rows of every stage, warp 3 the odd one's.  All of a lane's rows
        // are loaded before the first store (loads placed after stores to the same shared array would wait
        // for them), and the stage is released as soon as they are in registers.
        const int sset = warp >= 18 ? 1 : 0;          // set 0 takes the even stages, set 1 the odd
        const int h = warp & 1;
        float accx[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};    // rows 4 u + lane / 8 (u < n_pad / 4)
        bool ok = true;
        for (int kb = sset; kb < nkb && ok; kb += 2) {
            const uint32_t sround = small_div((uint32_t)kb, inv_stages), bround = small_div((uint32_t)kb, inv_abufs);
            const int s = kb - (int)sround * n_stages, gb = kb - (int)bround * n_abufs;
            ok = mbar_wait(bar_full(s), sround & 1, abortp);
            if (!ok) break;
            const uint8_t *st = ring + (size_t)s * stage_bytes;
            uint8_t *bop = bring + (size_t)gb * b_bytes;
            const float4 x4 = *reinterpret_cast<const float4 *>(st + off_x + h * 128 + (lane & 7) * 16);
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = 4 * u + (lane >> 3), c = lane & 7;
                v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                const int piece = a.wide ? 2 * j + h : h * n_pad + j;        // where row j of this warp's k-block landed
                if (4 * u < n_pad) v[u] = *reinterpret_cast<const float4 *>(st + off_raw + piece * 128 + ((c ^ (piece & 7)) << 4));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(s));
            ok = mbar_wait(bar_free(gb), (bround & 1) ^ 1, abortp);        // the MMAs that read this operand last are done
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (4 * u >= n_pad) break;
                const int j = 4 * u + (lane >> 3), c = lane & 7;
                const uint32_t sw = (uint32_t)j * 128 + ((c ^ (j & 7)) << 4);
                accx[u] = fmaf(v[u].x, x4.x, fmaf(v[u].y, x4.y, fmaf(v[u].z, x4.z, fmaf(v[u].w, x4.w, accx[u]))));
                const float4 hi = make_float4(tf32_hi(v[u].x), tf32_hi(v[u].y), tf32_hi(v[u].z), tf32_hi(v[u].w));
                // B operand rows: a_hi of the even k-block, a_hi of the odd one, then the two a_lo blocks
                // (n_pad % 8 == 0: every block starts in the same swizzle phase)
                *reinterpret_cast<float4 *>(bop + h * n_pad * 128 + sw) = hi;
                *reinterpret_cast<float4 *>(bop + (2 + h) * n_pad * 128 + sw) =
                    make_float4(v[u].x - hi.x, v[u].y - hi.y, v[u].z - hi.z, v[u].w - hi.w);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_ready(gb));
        }
        // A x: the eight lanes of a row add up
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            float t = accx[u];
            t += __shfl_xor_sync(0xffffffffu, t, 1);
            t += __shfl_xor_sync(0xffffffffu, t, 2);
            t += __shfl_xor_sync(0xffffffffu, t, 4);
            if ((lane & 7) == 0 && 4 * u + (lane >> 3) < 32) z0_s[2 * sset + h][4 * u + (lane >> 3)] = t;
        }
    } else if (warp >= 4 && warp < 12) {
        // ------------------------------------------------------------------ converters
        const int cset = (warp - 4) >> 2;             // set 0 takes the even k-blocks, set 1 the odd
        const int quad = warp & 3;
        const int row = quad * 32 + lane;             // TMEM lane: candidate row (half 0), row - 64 (half 1)
        const uint32_t a_bufs = tmem + ((uint32_t)(quad * 32) << 16) + a_base;
        float nrm4[4] = {0.f, 0.f, 0.f, 0.f};
        for (int kb = cset; kb < nkb; kb += 2) {
            const uint32_t it = (uint32_t)kb;
            const uint32_t sround = small_div(it, inv_stages), around = small_div(it, inv_abufs);
            const int s = (int)(it - sround * n_stages), g = (int)(it - around * n_abufs);
            if (!mbar_wait(bar_full(s), sround & 1, abortp)) break;
            // this lane's 128 bytes: box h, row r (two boxes one after the other), or row r, piece h (one box).
            // In the second layout the pieces of a quarter warp's eight lanes are two apart and their swizzle
            // phases take only four values: every other group of four lanes reads its 16-byte chunks in the
            // order 1, 0, 3, 2, .. (and swaps them back in registers), so that the eight lanes of a
            // shared-memory access fall into eight different bank groups.
            const int piece = a.wide ? (((row & 63) << 1) | (row >> 6)) : row;
            const int flip = a.wide ? ((row >> 2) & 1) : 0;
            const uint8_t *src = ring + (size_t)s * stage_bytes + piece * 128;
            float4 v[8];
            uint32_t hi[32], lo[32];
#pragma unroll
            for (int c = 0; c < 8; ++c) v[c] = *reinterpret_cast<const float4 *>(src + ((c ^ flip ^ (piece & 7)) << 4));
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty(s));
            if (flip) {
#pragma unroll
                for (int c = 0; c < 8; c += 2) {
                    const float4 t = v[c];
                    v[c] = v[c + 1];
                    v[c + 1] = t;
                }
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float e[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    nrm4[u] = fmaf(e[u], e[u], nrm4[u]);
                    const float h = tf32_hi(e[u]);
                    hi[4 * c + u] = __float_as_uint(h);
                    lo[4 * c + u] = __float_as_uint(e[u] - h);
                }
            }
            if (!mbar_wait(bar_free(g), (around & 1) ^ 1, abortp)) break;
            tc_fence_after();
            tc_st32(a_bufs + g * 64, hi);
            tc_st32(a_bufs + g * 64 + 32, lo);
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_ready(g));
        }
        nrm_s[cset][row] = (nrm4[0] + nrm4[1]) + (nrm4[2] + nrm4[3]);
    } else if (warp >= 12 && warp < 16) {
        // ------------------------------------------------------------------ drains
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const int h = row >> 6;                       // which half's columns are meaningful in this lane
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        float acc[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[j] = 0.f;
        for (int fl = 0; fl < n_flush; ++fl) {
            const int set = fl & 1;
            if (!mbar_wait(bar_dfull(set), ((uint32_t)fl >> 1) & 1, abortp)) break;
            tc_fence_after();
            const uint32_t d = tmem + lane_addr + set * set_cols + h * n_pad;    // this lane's k-block's columns
#pragma unroll
            for (int j0 = 0; j0 < 32; j0 += 16) {
                if (j0 >= n_pad) break;
                uint32_t big[16], s1[16], s2[16];
                tc_ld16(d + j0, big);                           // v_hi a_hi
                tc_ld16(d + 2 * n_pad + j0, s1);                // v_hi a_lo
                tc_ld16(d + 4 * n_pad + j0, s2);                // v_lo a_hi
                tc_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    acc[j0 + j] += __uint_as_float(big[j]) + (__uint_as_float(s1[j]) + __uint_as_float(s2[j]));
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_dempty(set));
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) res[row][j] = acc[j];
    }

    // ---------------------------------------------------------------------- teardown and the slab
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1 && abort_flag) drain_mmas(smem_u32(&drain_bar));
    if (tid == 0 && abort_flag) {
        for (int s = 0; s < n_stages; ++s)
            if (issued[s] > 0) {
                for (uint32_t i = 0; i < kSpinLimit; ++i) {
                    if (mbar_try_wait(bar_full(s), (uint32_t)(issued[s] - 1) & 1)) break;
                    __nanosleep(64);
                }
            }
        atomicCAS(a.status, 0, wait_code(3, abort_flag, smem_u32(bars)));   // the first block to give up is kept
    }
    // slab [m+1][n_r+1]: row 0 = A x, row 1+c = A v_c^T (both halves of the k-range), last column = sum of squares
    const int stride = a.n_r + 1;
    float *slab = a.part + (int64_t)blockIdx.x * (a.m + 1) * stride;
    for (int t = tid; t < (a.m + 1) * stride; t += kQThreads) {
        const int r = t / stride, j = t - r * stride;
        float v;
        if (r == 0) {
            v = j < a.n_r ? (z0_s[0][j] + z0_s[1][j]) + (z0_s[2][j] + z0_s[3][j]) : 0.f;
        } else {
            const int c = r - 1;
            v = j < a.n_r ? res[c][j] + res[c + kHalfRows][j]
                          : (nrm_s[0][c] + nrm_s[1][c]) + (nrm_s[0][c + kHalfRows] + nrm_s[1][c + kHalfRows]);
        }
        slab[t] = v;
    }
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kQTmemCols) : "memory");
    }
}

}  // namespace

// Rows a TMA box can step through (16-byte multiples), at most 64 candidates (one half tile) and
// 32 samples; the copies take the parameter index as a signed 32-bit coordinate, so d stays below 2^31
// (longer vectors go to the CUDA-core stream, which indexes in 64 bits).
bool lsq_tc_usable(const LsqArgs &a, bool aligned) {
    return aligned && a.m >= 1 && a.m <= kHalfRows && a.n_r >= 1 && a.n_r <= 32 && a.d % 4 == 0 && a.ldv % 4 == 0 &&
           a.d >= 4096 && a.d < (int64_t(1) << 31) && encode_tiled_fn() != nullptr;
}

// Fills a.part with one slab per block; *slabs = the number of slabs written.
cudaError_t launch_lsq_tc(Context &c, const LsqArgs &a, int max_slabs, int *slabs, cudaStream_t s) {
    if (!encode_tiled_fn()) return cudaErrorNotSupported;
    const int n_pad = a.n_r <= 16 ? 16 : 32;
    CUtensorMap map_v, map_a, map_x;
    const bool wide = a.d % kQBlockK == 0 && a.ldv % kQBlockK == 0;
    if (wide) {
        // [row][k-block][32]: the k-blocks of a row are 128 bytes apart, the rows ldv (or d) elements
        const cuuint64_t nkb_all = (cuuint64_t)(a.d / kQBlockK);
        {
            cuuint64_t dims[3] = {kQBlockK, nkb_all, (cuuint64_t)a.m};
            cuuint64_t strides[2] = {128, (cuuint64_t)a.ldv * 4};
            cuuint32_t box[3] = {kQBlockK, 2, kHalfRows};
            if (encode_cached(c, &map_v, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, a.V, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS)
                return cudaErrorInvalidValue;
        }
        {
            cuuint64_t dims[3] = {kQBlockK, nkb_all, (cuuint64_t)a.n_r};
            cuuint64_t strides[2] = {128, (cuuint64_t)a.d * 4};
            cuuint32_t box[3] = {kQBlockK, 2, (cuuint32_t)n_pad};
            if (encode_cached(c, &map_a, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, a.A, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS)
                return cudaErrorInvalidValue;
        }
        {
            cuuint64_t dims[3] = {(cuuint64_t)a.d, 1, 1};
            cuuint64_t strides[2] = {(cuuint64_t)a.d * 4, (cuuint64_t)a.d * 4};
            cuuint32_t box[3] = {2 * kQBlockK, 1, 1};
            if (encode_cached(c, &map_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, a.x, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE) != CUDA_SUCCESS)
                return cudaErrorInvalidValue;
        }
    } else {
    {
        cuuint64_t dims[3] = {(cuuint64_t)a.d, (cuuint64_t)a.m, 1};
        cuuint64_t strides[2] = {(cuuint64_t)a.ldv * 4, (cuuint64_t)a.ldv * 4 * (cuuint64_t)a.m};
        cuuint32_t box[3] = {kQBlockK, kHalfRows, 1};
        if (encode_cached(c, &map_v, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, a.V, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)a.d, (cuuint64_t)a.n_r, 1};
        cuuint64_t strides[2] = {(cuuint64_t)a.d * 4, (cuuint64_t)a.d * 4 * (cuuint64_t)a.n_r};
        cuuint32_t box[3] = {kQBlockK, (cuuint32_t)n_pad, 1};
        if (encode_cached(c, &map_a, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, a.A, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)a.d, 1, 1};
        cuuint64_t strides[2] = {(cuuint64_t)a.d * 4, (cuuint64_t)a.d * 4};
        cuuint32_t box[3] = {kQBlockK, 1, 1};
        if (encode_cached(c, &map_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, a.x, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    }
    const int64_t n_kblocks = (a.d + kQBlockK - 1) / kQBlockK;
    int blocks = c.sm_count > 0 ? c.sm_count : 148;
    if (blocks > max_slabs) blocks = max_slabs;
    if ((int64_t)blocks > (n_kblocks + 1) / 2) blocks = (int)((n_kblocks + 1) / 2);
    LsqTcArgs t;
    t.m = a.m;
    t.n_r = a.n_r;
    t.n_pad = n_pad;
    t.wide = wide ? 1 : 0;
    t.nkb = (int)((n_kblocks + 2 * (int64_t)blocks - 1) / (2 * (int64_t)blocks));
    const int stage_bytes = lsq_stage_bytes(n_pad), b_bytes = lsq_b_bytes(n_pad);
    t.n_abufs = (kQTmemCols - 2 * 6 * n_pad) / 64;
    if (t.n_abufs > kQMaxABufs) t.n_abufs = kQMaxABufs;
    t.stages = (kQSmem - 1024 - t.n_abufs * b_bytes) / stage_bytes;
    if (t.stages > kQMaxStages) t.stages = kQMaxStages;
    t.part = a.part;
    t.status = c.dev_status;
    t.spin_limit = c.spin_limit;
    static PerDeviceOnce attr_set;
    if (attr_set.need(c.device)) {
        cudaError_t e = cudaFuncSetAttribute(lsq_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kQSmem);
        if (e != cudaSuccess) return e;
        attr_set.mark(c.device);
    }
    *slabs = blocks;
    return launch_chained(lsq_tc_kernel, dim3(blocks), dim3(kQThreads), (size_t)t.stages * stage_bytes + (size_t)t.n_abufs * b_bytes + 1024, s,
                          chain_launches(c), map_v, map_a, map_x, t);
}

}  // namespace zeno
