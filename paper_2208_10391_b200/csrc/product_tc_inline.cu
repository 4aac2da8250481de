// Small and mid-size products on the tcgen05 tensor cores in ONE launch: C = A*B (+ Add terms), 3xTF32, with the
// operands read as stored and split into their tf32 halves in shared memory.
//
// The large-product kernel (product_tc.cu) takes its operands as hi / lo planes that a pre-pass writes to global
// memory, and with few output tiles it needs a split-K reduction pass: two or three launches, which is most of the
// time of a product below about 2000^3.  Here a product is one launch:
//   warp 0      TMA producer: per k-block of 32 the raw f32 tile of A (128 rows x 32 k, 128-byte swizzle) and the raw tile
//               of B (32 k-rows x BN columns, as BN / 32 swizzled boxes of 32 x 32);
//   warps 2-9   transform: a thread reads half of its row of A (the eight lanes of a load phase hit eight different
//               swizzled chunks), splits it in registers and stores the hi and lo halves into TENSOR MEMORY with
//               tcgen05.st (lane = row, one column per k): the MMA takes its A operand from there, so A is never
//               written back to shared memory nor read from it by the tensor core.  B is split AND transposed into
//               K-major hi / lo tiles in shared memory (BN rows of 32 k): a lane reads four columns of its k-row with
//               one 16-byte load and writes each value into its column's row, where the 32 lanes of a warp fill one
//               128-byte row: no bank conflict on either side;
//   warp 1      MMA issuer: 4 k-steps x 3 tcgen05.mma kind::tf32 (lo*hi, hi*lo, hi*hi; M128, N = BN; A from tensor memory,
//               B through a shared-memory descriptor) per k-block into one accumulator in tensor memory; tcgen05.commit
//               frees the stage;
//   warps 2-9   then the epilogue: tcgen05.ld (two warps per quarter of the tile's rows, each half of the columns), Add terms,
//               structure mask, 16-byte stores.
// With few output tiles the contraction is split over the CTAs of a thread-block cluster (up to 16): each leaves its partial
// tile in its own shared memory and CTA r finishes rows [r * 128 / s, (r + 1) * 128 / s) by adding the partial tiles through
// distributed shared memory in k order (deterministic; no atomics, no scratch in global memory, no second launch).
// The tile's structural k-range bounds the contraction as everywhere else.  Shared memory still moves more bytes per
// flop than in the plane kernel (the transform reads every operand byte and writes B once more), so this kernel tops out
// near half of the tensor peak; it is chosen where launches, not flops, are the cost.
// Operands stored transposed are read as stored: A as k x m arrives as four boxes of 32 k-rows x 32 columns and a transform thread
// gathers its row from a column of them; B as n x k is K-major already and is split where it lies.
// Every wait is bounded; a CTA that gives up still meets its cluster at both cluster barriers.
#include <algorithm>
#include <cstring>

#include <cooperative_groups.h>
#include <cuda.h>

#include "device_info.h"
#include "product_tc.h"
#include "tc_ptx.cuh"
#include "tc_wait.cuh"

namespace mom {

namespace {

namespace cg = cooperative_groups;

constexpr int IBM = 128, IBK = 32, ITHREADS = 320, IMAX_SPLIT = 16;    // warps: producer, MMA issuer, eight transform / epilogue warps
constexpr int XFORM_WARPS = 8;

template <int BN>
struct InlineCfg {
    // Two rings.  RAW: what TMA delivers (the f32 tiles of A and B), free again as soon as the transform warps have read it, so
    // that the loads run RAW stages ahead of the transform (a load takes about 1900 cycles, the transform of a k-block 800, its
    // MMAs 770).  SPLIT: what the MMA reads (A's halves in tensor memory, B's in shared memory), free once its MMAs are done.
    static constexpr int RAW = BN == 64 ? 5 : 4, SPLIT = BN == 64 ? 4 : 3;
    static constexpr int A_BYTES = IBM * IBK * 4;            // 16 KB: the raw tile of A
    static constexpr int B_RAW_BYTES = IBK * BN * 4;         // BN / 32 boxes of 32 k-rows x 32 columns
    static constexpr int B_PLANE_BYTES = BN * IBK * 4;       // K-major: BN rows of 32 k
    static constexpr int RAW_BYTES = A_BYTES + B_RAW_BYTES, SPLIT_BYTES = 2 * B_PLANE_BYTES;
    static constexpr int RING_BYTES = RAW * RAW_BYTES + SPLIT * SPLIT_BYTES;
    // tensor memory: the accumulator in columns [0, BN), then per SPLIT stage 32 columns of A's hi half and 32 of its lo half
    static constexpr int A_COLS = 2 * IBK, TMEM_COLS = 512;
    static_assert(BN + SPLIT * A_COLS <= TMEM_COLS, "tensor memory budget");
    static constexpr int LDP = BN + 4;                       // row length of the partial tile (floats)
    static constexpr int NUM_BARRIERS = 2 * RAW + 2 * SPLIT + 2;
    static constexpr int SMEM_BYTES = 1024 + RING_BYTES + 256;
    static_assert(IBM * LDP * 4 <= RING_BYTES, "the partial tile reuses the rings");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

struct InlineParams {
    int m, n, k;
    int pa, pb, pout;
    int split, tiles_n;
    float *C;
    AddTerms add;
    int32_t *status;
};

// hi = a rounded to tf32 (nearest, ties away from zero, done on the bit pattern with full-rate integer instructions);
// lo = a - hi, exact in f32 and handed over as it is: whatever the tensor core does with the bits below tf32 changes lo
// by at most 2^-11 of itself, i.e. 2^-22 of a, the size of the lo*lo term the scheme leaves out anyway
__device__ __forceinline__ float tf32_round(float a) { return __uint_as_float((__float_as_uint(a) + 0x1000u) & 0xFFFFE000u); }
__device__ __forceinline__ void split4(const float4 a, float4 &hi, float4 &lo) {
    hi.x = tf32_round(a.x); hi.y = tf32_round(a.y); hi.z = tf32_round(a.z); hi.w = tf32_round(a.w);
    lo.x = a.x - hi.x; lo.y = a.y - hi.y; lo.z = a.z - hi.z; lo.w = a.w - hi.w;
}

// K-major tile with 128-byte rows under the 128B swizzle: 8-row groups are 1024 bytes apart, a K = 8 step is 32 bytes
__device__ __forceinline__ uint64_t kmajor_desc128(uint32_t tile, int kstep) {
    return ptx::smem_desc(tile + kstep * 32, 16, 8 * 128, ptx::SWIZZLE_128B);
}

// The transform of one k-block, shared by the 1-CTA and the CTA-pair kernels: a warp of the eight transform warps (w2 = 0..7) splits
// its share of the raw tiles.  NB = columns of B this CTA holds.
//   A: the thread owns row 32 ((w2 + 2) % 4) + lane of the tile (the tensor-memory lane its warp may write) and half of its 32 k: four
//      16-byte loads from the swizzled raw tile, two tcgen05.st of 16 columns (hi, lo).
//   B: task t of the warp is (box j, group c) = columns 32 j + 4 c .. + 3 of k-row `lane`; value e of it lands in row
//      n = 32 j + 4 c + e of the K-major tile, at k = lane (group lane / 4, word lane % 4).
template <int NB, bool TA = false, bool TB = false>
struct Transform {
    static constexpr int TASKS = NB / 4 / XFORM_WARPS;
    uint32_t a_src[4], src_off[TASKS], dst_off[TASKS][4];
    uint32_t at_base, at_group;                              // TA: this thread's column of the raw boxes of A (stored k x m)
    __device__ __forceinline__ Transform(int w2, int lane) {
        const int arow = ((w2 + 2) & 3) * 32 + lane, ahalf = w2 >> 2;     // transform warp w2 is warp w2 + 2 of the CTA: lanes 32 (warp % 4) ..
#pragma unroll
        for (int u = 0; u < 4; ++u) a_src[u] = arow * 128 + (((4 * ahalf + u) ^ (arow & 7)) << 4);
        // TA: row arow of the tile is column `lane` of box (w2 + 2) % 4 (32 k-rows x 32 columns, 128-byte rows under the swizzle)
        at_base = ((w2 + 2) & 3) * 4096 + ahalf * 16 * 128 + (lane & 3) * 4;
        at_group = lane >> 2;
#pragma unroll
        for (int t = 0; t < TASKS; ++t) {
            const int task = w2 + XFORM_WARPS * t, j = task >> 3, c = task & 7;
            if (TB) {                                        // B stored n x k: the raw tile is K-major already; 16-byte groups stay where they are
                src_off[t] = ((w2 * 32 + lane) + 32 * XFORM_WARPS * t) * 16;
                continue;
            }
            src_off[t] = j * 4096 + lane * 128 + ((c ^ (lane & 7)) << 4);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int n = 32 * j + 4 * c + e;
                dst_off[t][e] = n * 128 + ((((uint32_t)lane >> 2) ^ (n & 7)) << 4) + ((lane & 3) << 2);
            }
        }
    }
    // araw / braw: the raw tiles of A and B; a_tmem: this thread's 16 columns of A's hi half in tensor memory (lo: + IBK);
    // bhi / blo: B's K-major tiles.  Ends with everything the MMA will read made visible to it.
    __device__ __forceinline__ void run(const uint8_t *araw, const uint8_t *braw, uint32_t a_tmem, uint8_t *bhi, uint8_t *blo) const {
        float4 av[4], bv[TASKS];
        if (TA) {
            float a16[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) a16[u] = *reinterpret_cast<const float *>(araw + at_base + u * 128 + ((at_group ^ (u & 7)) << 4));
#pragma unroll
            for (int u = 0; u < 4; ++u) av[u] = make_float4(a16[4 * u], a16[4 * u + 1], a16[4 * u + 2], a16[4 * u + 3]);
        } else {
#pragma unroll
            for (int u = 0; u < 4; ++u) av[u] = *reinterpret_cast<const float4 *>(araw + a_src[u]);
        }
#pragma unroll
        for (int t = 0; t < TASKS; ++t) bv[t] = *reinterpret_cast<const float4 *>(braw + src_off[t]);
        {
            uint32_t hi16[16], lo16[16];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float4 hi, lo;
                split4(av[u], hi, lo);
                hi16[4 * u] = __float_as_uint(hi.x); hi16[4 * u + 1] = __float_as_uint(hi.y);
                hi16[4 * u + 2] = __float_as_uint(hi.z); hi16[4 * u + 3] = __float_as_uint(hi.w);
                lo16[4 * u] = __float_as_uint(lo.x); lo16[4 * u + 1] = __float_as_uint(lo.y);
                lo16[4 * u + 2] = __float_as_uint(lo.z); lo16[4 * u + 3] = __float_as_uint(lo.w);
            }
            ptx::tmem_st_16cols(a_tmem, hi16);
            ptx::tmem_st_16cols(a_tmem + IBK, lo16);
        }
#pragma unroll
        for (int t = 0; t < TASKS; ++t) {
            float4 hi, lo;
            split4(bv[t], hi, lo);
            if (TB) {
                *reinterpret_cast<float4 *>(bhi + src_off[t]) = hi;
                *reinterpret_cast<float4 *>(blo + src_off[t]) = lo;
                continue;
            }
            *reinterpret_cast<float *>(bhi + dst_off[t][0]) = hi.x; *reinterpret_cast<float *>(blo + dst_off[t][0]) = lo.x;
            *reinterpret_cast<float *>(bhi + dst_off[t][1]) = hi.y; *reinterpret_cast<float *>(blo + dst_off[t][1]) = lo.y;
            *reinterpret_cast<float *>(bhi + dst_off[t][2]) = hi.z; *reinterpret_cast<float *>(blo + dst_off[t][2]) = lo.z;
            *reinterpret_cast<float *>(bhi + dst_off[t][3]) = hi.w; *reinterpret_cast<float *>(blo + dst_off[t][3]) = lo.w;
        }
        ptx::tmem_wait_st();
        ptx::fence_proxy_async_smem();                       // the MMA reads B's tiles through the asynchronous proxy
        ptx::tc_fence_before_sync();
        __syncwarp();
    }
};

// Epilogue store of a warp's 32 x 32 chunk of the tile (lane = row, v = its 32 columns): through a 32 x 36 staging tile of the warp
// in shared memory, so that the stores to C and the loads of the Add terms are row-contiguous (one instruction covers four rows of
// 128 bytes instead of 32 rows of 16).  Conflict-free both ways: a store phase's eight lanes are eight rows 36 words apart, a load
// phase's eight lanes one row's 32 words.
constexpr int STAGE_LD = 36, STAGE_FLOATS = 32 * STAGE_LD;
__device__ __forceinline__ void store_chunk(float *stage, const float (&v)[32], int lane, int row_base, int col0, const InlineParams &prm, bool vec) {
#pragma unroll
    for (int j = 0; j < 8; ++j)
        *reinterpret_cast<float4 *>(stage + lane * STAGE_LD + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
    __syncwarp();
    const int sub = lane >> 3, cc = col0 + (lane & 7) * 4;
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        const int row = 4 * it + sub, r = row_base + row;
        const float4 x = *reinterpret_cast<const float4 *>(stage + row * STAGE_LD + (lane & 7) * 4);
        if (r >= prm.m || cc >= prm.n) continue;
        float w[4] = {x.x, x.y, x.z, x.w};
        finish_row4(w, prm.add, 0, r, cc, prm.n, prm.n, prm.pout, vec);
        float *dst = prm.C + (long long)r * prm.n + cc;
        if (vec && cc + 3 < prm.n) {
            *reinterpret_cast<float4 *>(dst) = make_float4(w[0], w[1], w[2], w[3]);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (cc + e < prm.n) dst[e] = w[e];
        }
    }
    __syncwarp();                                            // the staging tile is free for the warp's next chunk
}

// Split contraction, last phase: CTA `rank` of the cluster finishes rows [rank * 128 / SPLIT, ...) of the tile, adding the cluster's
// partial tiles (P: this CTA's, at the same address in every CTA) in k order.  A load through distributed shared memory takes
// 500-700 cycles, so ALL the loads a thread needs (its items x SPLIT peers, at most 16 of 16 bytes) are issued before the first
// sum.  The cluster's second barrier is split: a CTA arrives once its sums are in registers (nobody needs its peers' shared memory
// any more on its behalf) and waits after its Add terms and stores (it may not leave while a peer still reads its tile).
template <int BN, int SPLIT>
__device__ __forceinline__ void reduce_partial_tiles(cg::cluster_group &cluster, const float *P, int rank, int r0, int c0, const InlineParams &prm) {
    constexpr int LDP = BN + 4, ROWS = IBM / SPLIT, ITEMS = ROWS * (BN / 4), NI = (ITEMS + ITHREADS - 1) / ITHREADS;
    const float *peer[SPLIT];
#pragma unroll
    for (int q = 0; q < SPLIT; ++q) peer[q] = cluster.map_shared_rank(P, q);
    float4 x[NI][SPLIT];
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        const int e = threadIdx.x + i * ITHREADS;
        const int off = (rank * ROWS + e / (BN / 4)) * LDP + ((e % (BN / 4)) << 2);
#pragma unroll
        for (int q = 0; q < SPLIT; ++q) x[i][q] = e < ITEMS ? *reinterpret_cast<const float4 *>(peer[q] + off) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float w[NI][4];
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        w[i][0] = w[i][1] = w[i][2] = w[i][3] = 0.f;
#pragma unroll
        for (int q = 0; q < SPLIT; ++q) { w[i][0] += x[i][q].x; w[i][1] += x[i][q].y; w[i][2] += x[i][q].z; w[i][3] += x[i][q].w; }
    }
    ptx::cluster_arrive();
    const bool vec = (reinterpret_cast<uintptr_t>(prm.C) & 15) == 0 && (prm.n & 3) == 0;
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        const int e = threadIdx.x + i * ITHREADS;
        const int r = r0 + rank * ROWS + e / (BN / 4), cc = c0 + ((e % (BN / 4)) << 2);
        if (e >= ITEMS || r >= prm.m || cc >= prm.n) continue;
        finish_row4(w[i], prm.add, 0, r, cc, prm.n, prm.n, prm.pout, vec);
        float *dst = prm.C + (long long)r * prm.n + cc;
        if (vec && cc + 3 < prm.n) {
            *reinterpret_cast<float4 *>(dst) = make_float4(w[i][0], w[i][1], w[i][2], w[i][3]);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (cc + j < prm.n) dst[j] = w[i][j];
        }
    }
    ptx::cluster_wait();
}

// TA / TB: the operand is stored transposed (A as k x m, B as n x k); the transform reads it accordingly, everything else is the same
template <int BN, bool TA = false, bool TB = false>
__global__ void __launch_bounds__(ITHREADS, 1)
product_tc_inline_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const InlineParams prm) {
    using Cfg = InlineCfg<BN>;
    constexpr int R = Cfg::RAW, S = Cfg::SPLIT;
    extern __shared__ uint8_t smem_raw[];
    __shared__ int abort_word;
    allow_dependents();
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *const base_ptr = smem_raw + (base - ptx::smem_u32(smem_raw));
    const uint32_t split_base = base + R * Cfg::RAW_BYTES;
    const uint32_t bars = base + Cfg::RING_BYTES;
    auto raw_full = [&](int s) { return bars + 8 * s; };                    // TMA has delivered raw stage s
    auto raw_empty = [&](int s) { return bars + 8 * (R + s); };             // the transform warps have read it
    auto ready = [&](int s) { return bars + 8 * (2 * R + s); };             // the transform warps have filled split stage s
    auto empty = [&](int s) { return bars + 8 * (2 * R + S + s); };         // its MMAs are done
    const uint32_t acc_full = bars + 8 * (2 * R + 2 * S), drain = acc_full + 8, tmem_slot = bars + 8 * Cfg::NUM_BARRIERS;
    volatile int *abort_flag = &abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    cg::cluster_group cluster = cg::this_cluster();
    const int split = prm.split;
    const int rank = split > 1 ? (int)cluster.block_rank() : 0;          // position in the cluster = k-slice
    const int tile = blockIdx.x / split;
    const int r0 = (tile / prm.tiles_n) * IBM, c0 = (tile % prm.tiles_n) * BN;

    int klo, khi;
    tile_k_range(prm.pa, prm.pb, r0, min(r0 + IBM, prm.m), c0, min(c0 + BN, prm.n), prm.k, &klo, &khi);
    klo &= ~(IBK - 1);                                                   // extra leading elements are stored zeros
    const int blocks = klo < khi ? (khi - klo + IBK - 1) / IBK : 0;
    const int per = (blocks + split - 1) / split;
    const int kb0 = min(rank * per, blocks), nk = min(kb0 + per, blocks) - kb0;

    if (threadIdx.x == 0) {
        abort_word = 0;
        for (int s = 0; s < R; ++s) { ptx::mbar_init(raw_full(s), 1); ptx::mbar_init(raw_empty(s), XFORM_WARPS); }
        for (int s = 0; s < S; ++s) { ptx::mbar_init(ready(s), XFORM_WARPS); ptx::mbar_init(empty(s), 1); }
        ptx::mbar_init(acc_full, 1);
        ptx::mbar_init(drain, 1);
        ptx::fence_barrier_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, Cfg::TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
    grid_dependency_wait();                      // barriers and tensor memory are set up; now the previous launch's results may be read
    asm volatile("fence.proxy.async;" ::: "memory");   // ... by TMA, i.e. through the asynchronous proxy

    bool acc_ok = nk > 0;                        // the accumulator holds this CTA's partial sums (epilogue warps)
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        bool ok = true;
        for (int i = 0; i < nk && ok; ++i) {
            const int s = i % R;
            if (lane == 0) ok = wait_barrier(raw_empty(s), ((i / R) & 1) ^ 1, abort_flag, prm.status, (11 << 24) | (s << 16) | (tile & 0xFFFF));
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            if (lane == 0) ptx::mbar_arrive_expect_tx(raw_full(s), Cfg::A_BYTES + Cfg::B_RAW_BYTES);
            __syncwarp();
            const int kb = klo + (kb0 + i) * IBK;
            const uint32_t st = base + s * Cfg::RAW_BYTES;
            // A as stored m x k: one box of 128 rows x 32 k; as k x m: four boxes of 32 k-rows x 32 columns (lanes 0..3).
            // B as stored k x n: BN / 32 boxes of 32 k-rows x 32 columns; as n x k: one box of BN rows x 32 k (lanes 4..7).
            if (lane < 4) {
                if (!TA && lane == 0) ptx::tma_load_2d(st, &map_a, kb, r0, raw_full(s));
                if (TA) ptx::tma_load_2d(st + lane * 4096, &map_a, r0 + 32 * lane, kb, raw_full(s));
            } else if (lane < 8) {
                const int j = lane - 4;
                if (!TB && j < BN / 32) ptx::tma_load_2d(st + Cfg::A_BYTES + j * 4096, &map_b, c0 + 32 * j, kb, raw_full(s));
                if (TB && j == 0) ptx::tma_load_2d(st + Cfg::A_BYTES, &map_b, kb, c0, raw_full(s));
            }
        }
        if (*abort_flag && lane == 0) {          // failure path: loads still in flight land before the CTA's memory goes away
            const unsigned long long t0 = global_ns();
            while (global_ns() - t0 < 200000ull) { }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::instr_desc_tf32(IBM, BN, 0, 0);
            uint32_t accumulate = 0;
            bool ok = true;
            // The wait for the NEXT k-block's operands sits before the last MMAs of this one: while the issuer is in it the tensor
            // pipe still has queued work, so the pipe does not run dry between k-blocks.
            const uint64_t desc0 = kmajor_desc128(split_base, 0);            // descriptors differ only in the address field
            if (nk > 0) ok = wait_barrier(ready(0), 0, abort_flag, prm.status, (12 << 24) | (tile & 0xFFFF));
            for (int i = 0; i < nk && ok; ++i) {
                const int s = i % S;
                ptx::tc_fence_after_sync();
                const uint32_t a_hi = tmem_base + BN + s * Cfg::A_COLS, a_lo = a_hi + IBK;      // tensor-memory columns
                const uint64_t db_hi = desc0 + (uint64_t)((s * Cfg::SPLIT_BYTES) >> 4), db_lo = db_hi + (Cfg::B_PLANE_BYTES >> 4);
#pragma unroll
                for (int ks = 0; ks < IBK / 8; ++ks) {
                    if (ks == IBK / 8 - 1 && i + 1 < nk) {
                        const int sn = (i + 1) % S;
                        ok = wait_barrier(ready(sn), ((i + 1) / S) & 1, abort_flag, prm.status, (12 << 24) | (sn << 16) | (tile & 0xFFFF));
                    }
                    ptx::mma_tf32_a_tmem(tmem_base, a_lo + 8 * ks, db_hi + 2 * ks, idesc, accumulate);   // small terms first
                    ptx::mma_tf32_a_tmem(tmem_base, a_hi + 8 * ks, db_lo + 2 * ks, idesc, 1);
                    ptx::mma_tf32_a_tmem(tmem_base, a_hi + 8 * ks, db_hi + 2 * ks, idesc, 1);
                    accumulate = 1;
                }
                ptx::mma_commit(empty(s));                   // the stage may be refilled once these MMAs have read it
            }
            if (ok && nk > 0) ptx::mma_commit(acc_full);
            if (*abort_flag) {                               // failure path: issued MMAs finish before tensor memory is freed
                ptx::mma_commit(drain);
                for (uint32_t i = 0; i < (1u << 20); ++i)
                    if (ptx::mbar_try_wait(drain, 0)) break;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ transform (warps 2..9), then epilogue
        const int w2 = warp - 2;
        const Transform<BN, TA, TB> xf(w2, lane);
        const uint32_t a_dst = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + BN + 16 * (w2 >> 2);
        bool ok = true;
        uint8_t *const split_ptr = base_ptr + R * Cfg::RAW_BYTES;
        for (int i = 0; i < nk && ok; ++i) {
            const int rs = i % R, s = i % S;
            if (lane == 0)
                ok = wait_barrier(raw_full(rs), (i / R) & 1, abort_flag, prm.status, (13 << 24) | (rs << 16) | (tile & 0xFFFF)) &&
                     wait_barrier(empty(s), ((i / S) & 1) ^ 1, abort_flag, prm.status, (15 << 24) | (s << 16) | (tile & 0xFFFF));
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            uint8_t *const st = base_ptr + rs * Cfg::RAW_BYTES;
            ptx::tc_fence_after_sync();                      // the MMAs that read this split stage (tensor memory and B's tiles) are done
            uint8_t *const bhi = split_ptr + s * Cfg::SPLIT_BYTES;
            xf.run(st, st + Cfg::A_BYTES, a_dst + s * Cfg::A_COLS, bhi, bhi + Cfg::B_PLANE_BYTES);
            if (lane == 0) { ptx::mbar_arrive(ready(s)); ptx::mbar_arrive(raw_empty(rs)); }
        }
        // ---- epilogue: this warp reads TMEM lanes 32 q .. 32 q + 31 = rows of the tile; the two warps of a quarter share the columns
        const int q = warp & 3, row = q * 32 + lane, half = w2 >> 2;
        if (nk > 0 && ok) {
            if (lane == 0) ok = wait_barrier(acc_full, 0, abort_flag, prm.status, (14 << 24) | (tile & 0xFFFF));
            ok = __shfl_sync(0xffffffffu, ok, 0);
            ptx::tc_fence_after_sync();
        }
        acc_ok = nk > 0 && ok;
        const bool vec = (reinterpret_cast<uintptr_t>(prm.C) & 15) == 0 && (prm.n & 3) == 0;
        float *const P = reinterpret_cast<float *>(base_ptr);
#pragma unroll 1
        for (int c = half; c < BN / 32; c += 2) {
            const int col0 = c0 + 32 * c;
            float v[32];
            if (acc_ok) {
                ptx::tmem_ld_32cols(tmem_base + c * 32 + ((uint32_t)(q * 32) << 16), v);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = 0.0f;
            }
            if (split > 1) {
                // partial sums into this CTA's shared memory (every stage has been consumed by now)
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    *reinterpret_cast<float4 *>(P + row * Cfg::LDP + 32 * c + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            } else {
                store_chunk(P + w2 * STAGE_FLOATS, v, lane, r0 + q * 32, col0, prm, vec);
            }
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    if (split > 1) ptx::cluster_arrive();                    // this CTA's partial tile is written (the wait follows below)
    if (warp == 1) ptx::tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
    if (split == 1) return;

    // ---- split contraction: CTA `rank` finishes its rows of the tile, adding the cluster's partial tiles in k order
    ptx::cluster_wait();
    const float *const P = reinterpret_cast<const float *>(base_ptr);
    switch (split) {
        case 2: reduce_partial_tiles<BN, 2>(cluster, P, rank, r0, c0, prm); break;
        case 4: reduce_partial_tiles<BN, 4>(cluster, P, rank, r0, c0, prm); break;
        case 8: reduce_partial_tiles<BN, 8>(cluster, P, rank, r0, c0, prm); break;
        default: reduce_partial_tiles<BN, 16>(cluster, P, rank, r0, c0, prm); break;
    }
}


// ---------------------------------------------------------------------------------------------
// CTA-pair variant (cta_group::2): the two CTAs of a cluster share one 256 x (2 BNH) tile of the result.  Each CTA loads,
// splits and keeps its own 128 rows of A (in its tensor memory) and only its own BNH columns of B (K-major hi / lo tiles in
// its shared memory); the pair's tensor cores exchange the B halves, so per flop a CTA moves half the B bytes through its
// shared memory and the MMAs (M 256, N = 2 BNH), not shared memory, bound the mainloop.  The leader (cluster rank 0) issues
// every MMA; the transform warps of BOTH CTAs arrive on the leader's "ready" barrier (the peer's over the cluster, releasing
// what they wrote), tcgen05.commit with a CTA mask frees the split stage in both CTAs and publishes the accumulator to both
// epilogues.  No split of the contraction here: the variant is chosen when the pairs fill most of the machine.
// ---------------------------------------------------------------------------------------------
template <int BNH>
struct PairCfg {
    static constexpr int BN2 = 2 * BNH;                      // columns of the pair's tile = N of the MMA
    static constexpr int RAW = BNH == 64 ? 5 : 4, SPLIT = BNH == 64 ? 4 : 3;
    static constexpr int A_BYTES = IBM * IBK * 4;
    static constexpr int B_RAW_BYTES = IBK * BNH * 4;
    static constexpr int B_PLANE_BYTES = BNH * IBK * 4;
    static constexpr int RAW_BYTES = A_BYTES + B_RAW_BYTES, SPLIT_BYTES = 2 * B_PLANE_BYTES;
    static constexpr int RING_BYTES = RAW * RAW_BYTES + SPLIT * SPLIT_BYTES;
    static constexpr int A_COLS = 2 * IBK, TMEM_COLS = 512;
    static_assert(BN2 + SPLIT * A_COLS <= TMEM_COLS, "tensor memory budget");
    static constexpr int NUM_BARRIERS = 2 * RAW + 2 * SPLIT + 2;
    static constexpr int SMEM_BYTES = 1024 + RING_BYTES + 256;
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
};

template <int BNH>
__global__ void __launch_bounds__(ITHREADS, 1)
product_tc_inline_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const InlineParams prm) {
    using Cfg = PairCfg<BNH>;
    constexpr int R = Cfg::RAW, S = Cfg::SPLIT, BN2 = Cfg::BN2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ int abort_word;
    allow_dependents();
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *const base_ptr = smem_raw + (base - ptx::smem_u32(smem_raw));
    const uint32_t split_base = base + R * Cfg::RAW_BYTES;
    const uint32_t bars = base + Cfg::RING_BYTES;
    auto raw_full = [&](int s) { return bars + 8 * s; };                    // own TMA has delivered raw stage s
    auto raw_empty = [&](int s) { return bars + 8 * (R + s); };             // own transform warps have read it
    auto ready = [&](int s) { return bars + 8 * (2 * R + s); };             // leader only: both CTAs' transform warps have filled split stage s
    auto empty = [&](int s) { return bars + 8 * (2 * R + S + s); };         // the pair's MMAs on split stage s are done
    const uint32_t acc_full = bars + 8 * (2 * R + 2 * S), drain = acc_full + 8, tmem_slot = bars + 8 * Cfg::NUM_BARRIERS;
    volatile int *abort_flag = &abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_cta_rank();                           // 0 = leader
    const int tile = blockIdx.x >> 1;
    const int r0 = (tile / prm.tiles_n) * (2 * IBM), c0 = (tile % prm.tiles_n) * BN2;      // the pair's tile
    const int my_r0 = r0 + (int)rank * IBM, my_c0 = c0 + (int)rank * BNH;                  // this CTA's rows of A, columns of B

    int klo, khi;                                                            // the same in both CTAs
    tile_k_range(prm.pa, prm.pb, r0, min(r0 + 2 * IBM, prm.m), c0, min(c0 + BN2, prm.n), prm.k, &klo, &khi);
    klo &= ~(IBK - 1);
    const int nk = klo < khi ? (khi - klo + IBK - 1) / IBK : 0;

    if (threadIdx.x == 0) {
        abort_word = 0;
        for (int s = 0; s < R; ++s) { ptx::mbar_init(raw_full(s), 1); ptx::mbar_init(raw_empty(s), XFORM_WARPS); }
        for (int s = 0; s < S; ++s) { ptx::mbar_init(ready(s), 2 * XFORM_WARPS); ptx::mbar_init(empty(s), 1); }
        ptx::mbar_init(acc_full, 1);
        ptx::mbar_init(drain, 1);
        ptx::fence_barrier_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(tmem_slot, Cfg::TMEM_COLS);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    ptx::cluster_sync();                         // the peer's barriers exist before anything signals them
    ptx::tc_fence_after_sync();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));
    grid_dependency_wait();
    asm volatile("fence.proxy.async;" ::: "memory");

    bool acc_ok = nk > 0;
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs, own barriers)
        bool ok = true;
        for (int i = 0; i < nk && ok; ++i) {
            const int s = i % R;
            if (lane == 0) ok = wait_barrier(raw_empty(s), ((i / R) & 1) ^ 1, abort_flag, prm.status, (21 << 24) | (s << 16) | (tile & 0xFFFF));
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            if (lane == 0) ptx::mbar_arrive_expect_tx(raw_full(s), Cfg::RAW_BYTES);
            __syncwarp();
            const int kb = klo + i * IBK;
            const uint32_t st = base + s * Cfg::RAW_BYTES;
            if (lane == 0) ptx::tma_load_2d(st, &map_a, kb, my_r0, raw_full(s));
            else if (lane <= BNH / 32) ptx::tma_load_2d(st + Cfg::A_BYTES + (lane - 1) * 4096, &map_b, my_c0 + 32 * (lane - 1), kb, raw_full(s));
        }
        if (*abort_flag && lane == 0) {
            const unsigned long long t0 = global_ns();
            while (global_ns() - t0 < 200000ull) { }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA, one thread)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = ptx::instr_desc_tf32(2 * IBM, BN2, 0, 0);
            uint32_t accumulate = 0;
            bool ok = true;
            const uint64_t desc0 = kmajor_desc128(split_base, 0);
            if (nk > 0) ok = wait_barrier<true>(ready(0), 0, abort_flag, prm.status, (22 << 24) | (tile & 0xFFFF));
            for (int i = 0; i < nk && ok; ++i) {
                const int s = i % S;
                ptx::tc_fence_after_sync();
                const uint32_t a_hi = tmem_base + BN2 + s * Cfg::A_COLS, a_lo = a_hi + IBK;
                const uint64_t db_hi = desc0 + (uint64_t)((s * Cfg::SPLIT_BYTES) >> 4), db_lo = db_hi + (Cfg::B_PLANE_BYTES >> 4);
#pragma unroll
                for (int ks = 0; ks < IBK / 8; ++ks) {
                    if (ks == IBK / 8 - 1 && i + 1 < nk) {
                        const int sn = (i + 1) % S;
                        ok = wait_barrier<true>(ready(sn), ((i + 1) / S) & 1, abort_flag, prm.status, (22 << 24) | (sn << 16) | (tile & 0xFFFF));
                    }
                    ptx::mma_tf32_pair_a_tmem(tmem_base, a_lo + 8 * ks, db_hi + 2 * ks, idesc, accumulate);
                    ptx::mma_tf32_pair_a_tmem(tmem_base, a_hi + 8 * ks, db_lo + 2 * ks, idesc, 1);
                    ptx::mma_tf32_pair_a_tmem(tmem_base, a_hi + 8 * ks, db_hi + 2 * ks, idesc, 1);
                    accumulate = 1;
                }
                ptx::mma_commit_pair(empty(s), 3);           // both CTAs may refill this split stage
            }
            if (ok && nk > 0) ptx::mma_commit_pair(acc_full, 3);
            if (*abort_flag) {
                ptx::mma_commit_pair(drain, 1);
                for (uint32_t i = 0; i < (1u << 20); ++i)
                    if (ptx::mbar_try_wait(drain, 0)) break;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ transform (warps 2..9, both CTAs), then epilogue
        const int w2 = warp - 2;
        const Transform<BNH> xf(w2, lane);
        const uint32_t a_dst = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + BN2 + 16 * (w2 >> 2);
        bool ok = true;
        uint8_t *const split_ptr = base_ptr + R * Cfg::RAW_BYTES;
        for (int i = 0; i < nk && ok; ++i) {
            const int rs = i % R, s = i % S;
            if (lane == 0)
                ok = wait_barrier(raw_full(rs), (i / R) & 1, abort_flag, prm.status, (23 << 24) | (rs << 16) | (tile & 0xFFFF)) &&
                     wait_barrier(empty(s), ((i / S) & 1) ^ 1, abort_flag, prm.status, (25 << 24) | (s << 16) | (tile & 0xFFFF));
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            uint8_t *const st = base_ptr + rs * Cfg::RAW_BYTES;
            ptx::tc_fence_after_sync();
            uint8_t *const bhi = split_ptr + s * Cfg::SPLIT_BYTES;
            xf.run(st, st + Cfg::A_BYTES, a_dst + s * Cfg::A_COLS, bhi, bhi + Cfg::B_PLANE_BYTES);
            if (lane == 0) {
                ptx::mbar_arrive_cluster(ptx::map_to_cta(ready(s), 0));      // the leader's barrier, from either CTA
                ptx::mbar_arrive(raw_empty(rs));
            }
        }
        // ---- epilogue: this CTA's 128 rows of the accumulator
        const int q = warp & 3, half = w2 >> 2;
        if (nk > 0 && ok) {
            if (lane == 0) ok = wait_barrier(acc_full, 0, abort_flag, prm.status, (24 << 24) | (tile & 0xFFFF));
            ok = __shfl_sync(0xffffffffu, ok, 0);
            ptx::tc_fence_after_sync();
        }
        acc_ok = nk > 0 && ok;
        const bool vec = (reinterpret_cast<uintptr_t>(prm.C) & 15) == 0 && (prm.n & 3) == 0;
#pragma unroll 1
        for (int c = half; c < BN2 / 32; c += 2) {
            const int col0 = c0 + 32 * c;
            if (col0 >= prm.n) break;
            float v[32];
            if (acc_ok) {
                ptx::tmem_ld_32cols(tmem_base + c * 32 + ((uint32_t)(q * 32) << 16), v);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = 0.0f;
            }
            store_chunk(reinterpret_cast<float *>(base_ptr) + w2 * STAGE_FLOATS, v, lane, my_r0 + q * 32, col0, prm, vec);
        }
    }

    ptx::tc_fence_before_sync();
    ptx::cluster_sync();                                     // nobody leaves while the peer may still signal it or read its B tiles
    ptx::tc_fence_after_sync();
    if (warp == 1) ptx::tmem_dealloc_pair(tmem_base, Cfg::TMEM_COLS);
}

}  // namespace

bool product_tc_inline_takes(int64_t m, int64_t n, int64_t k, int lhs_transposed, int rhs_transposed, int pa, int pb) {
    auto plain = [](int p) { return p == MOM_GENERAL || p == MOM_LOWER_TRI || p == MOM_UPPER_TRI || p == MOM_SYMMETRIC; };
    // every matrix's row pitch is a multiple of 16 bytes: A is m x k, or k x m when stored transposed; B is k x n, or n x k; C is m x n
    return (k & 3) == 0 && (n & 3) == 0 && (!lhs_transposed || (m & 3) == 0) && plain(pa) && plain(pb) && m < (1 << 30) && n < (1 << 30) &&
           k < (1 << 30);
}

cudaError_t launch_product_tc_inline(const ProductArgs &a, int32_t *status, cudaStream_t stream) {
    if (!product_tc_inline_takes(a.m, a.n, a.k, a.transA, a.transB, a.pa, a.pb) || !status) return cudaErrorNotSupported;
    if ((reinterpret_cast<uintptr_t>(a.A) | reinterpret_cast<uintptr_t>(a.B)) & 15) return cudaErrorNotSupported;
    if (a.scaleA || a.scaleB || a.packedA || a.packedB || a.packedC) return cudaErrorNotSupported;
    const int sm_count = current_sm_count();
    if (sm_count < 1) return cudaErrorInvalidDevice;
    const int tiles_m = (a.m + IBM - 1) / IBM;
    const int kblocks = (a.k + IBK - 1) / IBK;
    // Tile width and k-slices per tile: the pair with the shortest critical path.  A wave of CTAs costs its fixed part (set-up, epilogue:
    // about 2 us at 64 columns, 2.5 us at 128), its k-blocks (measured: 0.66 us each at 64 columns, 0.9 us at 128) and, when the
    // contraction is split, the cluster's reduction (1.5 us); the launch itself is the same for all.  A cluster of s CTAs must sit in
    // one GPC and every CTA takes a whole SM here, so far fewer than SMs / s clusters run at once (148 / 74 / 33 / 15 on a B200): ask
    // the runtime.
    int bn = 64, split = 1;
    double best = 1e300;
    for (int width : {64, 128}) {
        const long long tiles = (long long)tiles_m * ((a.n + width - 1) / width);
        if (tiles * IMAX_SPLIT > (1ll << 30)) return cudaErrorNotSupported;
        for (int s = 1; s <= IMAX_SPLIT; s *= 2) {
            if (s > 1 && a.k / s < 2 * IBK) break;                           // every slice keeps two k-blocks
            int fit = sm_count / s;                                            // clusters that can run at once
            {
                std::lock_guard<std::mutex> lock(device_info_mutex());
                DeviceInfo *info = current_device_info();
                if (!info) return cudaErrorInvalidDevice;
                int &known = info->inline_clusters[width == 128][s == 1 ? 0 : s == 2 ? 1 : s == 4 ? 2 : s == 8 ? 3 : 4];
                if (known == 0) {
                    known = -1;
                    cudaLaunchConfig_t probe = {};
                    probe.gridDim = dim3((unsigned)(s * sm_count));
                    probe.blockDim = dim3(ITHREADS);
                    probe.dynamicSmemBytes = width == 128 ? InlineCfg<128>::SMEM_BYTES : InlineCfg<64>::SMEM_BYTES;
                    cudaLaunchAttribute at[1];
                    at[0].id = cudaLaunchAttributeClusterDimension;
                    at[0].val.clusterDim.x = (unsigned)s; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
                    probe.attrs = at;
                    probe.numAttrs = 1;
                    int n = 0;
                    cudaError_t e = width == 128 ? raise_smem_limit_locked(product_tc_inline_kernel<128>, InlineCfg<128>::SMEM_BYTES, &info->inline128_attr)
                                                 : raise_smem_limit_locked(product_tc_inline_kernel<64>, InlineCfg<64>::SMEM_BYTES, &info->inline64_attr);
                    if (e == cudaSuccess && s > 8)                            // beyond the portable cluster size: allowed per kernel
                        e = width == 128 ? cudaFuncSetAttribute(product_tc_inline_kernel<128>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1)
                                         : cudaFuncSetAttribute(product_tc_inline_kernel<64>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
                    if (e == cudaSuccess)
                        e = width == 128 ? cudaOccupancyMaxActiveClusters(&n, product_tc_inline_kernel<128>, &probe)
                                         : cudaOccupancyMaxActiveClusters(&n, product_tc_inline_kernel<64>, &probe);
                    if (e == cudaSuccess && n > 0) known = n;
                    else cudaGetLastError();
                }
                if (known > 0) fit = known;
                else if (s > 8) fit = 0;                                       // no cluster of 16 unless the runtime says it fits
            }
            if (fit < 1) continue;
            const long long waves = (tiles + fit - 1) / fit;
            const double cost = (double)waves * ((width == 128 ? 2.5 : 2.0) + ((kblocks + s - 1) / s) * (width == 128 ? 0.9 : 0.66) + (s > 8 ? 2.0 : s > 1 ? 1.5 : 0.0));
            if (cost < best) { best = cost; bn = width; split = s; }
        }
    }
    // CTA pairs (256 x 256 tiles, no split of the contraction): a k-block costs a pair about 1.2 us (its MMAs with A from tensor
    // memory: 12 x 170 cycles) for four times the result a single CTA's 0.9 us pays for; it wins when the pairs fill one wave
    // where single CTAs would need two.  (Pairs on 256 x 128 tiles were measured too: their MMAs take as long as the 256-wide
    // ones, so they never win.)
    int pair_bnh = 0;
    for (int bnh : {128}) {
        if (a.transA || a.transB) break;                                       // the pair form reads its operands as stored only
        const long long pairs = (long long)((a.m + 2 * IBM - 1) / (2 * IBM)) * ((a.n + 2 * bnh - 1) / (2 * bnh));
        if (pairs * 2 > (1ll << 30)) continue;
        int fit = sm_count / 2;
        {
            std::lock_guard<std::mutex> lock(device_info_mutex());
            DeviceInfo *info = current_device_info();
            if (!info) return cudaErrorInvalidDevice;
            int &known = info->inline_pair_clusters[bnh == 128];
            if (known == 0) {
                known = -1;
                cudaLaunchConfig_t probe = {};
                probe.gridDim = dim3((unsigned)(2 * sm_count));
                probe.blockDim = dim3(ITHREADS);
                probe.dynamicSmemBytes = PairCfg<128>::SMEM_BYTES;
                cudaLaunchAttribute at[1];
                at[0].id = cudaLaunchAttributeClusterDimension;
                at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
                probe.attrs = at;
                probe.numAttrs = 1;
                int n = 0;
                cudaError_t e = raise_smem_limit_locked(product_tc_inline_pair_kernel<128>, PairCfg<128>::SMEM_BYTES, &info->inline_pair_attr[1]);
                if (e == cudaSuccess) e = cudaOccupancyMaxActiveClusters(&n, product_tc_inline_pair_kernel<128>, &probe);
                if (e == cudaSuccess && n > 0) known = n;
                else cudaGetLastError();
            }
            if (known <= 0) continue;                                          // the pair kernel cannot be launched here
            fit = known;
        }
        const long long waves = (pairs + fit - 1) / fit;
        const double cost = (double)waves * (3.0 + kblocks * 1.2);
        if (cost < best) { best = cost; pair_bnh = bnh; }
    }
    const int tiles_n = pair_bnh ? (a.n + 2 * pair_bnh - 1) / (2 * pair_bnh) : (a.n + bn - 1) / bn;
    const long long tiles = pair_bnh ? (long long)((a.m + 2 * IBM - 1) / (2 * IBM)) * tiles_n : (long long)tiles_m * tiles_n;

    CUtensorMap map_a, map_b;
    if (!(a.transA ? tc_make_map(&map_a, a.A, a.k, a.m, IBK, 32, CU_TENSOR_MAP_SWIZZLE_128B)
                   : tc_make_map(&map_a, a.A, a.m, a.k, IBM, IBK, CU_TENSOR_MAP_SWIZZLE_128B)) ||
        !(a.transB ? tc_make_map(&map_b, a.B, a.n, a.k, bn, IBK, CU_TENSOR_MAP_SWIZZLE_128B)
                   : tc_make_map(&map_b, a.B, a.k, a.n, IBK, 32, CU_TENSOR_MAP_SWIZZLE_128B)))
        return cudaErrorNotSupported;
    InlineParams prm;
    prm.m = a.m; prm.n = a.n; prm.k = a.k;
    prm.pa = a.pa; prm.pb = a.pb; prm.pout = a.pout;
    prm.split = split;
    prm.tiles_n = tiles_n;
    prm.C = a.C;
    prm.add = a.add;
    prm.status = status;

    if (pair_bnh == 128)
        return launch_dependent(product_tc_inline_pair_kernel<128>, dim3((unsigned)(tiles * 2)), dim3(ITHREADS), PairCfg<128>::SMEM_BYTES, stream, 2u,
                                map_a, map_b, prm);
    // the kernel for this width and these storage orders; its shared-memory limit (and the cluster size beyond 8) is set per kernel
    using Kernel = void (*)(CUtensorMap, CUtensorMap, InlineParams);
    static const Kernel kernels[2][2][2] = {
        {{product_tc_inline_kernel<64, false, false>, product_tc_inline_kernel<64, false, true>},
         {product_tc_inline_kernel<64, true, false>, product_tc_inline_kernel<64, true, true>}},
        {{product_tc_inline_kernel<128, false, false>, product_tc_inline_kernel<128, false, true>},
         {product_tc_inline_kernel<128, true, false>, product_tc_inline_kernel<128, true, true>}}};
    const int wide = bn == 128, ta = a.transA != 0, tb = a.transB != 0;
    const Kernel kernel = kernels[wide][ta][tb];
    const int smem = wide ? InlineCfg<128>::SMEM_BYTES : InlineCfg<64>::SMEM_BYTES;
    {
        std::lock_guard<std::mutex> lock(device_info_mutex());
        DeviceInfo *info = current_device_info();
        if (!info) return cudaErrorInvalidDevice;
        cudaError_t e = raise_smem_limit_locked(kernel, smem, &info->inline_variant_attr[wide][ta][tb]);
        if (e == cudaSuccess && split > 8 && !info->inline_variant_np[wide][ta][tb]) {
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
            if (e == cudaSuccess) info->inline_variant_np[wide][ta][tb] = true;
        }
        if (e != cudaSuccess) return e;
    }
    return launch_dependent(kernel, dim3((unsigned)(tiles * split)), dim3(ITHREADS), (size_t)smem, stream, (unsigned)split, map_a, map_b, prm);
}

}  // namespace mom
