// Tensor-core product kernel: C = A*B (+ Add terms) with f32-level accuracy from three tcgen05
// kind::tf32 MMAs per k-step (3xTF32): with a = a_hi + a_lo and b = b_hi + b_lo (both halves exactly
// representable in tf32), C accumulates a_lo*b_hi + a_hi*b_lo + a_hi*b_hi in f32 in tensor memory.
//
// Data flow of one product step
//   1. split_planes_kernel writes the hi and lo planes of A (m x k, as stored) and of B TRANSPOSED
//      (n x k), so that both MMA operands are K-major.  Blocks that lie wholly outside a triangular
//      operand's structure are skipped: no tile ever reads them.
//   2. product_tc_kernel, persistent, one CTA per SM, walks a work-sorted tile table.  Per tile:
//        warp 0   TMA producer: per k-block loads A_hi, A_lo (128 rows x 32 k) and Bt_hi, Bt_lo
//                 (256 rows x 32 k), 128-byte rows with the 128B swizzle, into a 2-stage ring of
//                 96 KiB stages (64-byte rows cost twice the TMA requests per byte and ran 30 % slower);
//        warp 1   MMA issuer: 4 k-steps x 3 MMAs (M128 N256 K8) per stage into one of two 256-column
//                 accumulators in tensor memory; tcgen05.commit releases the stage / publishes the tile;
//        warps 2-5 epilogue: tcgen05.ld 32 columns at a time, Add terms, structure mask, swizzled
//                 staging in shared memory, TMA store (coalesced, clipped at the matrix edge).
//      The k-range of a tile is the intersection of the operands' structural ranges, so all-zero
//      blocks of triangular operands are never loaded or multiplied, and structurally-zero output
//      tiles are only zero-filled.
// Every wait is bounded: after a time limit the CTA records MOM_ERR_DEVICE_TIMEOUT and leaves.
#include <algorithm>
#include <cstring>
#include <vector>

#include <cuda.h>

#include "device_info.h"
#include "packed.cuh"
#include "product_tc.h"
#include "tc_probe.h"
#include "tc_ptx.cuh"
#include "tc_wait.cuh"

namespace mom {

namespace {

constexpr int BM = TC_BM, BN = TC_BN;
constexpr int BK = 32;                       // f32 elements per pipeline stage: one 128-byte swizzle row, four K=8 MMA steps
constexpr int STAGES = 2;
constexpr int ROW_BYTES = BK * 4;
constexpr CUtensorMapSwizzle OPERAND_TMA_SWIZZLE = BK == 32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
constexpr int A_PLANE_BYTES = BM * BK * 4;   // 16 KiB
constexpr int B_PLANE_BYTES = BN * BK * 4;   // 32 KiB
constexpr int STAGE_BYTES = 2 * A_PLANE_BYTES + 2 * B_PLANE_BYTES;   // 96 KiB
constexpr int EPI_BOX_BYTES = 32 * 32 * 4;   // 32 rows x 32 columns staged per TMA store
constexpr int EPI_BYTES = 4 * 2 * EPI_BOX_BYTES;                     // 4 warps x 2 buffers
constexpr int NUM_BARRIERS = 2 * STAGES + 4 + 1;
constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + EPI_BYTES + 256;
constexpr int THREADS = 192;
constexpr uint32_t TMEM_COLS = 512;          // two accumulators of BN columns

static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
static_assert(BM * (BN + 4) * 4 <= STAGES * STAGE_BYTES, "a partial tile fits where the stages were");
static_assert(SPLIT_BLOCK % BM == 0 && SPLIT_BLOCK % BN == 0, "split blocks must cover whole tiles");

struct Shared {
    uint32_t stage[STAGES];      // shared-space byte address of each stage
    uint32_t epi;                // staging buffers
    uint32_t full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], drain;
    uint32_t tmem_slot;
    volatile int *abort_flag;
};

// tile table entry: x = first row | k-slice << 24, y = first column, z..w = k-range
constexpr int TILE_SLICE_SHIFT = 24;
constexpr int TILE_ROW_MASK = (1 << TILE_SLICE_SHIFT) - 1;

// 16 bytes from the shared memory of CTA `rank` of this cluster, at this CTA's offset `addr`
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr, uint32_t rank) {
    float4 v;
    const uint32_t remote = ptx::map_to_cta(addr, rank);
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
    return v;
}
constexpr int CLUSTER_LDP = TC_BN + 4;       // row length (floats) of a partial tile in shared memory: 16-byte rows, conflict-free per 8 lanes

struct TcParams {
    const int4 *tiles;
    int num_tiles;
    int m, n;
    int pout;
    int out_mode;            // 0: f32 result through map_c; 1: hi/lo planes (map_c, map_c2); 2: transposed hi/lo planes
    int slice_rows;          // split-K: rows between the partial-sum slabs of consecutive k-slices (0: no split)
    int cluster_split;       // > 1 (1-CTA kernel): the k-slices of a tile are the CTAs of one thread-block cluster; they leave their partial
                             // tiles in shared memory and share out the tile's rows, adding the slices through distributed shared memory
    float *c_out;            // cluster_split: the result matrix (plain stores from the reduction)
    float *packed_c;         // not null (out_mode 0 only): the result is a packed triangle written in place with plain
                             // 16-byte stores; entries the container does not hold are not written at all
    int mirror;              // Gram product Y * Y^T (CTA-pair kernel, out_mode 0, Symmetric Add terms only): the table holds the tiles on and
                             // below the diagonal; a tile below it is also written transposed to its mirror position
    AddTerms add;
    int32_t *status;
};

// K-major operand tile whose rows are one swizzle span long (128 bytes under the 128B swizzle, or 64
// under the 64B one): 8-row groups are 8 rows apart; a K=8 step is 32 bytes along the row.
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t tile, int kstep) {
    return ptx::smem_desc(tile + kstep * 32, 16, 8 * ROW_BYTES, BK == 32 ? ptx::SWIZZLE_128B : ptx::SWIZZLE_64B);
}
// the rate probe's resident tiles: 64-byte rows, 64B swizzle
__device__ __forceinline__ uint64_t kmajor_desc_64(uint32_t tile) {
    return ptx::smem_desc(tile, 16, 512, ptx::SWIZZLE_64B);
}

// Epilogue of one 32-row x 32-column chunk held as one row per thread: Add terms, structure mask, then
// one of three outputs, each staged in shared memory under the 128B swizzle and written by TMA (coalesced,
// clipped at the matrix edge):
//   out_mode 0  the f32 values (the equation's result, or an intermediate read by an FFMA step);
//   out_mode 1  the hi and lo planes of the values, for a tensor-core step that takes them as left operand;
//   out_mode 2  the same planes transposed, for a tensor-core step that takes them as right operand.
// Writing the planes here saves the consumer's split pass and the f32 round trip through HBM.
__device__ __forceinline__ uint32_t round_tf32_bits(float a) { return (__float_as_uint(a) + 0x1000u) & 0xFFFFE000u; }

__device__ __forceinline__ void epilogue_chunk(const TcParams &prm, const CUtensorMap *map_c, const CUtensorMap *map_c2,
                                               float (&v)[32], int r, int row0, int col0, int lane, uint32_t stage_buf,
                                               uint32_t &store_it, bool mirror_this = false) {
    const bool row_ok = r < prm.m;
    for (int a = 0; a < prm.add.count; ++a) {                   // Add terms, left to right
        const float *p = prm.add.ptr[a];
        if (p && ((prm.add.transposed >> a) & 1u)) {             // term stored as n x m: column-wise reads
            if (row_ok) {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (col0 + j < prm.n) v[j] += __ldcg(p + (long long)(col0 + j) * prm.m + r);
            }
        } else if (p) {
            if (row_ok) {
                const float4 *src = reinterpret_cast<const float4 *>(p + (long long)r * prm.n + col0);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (col0 + 4 * j < prm.n) {
                        const float4 x = __ldcg(src + j);
                        v[4 * j] += x.x; v[4 * j + 1] += x.y; v[4 * j + 2] += x.z; v[4 * j + 3] += x.w;
                    }
                }
            }
        } else {                                                 // Identity term
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] += (col0 + j == r) ? 1.0f : 0.0f;
        }
    }
    if (prm.pout != MOM_GENERAL) {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = in_structure(prm.pout, r, col0 + j) ? v[j] : 0.0f;
    }
    if (prm.packed_c) {
        // packed triangle: this thread's row holds columns [first, end); every 16-byte group of the chunk that lies in
        // that range goes straight to its place (a lane writes whole 16-byte groups of its own row)
        if (row_ok) {
            const PackedRow row = packed_row(prm.pout == MOM_LOWER_TRI, prm.m, r);
            float *dst = prm.packed_c + row.offset - row.first;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int c = col0 + 4 * j;
                if (c >= row.first && c < row.end)
                    *reinterpret_cast<float4 *>(dst + c) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            }
        }
        return;
    }
    const int passes = prm.out_mode == 0 ? (mirror_this ? 2 : 1) : 2;   // f32 (and its mirror image), or hi then lo
#pragma unroll 1
    for (int pass = 0; pass < passes; ++pass) {
        const uint32_t buf = stage_buf + (store_it & 1) * EPI_BOX_BYTES;
        if (lane == 0) ptx::tma_store_wait_read<1>();            // the store that last read this buffer is done
        __syncwarp();
        const bool transposed_box = prm.out_mode == 2 || (prm.out_mode == 0 && pass == 1);
        if (!transposed_box) {
            // 32 rows of 128 bytes: 16-byte chunk j of row i stored at chunk j ^ (i & 7)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float x = v[4 * j + e];
                    const float hi = __uint_as_float(round_tf32_bits(x));
                    w[e] = prm.out_mode == 0 ? x : pass == 0 ? hi : __uint_as_float(round_tf32_bits(x - hi));
                }
                const uint32_t dst = buf + lane * 128 + ((j ^ (lane & 7)) << 4);
                asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(w[0]), "f"(w[1]), "f"(w[2]), "f"(w[3]) : "memory");
            }
        } else {
            // transposed box: row j of the box is output column col0 + j, position lane is output row row0 + lane
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float x = v[j];
                const float hi = __uint_as_float(round_tf32_bits(x));
                const float w = prm.out_mode == 0 ? x : pass == 0 ? hi : __uint_as_float(round_tf32_bits(x - hi));
                const uint32_t dst = buf + j * 128 + ((((uint32_t)lane >> 2) ^ (j & 7)) << 4) + ((lane & 3) << 2);
                asm volatile("st.shared.f32 [%0], %1;" ::"r"(dst), "f"(w) : "memory");
            }
        }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            const CUtensorMap *map = pass == 0 || prm.out_mode == 0 ? map_c : map_c2;
            if (!transposed_box) ptx::tma_store_2d(map, col0, row0, buf);
            else ptx::tma_store_2d(map, row0, col0, buf);
            ptx::tma_store_commit();
        }
        ++store_it;
    }
}

__global__ void __launch_bounds__(THREADS, 1)
product_tc_kernel(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
                  const __grid_constant__ CUtensorMap map_b_hi, const __grid_constant__ CUtensorMap map_b_lo,
                  const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_c2, const TcParams prm) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ int abort_word;
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = base + STAGES * STAGE_BYTES + EPI_BYTES;
    Shared sh;
#pragma unroll
    for (int s = 0; s < STAGES; ++s) {
        sh.stage[s] = base + s * STAGE_BYTES;
        sh.full[s] = bars + 8 * s;
        sh.empty[s] = bars + 8 * (STAGES + s);
    }
    sh.epi = base + STAGES * STAGE_BYTES;
    sh.tmem_full[0] = bars + 8 * (2 * STAGES);
    sh.tmem_full[1] = bars + 8 * (2 * STAGES + 1);
    sh.tmem_empty[0] = bars + 8 * (2 * STAGES + 2);
    sh.tmem_empty[1] = bars + 8 * (2 * STAGES + 3);
    sh.drain = bars + 8 * (2 * STAGES + 4);
    sh.tmem_slot = bars + 8 * NUM_BARRIERS;
    sh.abort_flag = &abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        abort_word = 0;
#pragma unroll
        for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(sh.full[s], 1); ptx::mbar_init(sh.empty[s], 1); }
        ptx::mbar_init(sh.tmem_full[0], 1);
        ptx::mbar_init(sh.tmem_full[1], 1);
        ptx::mbar_init(sh.tmem_empty[0], 4);
        ptx::mbar_init(sh.tmem_empty[1], 4);
        ptx::mbar_init(sh.drain, 1);
        ptx::fence_barrier_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(sh.tmem_slot, TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(sh.tmem_slot));

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        uint32_t it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < prm.num_tiles && ok; t += gridDim.x) {
            const int4 tile = prm.tiles[t];
            for (int kb = tile.z; kb < tile.w; kb += BK, ++it) {
                const int s = it % STAGES;
                const uint32_t parity = ((it / STAGES) & 1) ^ 1;
                if (lane == 0) ok = wait_barrier(sh.empty[s], parity, sh.abort_flag, prm.status, (1 << 24) | (s << 16) | (t & 0xFFFF));
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                if (lane == 0) ptx::mbar_arrive_expect_tx(sh.full[s], STAGE_BYTES);
                __syncwarp();
                const int a_row = tile.x & TILE_ROW_MASK;            // (the k-slice index rides in the top bits)
                if (lane == 0) ptx::tma_load_2d(sh.stage[s], &map_a_hi, kb, a_row, sh.full[s]);
                else if (lane == 1) ptx::tma_load_2d(sh.stage[s] + A_PLANE_BYTES, &map_a_lo, kb, a_row, sh.full[s]);
                else if (lane == 2) ptx::tma_load_2d(sh.stage[s] + 2 * A_PLANE_BYTES, &map_b_hi, kb, tile.y, sh.full[s]);
                else if (lane == 3) ptx::tma_load_2d(sh.stage[s] + 2 * A_PLANE_BYTES + B_PLANE_BYTES, &map_b_lo, kb, tile.y, sh.full[s]);
            }
        }
        // On the failure path, let loads that are still in flight land before the CTA exits.
        if (*sh.abort_flag && lane == 0) {
            for (uint32_t back = 1; back <= (uint32_t)STAGES && back <= it; ++back) {
                const uint32_t j = it - back;
                for (uint32_t i = 0; i < (1u << 20); ++i)
                    if (ptx::mbar_try_wait(sh.full[j % STAGES], (j / STAGES) & 1)) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::instr_desc_tf32(BM, BN, 0, 0);
            uint32_t it = 0, acc_it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < prm.num_tiles && ok; t += gridDim.x) {
                const int4 tile = prm.tiles[t];
                if (tile.z >= tile.w) continue;                  // structurally zero: nothing to multiply
                const uint32_t acc = acc_it & 1;
                ok = wait_barrier(sh.tmem_empty[acc], ((acc_it >> 1) & 1) ^ 1, sh.abort_flag, prm.status, (2 << 24) | (acc << 16) | (t & 0xFFFF));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d = tmem_base + acc * BN;
                uint32_t accumulate = 0;
                for (int kb = tile.z; kb < tile.w; kb += BK, ++it) {
                    const int s = it % STAGES;
                    ok = wait_barrier(sh.full[s], (it / STAGES) & 1, sh.abort_flag, prm.status, (3 << 24) | (s << 16) | (t & 0xFFFF));
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_hi = sh.stage[s], a_lo = a_hi + A_PLANE_BYTES;
                    const uint32_t b_hi = a_hi + 2 * A_PLANE_BYTES, b_lo = b_hi + B_PLANE_BYTES;
#pragma unroll
                    for (int ks = 0; ks < BK / 8; ++ks) {
                        const uint64_t da_hi = kmajor_desc(a_hi, ks), da_lo = kmajor_desc(a_lo, ks);
                        const uint64_t db_hi = kmajor_desc(b_hi, ks), db_lo = kmajor_desc(b_lo, ks);
                        ptx::mma_tf32(d, da_lo, db_hi, idesc, accumulate);      // small terms first
                        ptx::mma_tf32(d, da_hi, db_lo, idesc, 1);
                        ptx::mma_tf32(d, da_hi, db_hi, idesc, 1);
                        accumulate = 1;
                    }
                    ptx::mma_commit(sh.empty[s]);                 // stage reusable once these MMAs have read it
                }
                if (!ok) break;
                ptx::mma_commit(sh.tmem_full[acc]);               // accumulator complete
                ++acc_it;
            }
            if (*sh.abort_flag) {                                 // failure path: let issued MMAs finish before TMEM is freed
                ptx::mma_commit(sh.drain);
                for (uint32_t i = 0; i < (1u << 20); ++i)
                    if (ptx::mbar_try_wait(sh.drain, 0)) break;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;                                   // TMEM lane quarter this warp may read
        const uint32_t stage_buf = sh.epi + (warp - 2) * 2 * EPI_BOX_BYTES;
        uint32_t acc_it = 0, store_it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < prm.num_tiles && ok; t += gridDim.x) {
            const int4 tile = prm.tiles[t];
            const bool zero_tile = tile.z >= tile.w;
            const uint32_t acc = acc_it & 1;
            if (!zero_tile) {
                ok = wait_barrier(sh.tmem_full[acc], (acc_it >> 1) & 1, sh.abort_flag, prm.status, (4 << 24) | (acc << 16) | (t & 0xFFFF));
                if (!ok) break;
                ptx::tc_fence_after_sync();
            }
            const int slab_row = (tile.x & TILE_ROW_MASK) + q * 32;   // first row of this warp's slab
            const int r = slab_row + lane;                        // this thread's output row
            const int rows_left = prm.m - slab_row;               // rows of the slab inside the matrix
            // split-K: slice i of a tile stores its partial sums into slab i of the scratch matrix
            const int store_row = slab_row + (int)((unsigned)tile.x >> TILE_SLICE_SHIFT) * prm.slice_rows;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                const int col0 = tile.y + c * 32;
                if (col0 >= prm.n) break;
                float v[32];
                if (!zero_tile) {
                    ptx::tmem_ld_32cols(tmem_base + acc * BN + c * 32 + ((uint32_t)(q * 32) << 16), v);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0.0f;
                }
                if (prm.cluster_split > 1) {
                    // every stage has been consumed by now (the accumulator is complete): the partial tile takes their place
                    const uint32_t dst = base + (uint32_t)((q * 32 + lane) * CLUSTER_LDP + c * 32) * 4u;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst + 16 * j), "f"(v[4 * j]), "f"(v[4 * j + 1]), "f"(v[4 * j + 2]),
                                     "f"(v[4 * j + 3]) : "memory");
                } else if (rows_left > 0) {
                    epilogue_chunk(prm, &map_c, &map_c2, v, r, store_row, col0, lane, stage_buf, store_it);
                }
            }
            if (!zero_tile) {
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(sh.tmem_empty[acc]);
                ++acc_it;
            }
        }
        if (lane == 0) ptx::tma_store_wait_all();
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    if (warp == 1) ptx::tmem_dealloc(tmem_base, TMEM_COLS);

    if (prm.cluster_split > 1) {
        // ---- split contraction inside a cluster: CTA `rank` finishes rows [rank * 128 / s, (rank + 1) * 128 / s) of the tile, adding the
        // cluster's partial tiles in k order (deterministic); Add terms and mask as in the ordinary epilogue, 16-byte stores
        const int split = prm.cluster_split;
        const uint32_t rank = ptx::cluster_cta_rank();
        const int4 tile = prm.tiles[blockIdx.x];
        const int r0 = tile.x & TILE_ROW_MASK, c0 = tile.y;
        ptx::cluster_sync();                                  // every CTA of the cluster comes here, also one that gave up
        const int rows_per = BM / split;
        const bool vec = (reinterpret_cast<uintptr_t>(prm.c_out) & 15) == 0;
        for (int e = threadIdx.x; e < rows_per * (BN / 4); e += THREADS) {
            const int row = (int)rank * rows_per + e / (BN / 4), col = (e % (BN / 4)) << 2;
            const int r = r0 + row, cc = c0 + col;
            if (r >= prm.m || cc >= prm.n) continue;
            float w[4] = {0.f, 0.f, 0.f, 0.f};
            for (int peer = 0; peer < split; ++peer) {
                const float4 x = ld_cluster_f4(base + (uint32_t)(row * CLUSTER_LDP + col) * 4u, (uint32_t)peer);
                w[0] += x.x; w[1] += x.y; w[2] += x.z; w[3] += x.w;
            }
            finish_row4(w, prm.add, 0, r, cc, prm.n, prm.n, prm.pout, vec);
            float *dst = prm.c_out + (long long)r * prm.n + cc;
            if (vec && cc + 3 < prm.n) {
                *reinterpret_cast<float4 *>(dst) = make_float4(w[0], w[1], w[2], w[3]);
            } else {
                for (int j = 0; j < 4; ++j)
                    if (cc + j < prm.n) dst[j] = w[j];
            }
        }
        ptx::cluster_sync();                                  // nobody leaves while a peer may still read its tile
    }
}

// ---------------------------------------------------------------------------------------------
// CTA-pair variant (cta_group::2): two CTAs of a cluster share one 256 x 256 output tile.  Each CTA
// loads its own 128 rows of A and only its own half (128 columns) of B -- the tensor cores of the pair
// exchange the B halves -- so a stage is 64 KiB instead of 96 (three stages fit) and the L2 / shared
// memory traffic per flop drops by a third.  The leader CTA (cluster rank 0) issues every MMA.  Only the
// leader's "full" barriers are used: the leader's producer arms one with the bytes of both CTAs' loads and
// the peer's TMA loads report their bytes there (cta_group::2 form), so no thread-level message crosses
// the pair on the way in.  (Two variants were slower: the peer also arriving remotely on that barrier, and
// each CTA counting its own loads with a per-stage relay to the leader.)  tcgen05.commit with a CTA mask
// releases the stage in both CTAs and publishes the accumulator to both epilogues; the peer's epilogue
// warps tell the leader over the cluster when an accumulator may be overwritten.
// ---------------------------------------------------------------------------------------------
constexpr int P_BM = 2 * BM;                  // rows of a pair tile
constexpr int P_STAGES = 3;
constexpr int P_A_PLANE_BYTES = BM * BK * 4;          // 16 KiB: this CTA's 128 rows
constexpr int P_B_PLANE_BYTES = (BN / 2) * BK * 4;    // 16 KiB: this CTA's 128 columns of B
constexpr int P_STAGE_BYTES = 2 * P_A_PLANE_BYTES + 2 * P_B_PLANE_BYTES;   // 64 KiB
constexpr int P_NUM_BARRIERS = 2 * P_STAGES + 4 + 1;
constexpr int P_SMEM_BYTES = 1024 + P_STAGES * P_STAGE_BYTES + EPI_BYTES + 256;
static_assert(P_SMEM_BYTES <= 227 * 1024, "shared memory budget");

__global__ void __launch_bounds__(THREADS, 1)
product_tc_pair_kernel(const __grid_constant__ CUtensorMap map_a_hi, const __grid_constant__ CUtensorMap map_a_lo,
                       const __grid_constant__ CUtensorMap map_b_hi, const __grid_constant__ CUtensorMap map_b_lo,
                       const __grid_constant__ CUtensorMap map_c, const __grid_constant__ CUtensorMap map_c2, const TcParams prm) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ int abort_word;
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t epi = base + P_STAGES * P_STAGE_BYTES;
    const uint32_t bars = epi + EPI_BYTES;
    auto stage_addr = [&](int s) { return base + s * P_STAGE_BYTES; };
    auto full_bar = [&](int s) { return bars + 8 * s; };
    auto empty_bar = [&](int s) { return bars + 8 * (P_STAGES + s); };
    auto tmem_full_bar = [&](int a) { return bars + 8 * (2 * P_STAGES + a); };
    auto tmem_empty_bar = [&](int a) { return bars + 8 * (2 * P_STAGES + 2 + a); };
    const uint32_t drain_bar = bars + 8 * (2 * P_STAGES + 4);
    const uint32_t tmem_slot = bars + 8 * P_NUM_BARRIERS;
    volatile int *abort_flag = &abort_word;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_cta_rank();           // 0 = leader
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        abort_word = 0;
        for (int s = 0; s < P_STAGES; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), 1); }
        ptx::mbar_init(tmem_full_bar(0), 1);
        ptx::mbar_init(tmem_full_bar(1), 1);
        ptx::mbar_init(tmem_empty_bar(0), 8);               // four epilogue warps in each CTA
        ptx::mbar_init(tmem_empty_bar(1), 8);
        ptx::mbar_init(drain_bar, 1);
        ptx::fence_barrier_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(tmem_slot, TMEM_COLS);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    ptx::cluster_sync();                                     // the peer's barriers exist before anything signals them
    ptx::tc_fence_after_sync();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(tmem_slot));

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        uint32_t it = 0;
        bool ok = true;
        for (int t = pair; t < prm.num_tiles && ok; t += num_pairs) {
            const int4 tile = prm.tiles[t];
            for (int kb = tile.z; kb < tile.w; kb += BK, ++it) {
                const int s = it % P_STAGES;
                const uint32_t parity = ((it / P_STAGES) & 1) ^ 1;
                if (lane == 0) ok = wait_barrier(empty_bar(s), parity, abort_flag, prm.status, (1 << 24) | (s << 16) | (t & 0xFFFF));
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                // Both CTAs' loads are counted on the leader's barrier: the leader alone arms it with the bytes of
                // the whole pair, the peer's TMA reports its bytes there (cta_group::2 form).
                const uint32_t bar = rank == 0 ? full_bar(s) : ptx::map_to_cta(full_bar(s), 0);
                if (lane == 0 && rank == 0) ptx::mbar_arrive_expect_tx(full_bar(s), 2 * P_STAGE_BYTES);
                __syncwarp();
                const uint32_t st = stage_addr(s);
                const int a_row = tile.x + (int)rank * BM, b_row = tile.y + (int)rank * (BN / 2);
                if (lane == 0) ptx::tma_load_2d_pair(st, &map_a_hi, kb, a_row, bar);
                else if (lane == 1) ptx::tma_load_2d_pair(st + P_A_PLANE_BYTES, &map_a_lo, kb, a_row, bar);
                else if (lane == 2) ptx::tma_load_2d_pair(st + 2 * P_A_PLANE_BYTES, &map_b_hi, kb, b_row, bar);
                else if (lane == 3) ptx::tma_load_2d_pair(st + 2 * P_A_PLANE_BYTES + P_B_PLANE_BYTES, &map_b_lo, kb, b_row, bar);
            }
        }
        // failure path: give loads that are still in flight time to land before this CTA's memory goes away
        if (*abort_flag && lane == 0) {
            const unsigned long long t0 = global_ns();
            while (global_ns() - t0 < 200000ull) { }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA, one thread)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = ptx::instr_desc_tf32(P_BM, BN, 0, 0);
            uint32_t it = 0, acc_it = 0;
            bool ok = true;
            for (int t = pair; t < prm.num_tiles && ok; t += num_pairs) {
                const int4 tile = prm.tiles[t];
                if (tile.z >= tile.w) continue;
                const uint32_t acc = acc_it & 1;
                ok = wait_barrier(tmem_empty_bar(acc), ((acc_it >> 1) & 1) ^ 1, abort_flag, prm.status, (2 << 24) | (acc << 16) | (t & 0xFFFF));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d = tmem_base + acc * BN;
                uint32_t accumulate = 0;
                for (int kb = tile.z; kb < tile.w; kb += BK, ++it) {
                    const int s = it % P_STAGES;
                    ok = wait_barrier(full_bar(s), (it / P_STAGES) & 1, abort_flag, prm.status, (3 << 24) | (s << 16) | (t & 0xFFFF));
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    const uint32_t a_hi = stage_addr(s), a_lo = a_hi + P_A_PLANE_BYTES;
                    const uint32_t b_hi = a_hi + 2 * P_A_PLANE_BYTES, b_lo = b_hi + P_B_PLANE_BYTES;
#pragma unroll
                    for (int ks = 0; ks < BK / 8; ++ks) {
                        const uint64_t da_hi = kmajor_desc(a_hi, ks), da_lo = kmajor_desc(a_lo, ks);
                        const uint64_t db_hi = kmajor_desc(b_hi, ks), db_lo = kmajor_desc(b_lo, ks);
                        ptx::mma_tf32_pair(d, da_lo, db_hi, idesc, accumulate);
                        ptx::mma_tf32_pair(d, da_hi, db_lo, idesc, 1);
                        ptx::mma_tf32_pair(d, da_hi, db_hi, idesc, 1);
                        accumulate = 1;
                    }
                    ptx::mma_commit_pair(empty_bar(s), 3);           // both CTAs may refill this stage
                }
                if (!ok) break;
                ptx::mma_commit_pair(tmem_full_bar(acc), 3);          // both epilogues may read
                ++acc_it;
            }
            if (*abort_flag) {
                ptx::mma_commit_pair(drain_bar, 1);
                for (uint32_t i = 0; i < (1u << 20); ++i)
                    if (ptx::mbar_try_wait(drain_bar, 0)) break;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
        const int q = warp & 3;
        const uint32_t stage_buf = epi + (warp - 2) * 2 * EPI_BOX_BYTES;
        uint32_t acc_it = 0, store_it = 0;
        bool ok = true;
        for (int t = pair; t < prm.num_tiles && ok; t += num_pairs) {
            const int4 tile = prm.tiles[t];
            const bool zero_tile = tile.z >= tile.w;
            const uint32_t acc = acc_it & 1;
            if (!zero_tile) {
                ok = wait_barrier(tmem_full_bar(acc), (acc_it >> 1) & 1, abort_flag, prm.status, (4 << 24) | (acc << 16) | (t & 0xFFFF));
                if (!ok) break;
                ptx::tc_fence_after_sync();
            }
            const int row0 = tile.x + (int)rank * BM + q * 32;   // first row of this warp's slab
            const int r = row0 + lane;
            const int rows_left = prm.m - row0;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                const int col0 = tile.y + c * 32;
                if (col0 >= prm.n) break;
                float v[32];
                if (!zero_tile) {
                    ptx::tmem_ld_32cols(tmem_base + acc * BN + c * 32 + ((uint32_t)(q * 32) << 16), v);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0.0f;
                }
                if (rows_left > 0)
                    epilogue_chunk(prm, &map_c, &map_c2, v, r, row0, col0, lane, stage_buf, store_it,
                                   prm.mirror != 0 && tile.y < (tile.x & TILE_ROW_MASK));
            }
            if (!zero_tile) {
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(tmem_empty_bar(acc), 0));
                ++acc_it;
            }
        }
        if (lane == 0) ptx::tma_store_wait_all();
    }

    ptx::tc_fence_before_sync();
    ptx::cluster_sync();                                     // nobody leaves while the peer may still signal it
    ptx::tc_fence_after_sync();
    if (warp == 1) ptx::tmem_dealloc_pair(tmem_base, TMEM_COLS);
}

// hi = rna_tf32(a), lo = rna_tf32(a - hi).  The planes keep the operand's layout (rows x cols) or, with
// TRANSPOSE, hold the transposed operand (cols x rows).  One CTA handles a 64 x 64 piece; pieces whose
// enclosing SPLIT_BLOCK x SPLIT_BLOCK block lies wholly outside a triangular operand's structure are
// skipped (no product tile reads them).  rows and cols are multiples of 4 wherever a vector access
// needs it: the plain path needs cols % 4 == 0, the transposing path rows % 4 == 0.
constexpr int SPLIT_PIECE = 64;

// Optional scaling folded into the split (a product with a Diagonal factor whose only reader is this
// operand): entry (r, c) of the matrix as stored is multiplied by d[r] (by_row) or d[c] before it is split;
// d's entries are `step` floats apart (the diagonal of a dense matrix).  d == NULL: no scaling.
struct SplitScale {
    const float *d;
    long long step;
    int by_row;
};

// `packed`: the source is a packed triangle (see packed.cuh) read in place: entry (r, c) sits at its row's offset, and
// what the container does not hold reads as zero.  The planes are dense either way (TMA addresses them).
template <bool TRANSPOSE>
__device__ __forceinline__ void split_piece(const float *__restrict__ src, float *__restrict__ hi, float *__restrict__ lo, int rows,
                                            int cols, int prop, const SplitScale &sc, int piece_x, int piece_y, int packed) {
    const int pr = piece_y * SPLIT_PIECE, pc = piece_x * SPLIT_PIECE;
    const int br = pr / SPLIT_BLOCK * SPLIT_BLOCK, bc = pc / SPLIT_BLOCK * SPLIT_BLOCK;
    if (prop == MOM_LOWER_TRI && bc > br + SPLIT_BLOCK - 1) return;     // block wholly above the diagonal
    if (prop == MOM_UPPER_TRI && br > bc + SPLIT_BLOCK - 1) return;     // wholly below
    if (!TRANSPOSE) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = threadIdx.x + 256 * i;                         // 64 rows x 16 float4
            const int r = pr + (e >> 4), c = pc + ((e & 15) << 2);
            if (r < rows && c < cols) {
                const size_t off = (size_t)r * cols + c;
                float4 a;
                if (packed) {
                    const PackedRow row = packed_row(prop == MOM_LOWER_TRI, rows, r);
                    a = c >= row.first && c < row.end ? __ldcg(reinterpret_cast<const float4 *>(src + row.offset + (c - row.first)))
                                                      : make_float4(0.f, 0.f, 0.f, 0.f);
                } else {
                    a = __ldcg(reinterpret_cast<const float4 *>(src + off));
                }
                if (sc.d) {
                    if (sc.by_row) {
                        const float f = __ldcg(sc.d + r * sc.step);
                        a.x *= f; a.y *= f; a.z *= f; a.w *= f;
                    } else {
                        a.x *= __ldcg(sc.d + c * sc.step); a.y *= __ldcg(sc.d + (c + 1) * sc.step);
                        a.z *= __ldcg(sc.d + (c + 2) * sc.step); a.w *= __ldcg(sc.d + (c + 3) * sc.step);
                    }
                }
                float4 h, l;
                h.x = ptx::to_tf32(a.x); h.y = ptx::to_tf32(a.y); h.z = ptx::to_tf32(a.z); h.w = ptx::to_tf32(a.w);
                l.x = ptx::to_tf32(a.x - h.x); l.y = ptx::to_tf32(a.y - h.y); l.z = ptx::to_tf32(a.z - h.z); l.w = ptx::to_tf32(a.w - h.w);
                *reinterpret_cast<float4 *>(hi + off) = h;
                *reinterpret_cast<float4 *>(lo + off) = l;
            }
        }
    } else {
        __shared__ float tile[SPLIT_PIECE][SPLIT_PIECE + 1];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int e = threadIdx.x + 256 * i;                         // 64 x 64 scalars, row-contiguous reads
            const int r = e >> 6, c = e & 63;
            float v = 0.0f;
            if (pr + r < rows && pc + c < cols) {
                if (packed) {
                    const PackedRow row = packed_row(prop == MOM_LOWER_TRI, rows, pr + r);
                    if (pc + c >= row.first && pc + c < row.end) v = __ldcg(src + row.offset + (pc + c - row.first));
                } else {
                    v = __ldcg(src + (size_t)(pr + r) * cols + pc + c);
                }
            }
            if (sc.d && pr + r < rows && pc + c < cols) v *= __ldcg(sc.d + (sc.by_row ? pr + r : pc + c) * sc.step);
            tile[r][c] = v;
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = threadIdx.x + 256 * i;                         // 64 plane rows x 16 float4
            const int c = e >> 4, r = (e & 15) << 2;                     // plane entry (pc + c, pr + r .. +3)
            if (pc + c < cols && pr + r < rows) {
                float4 h, l;
                const float a0 = tile[r][c], a1 = tile[r + 1][c], a2 = tile[r + 2][c], a3 = tile[r + 3][c];
                h.x = ptx::to_tf32(a0); h.y = ptx::to_tf32(a1); h.z = ptx::to_tf32(a2); h.w = ptx::to_tf32(a3);
                l.x = ptx::to_tf32(a0 - h.x); l.y = ptx::to_tf32(a1 - h.y); l.z = ptx::to_tf32(a2 - h.z); l.w = ptx::to_tf32(a3 - h.w);
                const size_t off = (size_t)(pc + c) * rows + pr + r;
                *reinterpret_cast<float4 *>(hi + off) = h;
                *reinterpret_cast<float4 *>(lo + off) = l;
            }
        }
    }
}

template <bool TRANSPOSE>
__global__ void __launch_bounds__(256)
split_planes_kernel(const float *__restrict__ src, float *__restrict__ hi, float *__restrict__ lo, int rows, int cols, int prop,
                    SplitScale sc, int packed) {
    split_piece<TRANSPOSE>(src, hi, lo, rows, cols, prop, sc, blockIdx.x, blockIdx.y, packed);
}

// Both operands of one product in ONE launch (a launch costs about as much as splitting a few MB): the first
// pieces_a CTAs split the left operand, the others the right one.
struct SplitJob {
    const float *src;
    float *hi, *lo;
    int rows, cols, prop, transpose, pieces_x;
    SplitScale sc;
    int packed;
};
__global__ void __launch_bounds__(256)
split_both_kernel(SplitJob a, SplitJob b, int pieces_a) {
    const bool first = (int)blockIdx.x < pieces_a;
    const SplitJob &j = first ? a : b;
    const int piece = first ? blockIdx.x : blockIdx.x - pieces_a;
    const int px = piece % j.pieces_x, py = piece / j.pieces_x;
    if (j.transpose) split_piece<true>(j.src, j.hi, j.lo, j.rows, j.cols, j.prop, j.sc, px, py, j.packed);
    else split_piece<false>(j.src, j.hi, j.lo, j.rows, j.cols, j.prop, j.sc, px, py, j.packed);
}

// Split-K: sum the k-slices' partial results, then the usual finish (Add terms, structure mask).
// partial is (slices x slice_rows) x n; n is a multiple of 4.
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float *__restrict__ partial, int slices, int slice_rows, float *__restrict__ C, int m, int n,
                     int pout, AddTerms add) {
    const int vec_per_row = n >> 2;
    const long long total = (long long)m * vec_per_row;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(e / vec_per_row), c = (int)(e % vec_per_row) << 2;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < slices; ++s) {
            const float4 v = __ldcg(reinterpret_cast<const float4 *>(partial + ((size_t)s * slice_rows + r) * n + c));
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        float4 o;
        o.x = finish_entry(acc.x, add, 0, r, c, n, pout);
        o.y = finish_entry(acc.y, add, 0, r, c + 1, n, pout);
        o.z = finish_entry(acc.z, add, 0, r, c + 2, n, pout);
        o.w = finish_entry(acc.w, add, 0, r, c + 3, n, pout);
        *reinterpret_cast<float4 *>(C + (size_t)r * n + c) = o;
    }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

// 2-D f32 row-major matrix (rows x cols), box of box_rows x box_cols elements
bool tc_make_map(CUtensorMap *map, const void *ptr, int rows, int cols, int box_rows, int box_cols, CUtensorMapSwizzle swz) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(ptr), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {
inline bool make_map(CUtensorMap *map, const void *ptr, int rows, int cols, int box_rows, int box_cols, CUtensorMapSwizzle swz) {
    return tc_make_map(map, ptr, rows, cols, box_rows, box_cols, swz);
}

}  // namespace

mom_status_t tc_prepare(const mom_plan &p, TcPlanState &s) {
    if (s.ready) return MOM_OK;
    const int ns = (int)p.steps.size();
    s.steps.assign(ns, TcStepState{});
    std::vector<std::vector<int4>> tables(ns), part_tables[2] = {std::vector<std::vector<int4>>(ns), std::vector<std::vector<int4>>(ns)};
    size_t total = 0;
    int sms = 0;
    {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    for (int i = 0; i < ns; ++i) {
        const mom_step_t &st = p.steps[i].pub;
        if (st.uses_tensor_cores != 1) continue;
        const int m = (int)st.m, n = (int)st.n, k = (int)st.k;
        std::vector<int4> &tab = tables[i];
        // CTA pairs (256-row tiles) once there are enough of them to occupy most of the GPU's 74 pairs
        const long long pair_tiles = (long long)((m + P_BM - 1) / P_BM) * ((n + BN - 1) / BN);
        s.steps[i].pair = m >= P_BM && pair_tiles >= 48;
        const int split = p.steps[i].split_k;
        if (split > 1) s.steps[i].pair = false;
        const int tile_rows = s.steps[i].pair ? P_BM : BM;
        // a mirrored Gram product computes the tiles on and below the diagonal only (square 256 x 256 pair tiles)
        s.steps[i].mirror = p.steps[i].mirror && s.steps[i].pair;
        for (int r0 = 0; r0 < m; r0 += tile_rows)
            for (int c0 = 0; c0 < n; c0 += BN) {
                if (s.steps[i].mirror && c0 > r0) continue;
                int klo, khi;
                tile_k_range(kernel_property(st.lhs_property), kernel_property(st.rhs_property), r0, std::min(r0 + tile_rows, m), c0, std::min(c0 + BN, n), k, &klo, &khi);
                if (klo >= khi) { klo = 0; khi = 0; }
                klo = klo / BK * BK;                      // leading extra elements are stored zeros
                if (split <= 1) {
                    tab.push_back(make_int4(r0, c0, klo, khi));
                } else {
                    // every slice of every tile gets an entry (an empty one only zero-fills its slab), so the
                    // reduction may read all slabs
                    const int len = ((khi - klo + split - 1) / split + BK - 1) / BK * BK;
                    for (int i2 = 0; i2 < split; ++i2) {
                        const int lo = std::min(klo + i2 * len, khi), hi = std::min(lo + len, khi);
                        tab.push_back(make_int4(r0 | (i2 << TILE_SLICE_SHIFT), c0, lo < hi ? lo : 0, lo < hi ? hi : 0));
                    }
                }
            }
        // Order.  Tiles that run at the same time should share operand panels in L2: the output is cut into
        // bands of BAND tile rows, bands are visited heaviest first (triangular operands make them unequal),
        // and inside a band the tiles go column by column, every other band backwards.  A wave of CTAs
        // (or CTA pairs) then covers BAND rows x about units / BAND columns, a near-square block in bytes
        // of A and B panels, wherever the wave starts.  Structurally zero tiles come last.
        // Equal tiles are taken round-robin in that order.  Unequal tiles are dealt out by list scheduling on
        // the host: each tile, in that order, to the unit with the least work so far; the last few waves'
        // worth of tiles (all of them when there are only a few waves) are taken heaviest first so that the
        // units finish together.  Unit u then owns table
        // entries u, u + units, u + 2*units, ...; rounds a unit has no tile for hold a dummy entry that lies
        // outside the matrix (nothing loaded or stored).
        auto order = [&](std::vector<int4> &tab) -> int {    // orders `tab` in place, returns the units it was laid out for
            if (tab.empty()) return 1;
            bool uniform = true;
            for (const int4 &t : tab) uniform &= (t.w - t.z) == (tab[0].w - tab[0].z);
            const int units = std::max(1, std::min((int)tab.size(), s.steps[i].pair ? sms / 2 : sms));   // CTAs, or CTA pairs
            if (split <= 1) {
                const int band = s.steps[i].pair ? 8 : 16;                 // tile rows per band (2048 rows)
                const int n_bands = ((m + tile_rows - 1) / tile_rows + band - 1) / band;
                auto band_of = [&](const int4 &t) { return (t.x & TILE_ROW_MASK) / tile_rows / band; };
                std::vector<long long> band_work(n_bands, 0);
                for (const int4 &t : tab) band_work[band_of(t)] += t.w - t.z;
                std::vector<int> by_work(n_bands), rank(n_bands);
                for (int b2 = 0; b2 < n_bands; ++b2) by_work[b2] = b2;
                std::stable_sort(by_work.begin(), by_work.end(), [&](int x, int y) { return band_work[x] > band_work[y]; });
                for (int r2 = 0; r2 < n_bands; ++r2) rank[by_work[r2]] = r2;
                std::stable_sort(tab.begin(), tab.end(), [&](const int4 &x, const int4 &y) {
                    const bool zx = x.w <= x.z, zy = y.w <= y.z;
                    if (zx != zy) return zy;
                    const int rx = rank[band_of(x)], ry = rank[band_of(y)];
                    if (rx != ry) return rx < ry;
                    if (x.y != y.y) return (rx & 1) ? x.y > y.y : x.y < y.y;
                    return (x.x & TILE_ROW_MASK) < (y.x & TILE_ROW_MASK);
                });
            }
            if (!uniform) {
                if (split <= 1) {
                    size_t busy = 0;
                    while (busy < tab.size() && tab[busy].w > tab[busy].z) ++busy;
                    // with few waves of tiles the makespan matters more than locality: everything heaviest first
                    const size_t tail = busy <= (size_t)6 * units ? busy : (size_t)3 * units;
                    std::stable_sort(tab.begin() + (busy - tail), tab.begin() + busy,
                                     [](const int4 &x, const int4 &y) { return (x.w - x.z) > (y.w - y.z); });
                } else {
                    std::stable_sort(tab.begin(), tab.end(), [](const int4 &x, const int4 &y) { return (x.w - x.z) > (y.w - y.z); });
                }
                constexpr long long TILE_OVERHEAD = 3 * BK;         // epilogue and pipeline fill, in k units
                std::vector<std::vector<int4>> mine(units);
                std::vector<long long> load(units, 0);
                for (const int4 &t : tab) {
                    int best = 0;
                    for (int u = 1; u < units; ++u)
                        if (load[u] < load[best]) best = u;
                    mine[best].push_back(t);
                    load[best] += (t.w - t.z) + TILE_OVERHEAD;
                }
                size_t rounds = 0;
                for (const auto &v : mine) rounds = std::max(rounds, v.size());
                const int4 dummy = make_int4(TILE_ROW_MASK & ~(P_BM - 1), n + BN, 0, 0);
                tab.assign(rounds * units, dummy);
                for (int u = 0; u < units; ++u)
                    for (size_t r = 0; r < mine[u].size(); ++r) tab[r * units + u] = mine[u][r];
            }
            return units;
        };
        // the product that writes X, when it is large and plain: also as two row ranges (see TcStepState)
        const bool top_root = p.steps[i].is_last && !p.steps[i].accumulate && p.steps[i].sum + 1 == (int)p.sums.size();
        if (top_root && s.steps[i].pair && split <= 1 && !s.steps[i].mirror && m >= 2048) {
            const int row = std::max(P_BM, (int)(0.4 * m) / P_BM * P_BM);
            for (const int4 &t : tab) part_tables[(t.x & TILE_ROW_MASK) < row ? 0 : 1][i].push_back(t);
            s.steps[i].part_row = row;
            for (int q = 0; q < 2; ++q) {
                s.steps[i].part_units[q] = order(part_tables[q][i]);
                total += part_tables[q][i].size();
            }
        }
        // a product inside the plan whose left operand is a stored general matrix, read as stored and split here: two
        // row ranges as well, so that a caller who is still uploading that operand can start on its first half
        const int n_factors = (int)p.factor_ptr.size();
        const bool stored_lhs = st.lhs >= 0 && st.lhs < n_factors && p.factor_ptr[st.lhs] >= 0 && !st.lhs_transposed &&
                                st.lhs_property == MOM_GENERAL && !p.steps[i].a_planes_ready && p.steps[i].fold_a < 0;
        if (!p.steps[i].is_last && stored_lhs && s.steps[i].pair && split <= 1 && !s.steps[i].mirror && m >= 2048) {
            const int row = std::max(P_BM, (m / 2) / P_BM * P_BM);
            for (const int4 &t : tab) part_tables[(t.x & TILE_ROW_MASK) < row ? 0 : 1][i].push_back(t);
            s.steps[i].part_row = row;
            s.steps[i].split_a_by_part = true;
            for (int q = 0; q < 2; ++q) {
                s.steps[i].part_units[q] = order(part_tables[q][i]);
                total += part_tables[q][i].size();
            }
        }
        // Split-K with up to 8 slices per tile: the slices of a tile form a thread-block cluster and add their partial tiles through
        // distributed shared memory (no scratch, no reduction launch), provided all the clusters can run at once (a cluster sits in one
        // GPC and every CTA here takes a whole SM).  The table then stays in tile order, slice by slice: CTA i takes entry i.
        if (split > 1 && split <= 8 && (split & (split - 1)) == 0 && BM % split == 0 && (int)tab.size() <= sms) {
            int fit = 0;
            cudaLaunchConfig_t probe = {};
            probe.gridDim = dim3((unsigned)tab.size());
            probe.blockDim = dim3(THREADS);
            probe.dynamicSmemBytes = SMEM_BYTES;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = (unsigned)split; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            probe.attrs = at;
            probe.numAttrs = 1;
            if (raise_smem_limit_once(product_tc_kernel, SMEM_BYTES, &DeviceInfo::tc_attr) == cudaSuccess &&
                cudaOccupancyMaxActiveClusters(&fit, product_tc_kernel, &probe) == cudaSuccess && fit * split >= (int)tab.size())
                s.steps[i].cluster_split = split;
            else
                cudaGetLastError();
        }
        s.steps[i].units = s.steps[i].cluster_split > 1 ? (int)tab.size() : order(tab);
        total += tab.size();
    }
    if (total == 0) { s.ready = true; return MOM_OK; }
    if (cudaMalloc(&s.block, total * sizeof(int4)) != cudaSuccess) return MOM_ERR_ALLOC;
    int4 *cur = static_cast<int4 *>(s.block);
    for (int i = 0; i < ns; ++i) {
        if (tables[i].empty()) continue;
        if (cudaMemcpy(cur, tables[i].data(), tables[i].size() * sizeof(int4), cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaFree(s.block);
            s.block = nullptr;
            return MOM_ERR_CUDA;
        }
        s.steps[i].tiles = cur;
        s.steps[i].num_tiles = (int)tables[i].size();
        cur += tables[i].size();
        for (int q = 0; q < 2; ++q) {
            const std::vector<int4> &pt = part_tables[q][i];
            if (pt.empty()) continue;
            if (cudaMemcpy(cur, pt.data(), pt.size() * sizeof(int4), cudaMemcpyHostToDevice) != cudaSuccess) {
                cudaFree(s.block);
                s.block = nullptr;
                return MOM_ERR_CUDA;
            }
            s.steps[i].part_tiles[q] = cur;
            s.steps[i].part_num[q] = (int)pt.size();
            cur += pt.size();
        }
    }
    s.ready = true;
    return MOM_OK;
}

void tc_release(TcPlanState &s) {
    if (s.block) cudaFree(s.block);
    s.block = nullptr;
    s.steps.clear();
    s.ready = false;
}

mom_status_t tc_launch_step(const mom_plan &p, TcPlanState &s, int step, const ProductArgs &a, char *workspace,
                            int32_t *status, cudaStream_t stream, int *launches, cudaEvent_t before_product, int part) {
    const StepImpl &st = p.steps[step];
    if (!s.ready || step >= (int)s.steps.size() || !s.steps[step].tiles) return MOM_ERR_INVALID_ARG;
    if (part < 0 || part > 2 || (part > 0 && (s.steps[step].part_row == 0 || !s.steps[step].part_tiles[part - 1]))) return MOM_ERR_INVALID_ARG;
    const int4 *tiles = part ? s.steps[step].part_tiles[part - 1] : s.steps[step].tiles;
    const int num_tiles = part ? s.steps[step].part_num[part - 1] : s.steps[step].num_tiles;
    const int units = part ? s.steps[step].part_units[part - 1] : s.steps[step].units;
    const int sm_count = current_sm_count();
    if (sm_count < 1) return MOM_ERR_CUDA;
    if (raise_smem_limit_once(product_tc_kernel, SMEM_BYTES, &DeviceInfo::tc_attr) != cudaSuccess) return MOM_ERR_CUDA;
    float *a_hi = reinterpret_cast<float *>(workspace + st.a_hi_off), *a_lo = reinterpret_cast<float *>(workspace + st.a_lo_off);
    float *b_hi = reinterpret_cast<float *>(workspace + st.b_hi_off), *b_lo = reinterpret_cast<float *>(workspace + st.b_lo_off);

    // operand planes: written by the producing step's epilogue, or split here from the f32 operand
    auto blocks = [](int x) { return (x + SPLIT_PIECE - 1) / SPLIT_PIECE; };
    int split_launches = 0;
    // The MMA wants A as m x k and B as n x k (both K-major).  An operand stored the other way round
    // (a transposed chain operand) only swaps which of the two split kernels reads it; the structure
    // argument is the one of the matrix as stored (the transpose of a lower triangle is an upper one).
    auto stored_prop = [](int prop_as_used) {
        return prop_as_used == MOM_LOWER_TRI ? (int)MOM_UPPER_TRI : prop_as_used == MOM_UPPER_TRI ? (int)MOM_LOWER_TRI : prop_as_used;
    };
    // a folded scaling: rows of the operand as used <-> rows of the matrix as stored unless it is stored transposed
    const SplitScale sa{a.scaleA, a.scaleA_step, a.scaleA ? (a.scaleA_rows != 0) != (a.transA != 0) : 0};
    const SplitScale sb{a.scaleB, a.scaleB_step, a.scaleB ? (a.scaleB_rows != 0) != (a.transB != 0) : 0};
    // as stored: rows x cols and the property of the matrix the kernel reads
    SplitJob ja{a.A, a_hi, a_lo, a.transA ? a.k : a.m, a.transA ? a.m : a.k, a.transA ? stored_prop(a.pa) : a.pa, a.transA ? 1 : 0,
                blocks(a.transA ? a.m : a.k), sa, a.packedA};
    const bool a_by_part = part > 0 && s.steps[step].split_a_by_part;     // a general m x k matrix read as stored
    if (a_by_part) {
        const int row = s.steps[step].part_row, r0 = part == 1 ? 0 : row;
        ja.src += (size_t)r0 * a.k;
        ja.hi += (size_t)r0 * a.k;
        ja.lo += (size_t)r0 * a.k;
        ja.rows = part == 1 ? row : a.m - row;
    }
    const SplitJob jb{a.B, b_hi, b_lo, a.transB ? a.n : a.k, a.transB ? a.k : a.n, a.transB ? stored_prop(a.pb) : a.pb, a.transB ? 0 : 1,
                      blocks(a.transB ? a.k : a.n), sb, a.packedB};
    const bool do_a = !st.a_planes_ready && (part != 2 || a_by_part), do_b = !st.b_planes_ready && part != 2;
    auto pieces = [&](const SplitJob &j) { return j.pieces_x * blocks(j.rows); };
    if (do_a && do_b) {
        split_both_kernel<<<pieces(ja) + pieces(jb), 256, 0, stream>>>(ja, jb, pieces(ja));
        ++split_launches;
    } else if (do_a || do_b) {
        const SplitJob &j = do_a ? ja : jb;
        if (j.transpose) split_planes_kernel<true><<<dim3(j.pieces_x, blocks(j.rows)), 256, 0, stream>>>(j.src, j.hi, j.lo, j.rows, j.cols, j.prop, j.sc, j.packed);
        else split_planes_kernel<false><<<dim3(j.pieces_x, blocks(j.rows)), 256, 0, stream>>>(j.src, j.hi, j.lo, j.rows, j.cols, j.prop, j.sc, j.packed);
        ++split_launches;
    }
    if (cudaGetLastError() != cudaSuccess) return MOM_ERR_CUDA;
    if (before_product) cudaEventRecord(before_product, stream);

    // A planes are m x k, B planes are n x k (transposed): both K-major with 32-element (128-byte) box rows.
    // Output: the f32 matrix, or the consumer's planes (m x n as stored, or n x m transposed).
    CUtensorMap ma_hi, ma_lo, mb_hi, mb_lo, mc, mc2;
    bool ok = make_map(&ma_hi, a_hi, a.m, a.k, BM, BK, OPERAND_TMA_SWIZZLE) &&
              make_map(&ma_lo, a_lo, a.m, a.k, BM, BK, OPERAND_TMA_SWIZZLE) &&
              make_map(&mb_hi, b_hi, a.n, a.k, s.steps[step].pair ? BN / 2 : BN, BK, OPERAND_TMA_SWIZZLE) &&
              make_map(&mb_lo, b_lo, a.n, a.k, s.steps[step].pair ? BN / 2 : BN, BK, OPERAND_TMA_SWIZZLE);
    const int slice_rows = st.split_k > 1 ? (a.m + BM - 1) / BM * BM : 0;
    float *partial = st.split_k > 1 ? reinterpret_cast<float *>(workspace + st.partial_off) : nullptr;
    if (st.split_k > 1) {
        ok = ok && make_map(&mc, partial, st.split_k * slice_rows, a.n, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
        mc2 = mc;
    } else if (st.planes_out == 0) {
        ok = ok && make_map(&mc, a.C, a.m, a.n, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
        mc2 = mc;
    } else {
        float *p_hi = reinterpret_cast<float *>(workspace + st.planes_hi_off), *p_lo = reinterpret_cast<float *>(workspace + st.planes_lo_off);
        const int rows = st.planes_out == 1 ? a.m : a.n, cols = st.planes_out == 1 ? a.n : a.m;
        ok = ok && make_map(&mc, p_hi, rows, cols, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B) &&
             make_map(&mc2, p_lo, rows, cols, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    }
    if (!ok) return MOM_ERR_CUDA;

    TcParams prm;
    prm.tiles = tiles;
    prm.num_tiles = num_tiles;
    prm.m = a.m;
    prm.n = a.n;
    const bool separate_reduction = st.split_k > 1 && !(part == 0 && s.steps[step].cluster_split > 1);
    prm.pout = separate_reduction ? (int)MOM_GENERAL : a.pout;   // split-K with a reduction launch: it applies mask and Add terms
    prm.out_mode = st.planes_out;
    prm.slice_rows = slice_rows;
    const int cluster_split = part == 0 ? s.steps[step].cluster_split : 0;
    prm.cluster_split = cluster_split;
    prm.c_out = a.C;
    if (s.steps[step].mirror && st.planes_out != 0) return MOM_ERR_INVALID_ARG;   // the planner never asks for this
    prm.mirror = s.steps[step].mirror ? 1 : 0;
    prm.packed_c = nullptr;
    if (a.packedC) {
        // only a plain f32 result of a triangular product is ever written packed (the planner checks as much)
        if (st.planes_out != 0 || st.split_k > 1 || s.steps[step].mirror || (a.pout != MOM_LOWER_TRI && a.pout != MOM_UPPER_TRI)) return MOM_ERR_INVALID_ARG;
        prm.packed_c = a.C;
    }
    prm.add = a.add;
    if (separate_reduction) prm.add.count = 0;
    prm.status = status;
    if (s.steps[step].pair) {
        if (raise_smem_limit_once(product_tc_pair_kernel, P_SMEM_BYTES, &DeviceInfo::pair_attr) != cudaSuccess) return MOM_ERR_CUDA;
        cudaLaunchConfig_t cfg;
        std::memset(&cfg, 0, sizeof(cfg));
        cfg.gridDim = dim3(sm_count / 2 * 2);
        cfg.blockDim = dim3(THREADS);
        cfg.dynamicSmemBytes = P_SMEM_BYTES;
        cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        // A persistent grid must not exceed what is co-resident: not every SM can host half of a CTA pair
        // (the pair must sit on one TPC), so ask how many clusters fit instead of assuming SMs / 2.
        int max_pairs = 0;
        {
            std::lock_guard<std::mutex> lock(device_info_mutex());
            DeviceInfo *info = current_device_info();
            if (!info) return MOM_ERR_CUDA;
            if (!info->max_pairs) {
                int n = 0;
                if (cudaOccupancyMaxActiveClusters(&n, product_tc_pair_kernel, &cfg) != cudaSuccess || n < 1) return MOM_ERR_CUDA;
                info->max_pairs = n;
            }
            max_pairs = info->max_pairs;
        }
        if (max_pairs < units) return MOM_ERR_CUDA;   // the table was laid out for co-resident pairs
        cfg.gridDim = dim3(2 * units);
        if (cudaLaunchKernelEx(&cfg, product_tc_pair_kernel, ma_hi, ma_lo, mb_hi, mb_lo, mc, mc2, prm) != cudaSuccess) return MOM_ERR_CUDA;
    } else {
        const int grid = std::min(units, sm_count);
        if (cluster_split > 1) {
            if (grid != units || grid % cluster_split != 0) return MOM_ERR_CUDA;      // one table entry per CTA, whole clusters
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(grid);
            cfg.blockDim = dim3(THREADS);
            cfg.dynamicSmemBytes = SMEM_BYTES;
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)cluster_split;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            if (cudaLaunchKernelEx(&cfg, product_tc_kernel, ma_hi, ma_lo, mb_hi, mb_lo, mc, mc2, prm) != cudaSuccess) return MOM_ERR_CUDA;
        } else {
            product_tc_kernel<<<grid, THREADS, SMEM_BYTES, stream>>>(ma_hi, ma_lo, mb_hi, mb_lo, mc, mc2, prm);
        }
    }
    if (cudaGetLastError() != cudaSuccess) return MOM_ERR_CUDA;
    *launches = 1 + split_launches;
    if (separate_reduction) {
        const long long vecs = (long long)a.m * (a.n / 4);
        const int blocks_r = (int)std::min<long long>((vecs + 255) / 256, (long long)sm_count * 8);
        splitk_reduce_kernel<<<blocks_r, 256, 0, stream>>>(partial, st.split_k, slice_rows, a.C, a.m, a.n, a.pout, a.add);
        if (cudaGetLastError() != cudaSuccess) return MOM_ERR_CUDA;
        ++*launches;
    }
    return MOM_OK;
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded wait: one thread waits, with the product kernels' own wait_barrier, on an mbarrier
// that nothing ever arrives on.  The wait gives up after `limit_ns`, records MOM_ERR_DEVICE_TIMEOUT and
// `detail` in the status block exactly as a product kernel would, and the kernel returns by itself.
// ---------------------------------------------------------------------------------------------
namespace {
__global__ void __launch_bounds__(32, 1) wait_timeout_kernel(int32_t *status, unsigned long long limit_ns, int detail) {
    __shared__ __align__(8) unsigned long long barrier_word;
    __shared__ int abort_word;
    if (threadIdx.x == 0) {
        abort_word = 0;
        const uint32_t bar = ptx::smem_u32(&barrier_word);
        ptx::mbar_init(bar, 1);
        ptx::fence_barrier_init();
        wait_barrier(bar, 0, &abort_word, status, detail, limit_ns);
    }
}
}  // namespace

cudaError_t launch_wait_timeout_probe(int32_t *status, unsigned long long limit_ns, int detail, cudaStream_t stream) {
    wait_timeout_kernel<<<1, 32, 0, stream>>>(status, limit_ns, detail);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// TF32 rate probe: every SM issues M128 N256 K8 kind::tf32 MMAs on resident shared-memory tiles.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int PROBE_BATCH = 64;                 // MMAs between commits
constexpr int PROBE_SMEM = 1024 + 8192 + 16384 + 64;

__global__ void __launch_bounds__(128, 1) tf32_probe_kernel(int batches, int32_t *status) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ int abort_word;
    const uint32_t base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_tile = base, b_tile = base + 8192, bar0 = base + 8192 + 16384, bar1 = bar0 + 8, slot = bar0 + 16;
    // finite, tf32-representable operand values
    for (int i = threadIdx.x; i < (8192 + 16384) / 4; i += blockDim.x) {
        const float v = (float)((i * 37 + blockIdx.x) % 61 - 30) * 0.03125f;
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(base + 4 * i), "f"(v) : "memory");
    }
    if (threadIdx.x == 0) {
        abort_word = 0;
        ptx::mbar_init(bar0, 1);
        ptx::mbar_init(bar1, 1);
        ptx::fence_barrier_init();
    }
    ptx::fence_proxy_async_smem();
    if (threadIdx.x < 32) {
        ptx::tmem_alloc(slot, 256);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    uint32_t tmem_base;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tmem_base) : "r"(slot));
    if (threadIdx.x == 0) {
        constexpr uint32_t idesc = ptx::instr_desc_tf32(128, 256, 0, 0);
        const uint64_t da = kmajor_desc_64(a_tile), db = kmajor_desc_64(b_tile);
        bool ok = true;
        for (int b = 0; b < batches && ok; ++b) {
            for (int i = 0; i < PROBE_BATCH; ++i) ptx::mma_tf32(tmem_base, da, db, idesc, (b | i) ? 1u : 0u);
            ptx::mma_commit((b & 1) ? bar1 : bar0);
            if (b >= 1) ok = wait_barrier(((b - 1) & 1) ? bar1 : bar0, ((b - 1) >> 1) & 1, &abort_word, status, (5 << 24) | (b & 0xFFFF));
        }
        if (ok && batches > 0) wait_barrier(((batches - 1) & 1) ? bar1 : bar0, ((batches - 1) >> 1) & 1, &abort_word, status, (6 << 24));
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    if (threadIdx.x < 32) ptx::tmem_dealloc(tmem_base, 256);
}

}  // namespace

mom_status_t tc_probe_tf32(double milliseconds, void *scratch, cudaStream_t stream, double *tflops) {
    int dev = 0, sms = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MOM_ERR_CUDA;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (major != 10) return MOM_ERR_ARCH;
    if (cudaFuncSetAttribute(tf32_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PROBE_SMEM) != cudaSuccess) return MOM_ERR_CUDA;
    int32_t *status = static_cast<int32_t *>(scratch);
    if (cudaMemsetAsync(status, 0, 16, stream) != cudaSuccess) return MOM_ERR_CUDA;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return MOM_ERR_CUDA;
    auto run = [&](int batches, float *ms) -> bool {
        cudaEventRecord(e0, stream);
        tf32_probe_kernel<<<sms, 128, PROBE_SMEM, stream>>>(batches, status);
        cudaEventRecord(e1, stream);
        return cudaEventSynchronize(e1) == cudaSuccess && cudaGetLastError() == cudaSuccess &&
               cudaEventElapsedTime(ms, e0, e1) == cudaSuccess;
    };
    float ms = 0.0f;
    int batches = 256;
    bool ok = run(batches, &ms) && run(batches, &ms);
    if (ok) {
        double scale = milliseconds / (ms > 1e-3f ? ms : 1e-3f);
        if (scale > 1.0) batches = (int)(batches * (scale < 50000.0 ? scale : 50000.0));
        ok = run(batches, &ms);
    }
    int32_t host[2] = {0, 0};
    if (ok) ok = cudaMemcpy(host, status, sizeof(host), cudaMemcpyDeviceToHost) == cudaSuccess;
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (!ok) return MOM_ERR_CUDA;
    if (host[0] != 0) return MOM_ERR_DEVICE_TIMEOUT;
    *tflops = (double)sms * batches * PROBE_BATCH * 2.0 * 128 * 256 * 8 / (ms * 1e-3) * 1e-12;
    return MOM_OK;
}

}  // namespace mom

// ---------------------------------------------------------------------------------------------
// Allocation-free single product (mom_product_3xtf32_noalloc).  The hi/lo planes, the tile table
// and a status word live in one fixed array that is part of the loaded module, so the call needs
// neither a caller workspace nor any allocation.
// ---------------------------------------------------------------------------------------------
namespace mom {
namespace {

constexpr size_t NOALLOC_PLANES_BYTES = (size_t)16 << 20;            // A_hi, A_lo, Bt_hi, Bt_lo together
constexpr int NOALLOC_MAX_TILES = 2048;
constexpr size_t NOALLOC_TABLE_OFFSET = NOALLOC_PLANES_BYTES;
constexpr size_t NOALLOC_STATUS_OFFSET = NOALLOC_TABLE_OFFSET + (size_t)NOALLOC_MAX_TILES * sizeof(int4);
constexpr size_t NOALLOC_TOTAL_BYTES = NOALLOC_STATUS_OFFSET + 256;
constexpr int NOALLOC_MAX_DEVICES = 64;

// Held by every GPU that loads the library until the process exits.  In host code this name is only a
// handle for cudaGetSymbolAddress; the device address is looked up once per device below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_TOTAL_BYTES];

unsigned char *g_noalloc_device_ptr[NOALLOC_MAX_DEVICES] = {};

// one thread per output tile, row-major tile order
__global__ void noalloc_build_tiles_kernel(int4 *tiles, int m, int n, int k, int pa, int pb) {
    const int cols = (n + BN - 1) / BN, total = ((m + BM - 1) / BM) * cols;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= total) return;
    const int r0 = (t / cols) * BM, c0 = (t % cols) * BN;
    int klo, khi;
    tile_k_range(pa, pb, r0, min(r0 + BM, m), c0, min(c0 + BN, n), k, &klo, &khi);
    if (klo >= khi) { klo = 0; khi = 0; }
    tiles[t] = make_int4(r0, c0, klo / BK * BK, khi);
}

}  // namespace
}  // namespace mom

extern "C" mom_status_t mom_product_3xtf32_noalloc(int64_t m64, int64_t n64, int64_t k64, mom_property_t pa,
                                                   mom_property_t pb, const float *A, const float *B, float *C,
                                                   int32_t *device_status, mom_stream_t stream_) {
    using namespace mom;
    if (!A || !B || !C || m64 < 1 || n64 < 1 || k64 < 1) return MOM_ERR_INVALID_ARG;
    if (pa < MOM_GENERAL || pa > MOM_UPPER_TRI || pb < MOM_GENERAL || pb > MOM_UPPER_TRI) return MOM_ERR_INVALID_ARG;
    if ((pa != MOM_GENERAL && m64 != k64) || (pb != MOM_GENERAL && k64 != n64)) return MOM_ERR_PROPERTY;
    if (k64 % 4 != 0 || n64 % 4 != 0) return MOM_ERR_INVALID_ARG;      // leading dimensions TMA can address
    if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(C)) & 15) return MOM_ERR_ALIGNMENT;
    if (m64 > (1 << 20) || n64 > (1 << 20) || k64 > (1 << 20)) return MOM_ERR_LIMIT;
    const int m = (int)m64, n = (int)n64, k = (int)k64;
    const size_t a_bytes = align_up((size_t)m * k * sizeof(float), WS_ALIGN);
    const size_t b_bytes = align_up((size_t)k * n * sizeof(float), WS_ALIGN);
    const long long tiles = (long long)((m + BM - 1) / BM) * ((n + BN - 1) / BN);
    if (2 * a_bytes + 2 * b_bytes > NOALLOC_PLANES_BYTES || tiles > NOALLOC_MAX_TILES) return MOM_ERR_LIMIT;

    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MOM_ERR_CUDA;
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return MOM_ERR_LIMIT;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return MOM_ERR_CUDA;
    if (major != 10) return MOM_ERR_ARCH;
    if (!g_noalloc_device_ptr[dev]) {          // once per device, with that device current
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return MOM_ERR_CUDA;
        g_noalloc_device_ptr[dev] = static_cast<unsigned char *>(p);
    }
    const int sm_count = current_sm_count();
    if (sm_count < 1) return MOM_ERR_CUDA;
    if (raise_smem_limit_once(product_tc_kernel, SMEM_BYTES, &DeviceInfo::tc_attr) != cudaSuccess) return MOM_ERR_CUDA;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    unsigned char *base = g_noalloc_device_ptr[dev];
    float *a_hi = reinterpret_cast<float *>(base), *a_lo = reinterpret_cast<float *>(base + a_bytes);
    float *b_hi = reinterpret_cast<float *>(base + 2 * a_bytes), *b_lo = reinterpret_cast<float *>(base + 2 * a_bytes + b_bytes);
    int4 *table = reinterpret_cast<int4 *>(base + NOALLOC_TABLE_OFFSET);
    int32_t *status = device_status ? device_status : reinterpret_cast<int32_t *>(base + NOALLOC_STATUS_OFFSET);
    // the array keeps whatever the previous call left: the status word must start at zero, the tile
    // table and every plane block a tile can read are rewritten below
    if (!device_status && cudaMemsetAsync(status, 0, 4 * sizeof(int32_t), stream) != cudaSuccess) return MOM_ERR_CUDA;

    auto blocks = [](int x) { return (x + SPLIT_PIECE - 1) / SPLIT_PIECE; };
    noalloc_build_tiles_kernel<<<(unsigned)((tiles + 127) / 128), 128, 0, stream>>>(table, m, n, k, (int)pa, (int)pb);
    split_planes_kernel<false><<<dim3(blocks(k), blocks(m)), 256, 0, stream>>>(A, a_hi, a_lo, m, k, (int)pa, SplitScale{nullptr, 0, 0}, 0);
    split_planes_kernel<true><<<dim3(blocks(n), blocks(k)), 256, 0, stream>>>(B, b_hi, b_lo, k, n, (int)pb, SplitScale{nullptr, 0, 0}, 0);
    if (cudaGetLastError() != cudaSuccess) return MOM_ERR_CUDA;

    CUtensorMap ma_hi, ma_lo, mb_hi, mb_lo, mc;
    const bool ok = make_map(&ma_hi, a_hi, m, k, BM, BK, OPERAND_TMA_SWIZZLE) &&
                    make_map(&ma_lo, a_lo, m, k, BM, BK, OPERAND_TMA_SWIZZLE) &&
                    make_map(&mb_hi, b_hi, n, k, BN, BK, OPERAND_TMA_SWIZZLE) &&
                    make_map(&mb_lo, b_lo, n, k, BN, BK, OPERAND_TMA_SWIZZLE) &&
                    make_map(&mc, C, m, n, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    if (!ok) return MOM_ERR_CUDA;
    TcParams prm;
    prm.tiles = table;
    prm.num_tiles = (int)tiles;
    prm.m = m;
    prm.n = n;
    prm.pout = pa == MOM_GENERAL || pb == MOM_GENERAL || pa != pb ? (int)MOM_GENERAL : (int)pa;
    prm.out_mode = 0;
    prm.slice_rows = 0;
    prm.cluster_split = 0;
    prm.c_out = nullptr;
    prm.mirror = 0;
    prm.packed_c = nullptr;
    prm.add.count = 0;
    prm.status = status;
    product_tc_kernel<<<std::min(prm.num_tiles, sm_count), THREADS, SMEM_BYTES, stream>>>(ma_hi, ma_lo, mb_hi, mb_lo, mc, mc, prm);
    return cudaGetLastError() == cudaSuccess ? MOM_OK : MOM_ERR_CUDA;
}
