// Warp-level tensor-core product kernel: C = A*B (+ Add terms) with mma.sync m16n8k8 tf32 and the 3xTF32
// split done in registers, for products that are too small to pay for the tcgen05 path (its operand-split
// passes, tile tables and, with few output tiles, a split-K reduction pass cost three or four launches of
// 5-14 us each).  This kernel is ONE launch per product: it reads the f32 operands as stored, and when
// the output has few tiles it splits the contraction over the CTAs of a thread-block cluster, which add
// their partial tiles up through distributed shared memory in a fixed order (deterministic, no atomics,
// no scratch in global memory).  Structure is handled as everywhere else: the tile's structural k-range
// (tile_k_range) bounds the contraction, the epilogue adds the terms and masks the result.
#include <cooperative_groups.h>

#include "device_common.cuh"
#include "device_info.h"
#include "kernels.h"

namespace mom {

namespace {

namespace cg = cooperative_groups;

constexpr int BM = 64, BN = 32, BK = 32, THREADS = 256, STAGES = 3;
// leading dimensions that keep the fragment loads free of bank conflicts: thread (g, t) of a warp reads
// A[g][t] (rows 4 mod 8 words apart) and B[t][g] (rows 8 mod 16 words apart)
constexpr int LDA = BK + 4, LDB = BN + 8, LDP = BN + 4;
constexpr int A_STAGE = BM * LDA, B_STAGE = BK * LDB;        // floats per pipeline stage
constexpr int MAX_SPLIT = 16;                                // 8 is the portable cluster size; 16 where the device takes it

static_assert(BM * LDP <= STAGES * A_STAGE, "the partial tile reuses the A stages");

__device__ __forceinline__ void cp_async16(float *dst, const float *src, bool valid) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(valid ? 16 : 0) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// a = hi + lo: hi is a rounded to tf32 on the bit pattern (ties away from zero), lo = a - hi is exact in
// f32 and handed over as it is (the MMA reads only the tf32 part of a register: what it drops is at most
// 2^-21 of a, the size of the lo*lo term the scheme leaves out anyway)
__device__ __forceinline__ void split_tf32(float a, uint32_t &hi, uint32_t &lo) {
    hi = (__float_as_uint(a) + 0x1000u) & 0xFFFFE000u;
    lo = __float_as_uint(a - __uint_as_float(hi));
}

__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

__global__ void __launch_bounds__(THREADS)
product_mma_kernel(const ProductArgs a, const int split, const int tiles_n) {
    __shared__ __align__(16) float As[STAGES * A_STAGE];
    __shared__ __align__(16) float Bs[STAGES * B_STAGE];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int wm = warp >> 1, wn = warp & 1;                 // 4 x 2 warps, 16 x 16 outputs each
    const long long inst = blockIdx.z;
    const int rank = split > 1 ? (int)(blockIdx.x % split) : 0;      // position in the cluster = k-slice
    const int tile = blockIdx.x / split;
    const int m = a.m, n = a.n, k = a.k;
    const int r0 = (tile / tiles_n) * BM, c0 = (tile % tiles_n) * BN;
    const float *__restrict__ A = a.A + inst * a.strideA;
    const float *__restrict__ B = a.B + inst * a.strideB;
    float *__restrict__ C = a.C + inst * a.strideC;

    int klo, khi;
    tile_k_range(a.pa, a.pb, r0, min(r0 + BM, m), c0, min(c0 + BN, n), k, &klo, &khi);
    klo &= ~(BK - 1);                                        // extra leading elements are stored zeros
    const int blocks = klo < khi ? (khi - klo + BK - 1) / BK : 0;
    const int per = (blocks + split - 1) / split;
    const int kb0 = min(rank * per, blocks), nk = min(kb0 + per, blocks) - kb0;

    const bool a_fast = !a.transA && (k & 3) == 0 && (reinterpret_cast<uintptr_t>(A) & 15) == 0;
    const bool b_fast = !a.transB && (n & 3) == 0 && (reinterpret_cast<uintptr_t>(B) & 15) == 0;

    // global -> shared: the A tile is 64 rows x 8 quads (two per thread), the B tile 32 k-rows x 8 quads
    auto load_stage = [&](int stage, int k0) {
        float *as = As + stage * A_STAGE, *bs = Bs + stage * B_STAGE;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int q = tid + THREADS * i, row = q >> 3, kq = (q & 7) << 2;
            const int r = r0 + row, kk = k0 + kq;
            float *dst = as + row * LDA + kq;
            if (a_fast) {
                const bool ok = r < m && kk < k;
                cp_async16(dst, ok ? A + (long long)r * k + kk : A, ok);
            } else {
                float v[4] = {0.f, 0.f, 0.f, 0.f};
                if (r < m) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (kk + j < k) v[j] = __ldg(a.transA ? A + (long long)(kk + j) * m + r : A + (long long)r * k + kk + j);
                }
                *reinterpret_cast<float4 *>(dst) = make_float4(v[0], v[1], v[2], v[3]);
            }
        }
        const int krow = tid >> 3, cq = (tid & 7) << 2;
        const int kk = k0 + krow, c = c0 + cq;
        float *dst = bs + krow * LDB + cq;
        if (b_fast) {
            const bool ok = kk < k && c < n;
            cp_async16(dst, ok ? B + (long long)kk * n + c : B, ok);
        } else {
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (kk < k) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (c + j < n) v[j] = __ldg(a.transB ? B + (long long)(c + j) * k + kk : B + (long long)kk * n + c + j);
            }
            *reinterpret_cast<float4 *>(dst) = make_float4(v[0], v[1], v[2], v[3]);
        }
    };

    // the small terms (lo*hi, hi*lo) and the main term (hi*hi) go to separate accumulators
    float main_acc[2][4], small_acc[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int q = 0; q < 4; ++q) main_acc[j][q] = small_acc[j][q] = 0.f;

    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < nk) load_stage(s, klo + (kb0 + s) * BK);
        cp_async_commit();
    }
    for (int i = 0; i < nk; ++i) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();                                     // block i has landed; everybody is done with block i - 1
        if (i + STAGES - 1 < nk) load_stage((i + STAGES - 1) % STAGES, klo + (kb0 + i + STAGES - 1) * BK);
        cp_async_commit();
        const float *as = As + (i % STAGES) * A_STAGE + (wm * 16 + g) * LDA + t;
        const float *bs = Bs + (i % STAGES) * B_STAGE + t * LDB + wn * 16 + g;
#pragma unroll
        for (int kk = 0; kk < BK; kk += 8) {
            uint32_t a_hi[4], a_lo[4];
            split_tf32(as[kk], a_hi[0], a_lo[0]);
            split_tf32(as[8 * LDA + kk], a_hi[1], a_lo[1]);
            split_tf32(as[kk + 4], a_hi[2], a_lo[2]);
            split_tf32(as[8 * LDA + kk + 4], a_hi[3], a_lo[3]);
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                uint32_t b_hi[2], b_lo[2];
                split_tf32(bs[kk * LDB + 8 * j], b_hi[0], b_lo[0]);
                split_tf32(bs[(kk + 4) * LDB + 8 * j], b_hi[1], b_lo[1]);
                mma_tf32(small_acc[j], a_lo, b_hi);
                mma_tf32(main_acc[j], a_hi, b_hi);
                mma_tf32(small_acc[j], a_hi, b_lo);
            }
        }
    }
    cp_async_wait<0>();

    if (split == 1) {
        // fused epilogue straight from the accumulators: entries (row, col) and (row, col + 1) per pair
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = r0 + wm * 16 + g + 8 * h, c = c0 + wn * 16 + 8 * j + 2 * t;
                if (r >= m || c >= n) continue;
                const float v0 = finish_entry_compact(main_acc[j][2 * h] + small_acc[j][2 * h], a.add, inst, r, c, n, a.pout);
                float *p = C + (long long)r * n + c;
                if (c + 1 < n) {
                    const float v1 = finish_entry_compact(main_acc[j][2 * h + 1] + small_acc[j][2 * h + 1], a.add, inst, r, c + 1, n, a.pout);
                    if ((reinterpret_cast<uintptr_t>(p) & 7) == 0) *reinterpret_cast<float2 *>(p) = make_float2(v0, v1);
                    else { p[0] = v0; p[1] = v1; }
                } else {
                    p[0] = v0;
                }
            }
        return;
    }

    // Split contraction: every CTA of the cluster leaves its partial tile in its own shared memory, then
    // CTA `rank` finishes rows [rank * BM / split, (rank + 1) * BM / split) of the tile, adding the partial
    // tiles in the order of the k-slices.
    cg::cluster_group cluster = cg::this_cluster();
    __syncthreads();                                         // the pipeline's stages are free
    float *P = As;
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float *p = P + (wm * 16 + g + 8 * h) * LDP + wn * 16 + 8 * j + 2 * t;
            p[0] = main_acc[j][2 * h] + small_acc[j][2 * h];
            p[1] = main_acc[j][2 * h + 1] + small_acc[j][2 * h + 1];
        }
    cluster.sync();
    const int rows_per = BM / split;
    for (int e = tid; e < rows_per * BN; e += THREADS) {
        const int row = rank * rows_per + e / BN, col = e % BN;
        const int r = r0 + row, c = c0 + col;
        if (r >= m || c >= n) continue;
        float sum = 0.f;
        for (int q = 0; q < split; ++q) sum += cluster.map_shared_rank(P, q)[row * LDP + col];
        C[(long long)r * n + c] = finish_entry_compact(sum, a.add, inst, r, c, n, a.pout);
    }
    cluster.sync();                                          // nobody leaves while a peer may still read its tile
}

}  // namespace

cudaError_t launch_product_mma(const ProductArgs &a, int batch, cudaStream_t stream) {
    const int sm_count = current_sm_count();
    if (sm_count < 1) return cudaErrorInvalidDevice;
    const int tiles_n = (a.n + BN - 1) / BN;
    const long long tiles = (long long)((a.m + BM - 1) / BM) * tiles_n;
    // few tiles and a long contraction: split k over a cluster, as long as every slice keeps a few k-blocks
    // (the longest structural k-range of a tile is at most k)
    int split = 1;
    const long long resident = 4LL * sm_count;
    while (split < MAX_SPLIT && tiles * batch * split * 2 <= resident && a.k / (split * 2) >= 4 * BK) split *= 2;
    if (split == 16) {
        // a cluster of 16 needs the non-portable size allowed on this kernel, and room for all clusters at once
        std::lock_guard<std::mutex> lock(device_info_mutex());
        DeviceInfo *info = current_device_info();
        if (!info) return cudaErrorInvalidDevice;
        if (info->mma_clusters16 == 0) {
            info->mma_clusters16 = -1;
            if (cudaFuncSetAttribute(product_mma_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
                cudaLaunchConfig_t probe = {};
                probe.gridDim = dim3((unsigned)(16 * sm_count));
                probe.blockDim = dim3(THREADS);
                cudaLaunchAttribute at[1];
                at[0].id = cudaLaunchAttributeClusterDimension;
                at[0].val.clusterDim.x = 16; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
                probe.attrs = at;
                probe.numAttrs = 1;
                int n = 0;
                if (cudaOccupancyMaxActiveClusters(&n, product_mma_kernel, &probe) == cudaSuccess && n > 0) info->mma_clusters16 = n;
            }
            cudaGetLastError();
        }
        if (info->mma_clusters16 < tiles * batch) split = 8;
    }
    // An ordinary launch: with the programmatic-dependent-launch attribute (the prologue overlapping the previous launch's tail) the
    // large cluster-split products of this kernel gained 2 us, but the small ones lost more (384^3: 10.3 -> 16.2 us; the five-matrix
    // chain 34.9 -> 37.4 us): measured, not kept.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles * split), 1, (unsigned)batch);
    cfg.blockDim = dim3(THREADS);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)split;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = split > 1 ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, product_mma_kernel, a, split, tiles_n);
}

}  // namespace mom
