// Fused small-equation kernel: a whole plan (every product, the Add terms, the structure mask) for
// one instance per CTA, with the operands and all intermediates resident in shared memory.  Batched
// small equations are bound by HBM traffic, so each operand is read exactly once (only the
// structural part of triangular operands), nothing intermediate touches global memory, and several
// CTAs per SM overlap one instance's loads with another's arithmetic.  The kernel is bound by
// instruction issue as much as by memory, so the per-instance code is kept short: the epilogue loops over
// the Add terms instead of unrolling them, and the low part of the operand split is not rounded.
//
// Two arithmetic variants of the products:
//   MMA   warp-level mma.sync m16n8k8 tf32 with the 3xTF32 split done in registers on the
//         fragments (a = hi + lo; lo*hi + hi*lo + hi*hi accumulated in f32).  The problem per CTA
//         is far too small for a tcgen05/TMEM pipeline, and the bound here is HBM, not the tensor pipe.
//   FFMA  plain f32 FMA on cells of 2 rows x 4 columns.
#include <cstring>

#include "device_info.h"
#include "fused_small.h"

namespace mom {

namespace {

constexpr int THREADS = FUSED_THREADS;
constexpr int WARPS = THREADS / 32;

// Copy one operand (rows x cols, row-major, leading dimension cols) into shared memory with leading
// dimension ld.  Only the part inside the structure is read; the rest is zero-filled.  16-byte
// asynchronous copies (cp.async) keep every load of every operand in flight at once; a copy with
// source size 0 writes zeros.  The caller waits with cp_async_wait_all() + __syncthreads().
__device__ void load_operand(float *__restrict__ dst, const float *__restrict__ src, int rows, int cols, int ld, int prop,
                             int transposed) {
    const int vec_per_row = (cols + 3) >> 2;
    const bool vec_ok = !transposed && (cols & 3) == 0 && (reinterpret_cast<uintptr_t>(src) & 15) == 0;
    // thread -> (row, float4 column); when the row length divides the block the column stays fixed and
    // the row advances by a constant, which avoids a division per copy
    const bool regular = (THREADS % vec_per_row) == 0;
    int r = threadIdx.x / vec_per_row, c = (threadIdx.x - r * vec_per_row) << 2;
    const int r_step = THREADS / vec_per_row;
    for (int e = threadIdx.x; e < rows * vec_per_row; e += THREADS, r += r_step) {
        if (!regular) { r = e / vec_per_row; c = (e - r * vec_per_row) << 2; }
        // columns [c, c+4) intersect the structure of row r?
        const bool needed = prop == MOM_GENERAL || prop == MOM_SYMMETRIC || (prop == MOM_LOWER_TRI && c <= r) || (prop == MOM_UPPER_TRI && c + 3 >= r) ||
                            (prop == MOM_DIAGONAL && c <= r && c + 3 >= r);
        float *d = dst + r * ld + c;
        const float *p = src + (size_t)r * cols + c;
        if (vec_ok) {
            const uint32_t daddr = static_cast<uint32_t>(__cvta_generic_to_shared(d));
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(daddr), "l"(p), "r"(needed ? 16 : 0) : "memory");
        } else {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (needed && transposed) {          // stored cols x rows: entry (r, c) is at c * rows + r
                if (c < cols) v.x = __ldg(src + (size_t)c * rows + r);
                if (c + 1 < cols) v.y = __ldg(src + (size_t)(c + 1) * rows + r);
                if (c + 2 < cols) v.z = __ldg(src + (size_t)(c + 2) * rows + r);
                if (c + 3 < cols) v.w = __ldg(src + (size_t)(c + 3) * rows + r);
            } else if (needed) {
                if (c < cols) v.x = __ldg(p);
                if (c + 1 < cols) v.y = __ldg(p + 1);
                if (c + 2 < cols) v.z = __ldg(p + 2);
                if (c + 3 < cols) v.w = __ldg(p + 3);
            }
            *reinterpret_cast<float4 *>(d) = v;
        }
    }
}

__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

// a = hi + lo with both halves representable in tf32.  Rounding to tf32 (10 mantissa bits, ties away
// from zero) is done on the bit pattern with full-rate integer instructions: add half a unit of the
// last kept place to the magnitude, clear the 13 dropped bits.  (The cvt.rna.tf32.f32 instruction gives
// the same result but issues at conversion-pipe rate, which made it the bottleneck of this kernel.)
__device__ __forceinline__ uint32_t round_tf32_bits(float a) { return (__float_as_uint(a) + 0x1000u) & 0xFFFFE000u; }
// The low part a - hi is exact in f32 and is handed to the MMA as it is: the tensor core reads only the
// tf32 part of an operand register (sign, exponent, 10 mantissa bits), i.e. it drops bits that are worth
// at most 2^-21 of a -- the size of the lo*lo term this scheme leaves out anyway.
__device__ __forceinline__ void split_tf32(float a, uint32_t &hi, uint32_t &lo) {
    hi = round_tf32_bits(a);
    lo = __float_as_uint(a - __uint_as_float(hi));
}

__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// What the kernel's loop hands to the products of one instance.
struct Instance {
    long long inst;
    float *smem;
};
__device__ __forceinline__ float *at(const Instance &in, int off) { return in.smem + off; }

// the equation's value at (r, c) and (r, c + 1) given the chain's values there: Add terms left to right
// in a compact loop, then the structure mask
__device__ __forceinline__ void finish_pair(const FusedPlan &fp, const Instance &in, int r, int c, int n, int pout, bool two,
                                            float &x0, float &x1) {
#pragma unroll 1
    for (int t = 0; t < fp.add.count; ++t) {
        const float *p = fp.add.ptr[t];
        if (!p) {
            x0 += r == c ? 1.0f : 0.0f;
            x1 += r == c + 1 ? 1.0f : 0.0f;
            continue;
        }
        p += in.inst * fp.add.stride[t];
        const bool tr = (fp.add.transposed >> t) & 1u;
        x0 += __ldg(p + (tr ? (long long)c * fp.add.rows + r : (long long)r * n + c));
        if (two) x1 += __ldg(p + (tr ? (long long)(c + 1) * fp.add.rows + r : (long long)r * n + c + 1));
    }
    x0 = in_structure(pout, r, c) ? x0 : 0.0f;
    x1 = in_structure(pout, r, c + 1) ? x1 : 0.0f;
}

// store one output entry pair (r, c), (r, c+1) of a step: into shared memory for an intermediate
// (masked to its structure, padded columns zero) or, on the last step, into X with the Add terms
__device__ __forceinline__ void store_pair(const FusedPlan &fp, const FusedStep &st, const Instance &in, int r, int c,
                                           float v0, float v1) {
    if (r >= st.m) return;
    if (st.out_off >= 0) {
        if (c >= st.ldc) return;
        float *C = at(in, st.out_off) + r * st.ldc + c;
        C[0] = (c < st.n && in_structure(st.pout, r, c)) ? v0 : 0.f;
        if (c + 1 < st.ldc) C[1] = (c + 1 < st.n && in_structure(st.pout, r, c + 1)) ? v1 : 0.f;
    } else {
        if (c >= st.n) return;
        float *X = fp.out + in.inst * fp.out_stride + (size_t)r * st.n + c;
        const bool two = c + 1 < st.n;
        finish_pair(fp, in, r, c, st.n, st.pout, two, v0, v1);
        if (two) {
            if ((reinterpret_cast<uintptr_t>(X) & 7) == 0) *reinterpret_cast<float2 *>(X) = make_float2(v0, v1);
            else { X[0] = v0; X[1] = v1; }
        } else {
            X[0] = v0;
        }
    }
}

// Whole-tile tensor-core product (m, n multiples of 16 resp. 8*NTW, k a multiple of 8): output tiles of
// 16 x (8*NTW) dealt round-robin to the warps; no clamping, pointers advance by constants.  The small
// terms (lo*hi, hi*lo) and the main term (hi*hi) go to separate accumulators: two independent MMA
// chains per 8-column tile instead of one three times as long.
template <int NTW>
__device__ void product_mma_whole(const FusedPlan &fp, const FusedStep &st, const Instance &in) {
    const float *__restrict__ A = at(in, st.a_off);
    const float *__restrict__ B = at(in, st.b_off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    constexpr int TW = 8 * NTW;
    const int tiles_n = st.n / TW, tiles = (st.m >> 4) * tiles_n;
    for (int tile = warp; tile < tiles; tile += WARPS) {
        const int r0 = (tile / tiles_n) << 4, c0 = (tile % tiles_n) * TW;
        int klo, khi;
        tile_k_range(st.pa, st.pb, r0, r0 + 16, c0, c0 + TW, st.k, &klo, &khi);
        klo &= ~7;
        float main_acc[NTW][4], small_acc[NTW][4];
#pragma unroll
        for (int j = 0; j < NTW; ++j)
#pragma unroll
            for (int q = 0; q < 4; ++q) main_acc[j][q] = small_acc[j][q] = 0.f;
        const float *a0p = A + (r0 + g) * st.lda + klo + t, *a1p = a0p + 8 * st.lda;
        const float *bp = B + (klo + t) * st.ldb + c0 + g;
        const int b4 = 4 * st.ldb, b8 = 8 * st.ldb;
#pragma unroll 2
        for (int l = klo; l < khi; l += 8, a0p += 8, a1p += 8, bp += b8) {
            uint32_t a_hi[4], a_lo[4];
            split_tf32(a0p[0], a_hi[0], a_lo[0]);
            split_tf32(a1p[0], a_hi[1], a_lo[1]);
            split_tf32(a0p[4], a_hi[2], a_lo[2]);
            split_tf32(a1p[4], a_hi[3], a_lo[3]);
#pragma unroll
            for (int j = 0; j < NTW; ++j) {
                uint32_t b_hi[2], b_lo[2];
                split_tf32(bp[8 * j], b_hi[0], b_lo[0]);
                split_tf32(bp[b4 + 8 * j], b_hi[1], b_lo[1]);
                mma_tf32(small_acc[j], a_lo, b_hi);
                mma_tf32(main_acc[j], a_hi, b_hi);
                mma_tf32(small_acc[j], a_hi, b_lo);
            }
        }
        // Whole tiles need no bounds checks, and all addresses derive from one base: entries (ra, c), (ra, c + 1),
        // (ra + 8, c), (ra + 8, c + 1) with c = c0 + 8 j + 2 t.  Row lengths are multiples of 8 here, so pairs are
        // 8-byte aligned.
        const int ra = r0 + g, c = c0 + 2 * t;
        const bool masked = st.pout != MOM_GENERAL && st.pout != MOM_SYMMETRIC;
        if (st.out_off >= 0) {
            float *C = at(in, st.out_off) + ra * st.ldc + c;
#pragma unroll
            for (int j = 0; j < NTW; ++j) {
                float2 lo2 = make_float2(main_acc[j][0] + small_acc[j][0], main_acc[j][1] + small_acc[j][1]);
                float2 hi2 = make_float2(main_acc[j][2] + small_acc[j][2], main_acc[j][3] + small_acc[j][3]);
                if (masked) {
                    const int cc = c + 8 * j;
                    lo2.x = in_structure(st.pout, ra, cc) ? lo2.x : 0.f;       lo2.y = in_structure(st.pout, ra, cc + 1) ? lo2.y : 0.f;
                    hi2.x = in_structure(st.pout, ra + 8, cc) ? hi2.x : 0.f;   hi2.y = in_structure(st.pout, ra + 8, cc + 1) ? hi2.y : 0.f;
                }
                *reinterpret_cast<float2 *>(C + 8 * j) = lo2;
                *reinterpret_cast<float2 *>(C + 8 * st.ldc + 8 * j) = hi2;
            }
        } else if (fp.add.transposed == 0 && (reinterpret_cast<uintptr_t>(fp.out) & 7) == 0 && (fp.out_stride & 1) == 0) {
            const long long at0 = (long long)ra * st.n + c, at8 = at0 + 8LL * st.n;
            float2 lo2[NTW], hi2[NTW];
#pragma unroll
            for (int j = 0; j < NTW; ++j) {
                lo2[j] = make_float2(main_acc[j][0] + small_acc[j][0], main_acc[j][1] + small_acc[j][1]);
                hi2[j] = make_float2(main_acc[j][2] + small_acc[j][2], main_acc[j][3] + small_acc[j][3]);
            }
#pragma unroll 1
            for (int term = 0; term < fp.add.count; ++term) {                  // Add terms, left to right
                const float *p = fp.add.ptr[term];
                if (!p) {                                                       // Identity
#pragma unroll
                    for (int j = 0; j < NTW; ++j) {
                        const int cc = c + 8 * j;
                        lo2[j].x += ra == cc ? 1.f : 0.f;       lo2[j].y += ra == cc + 1 ? 1.f : 0.f;
                        hi2[j].x += ra + 8 == cc ? 1.f : 0.f;   hi2[j].y += ra + 8 == cc + 1 ? 1.f : 0.f;
                    }
                    continue;
                }
                p += in.inst * fp.add.stride[term];
                const bool vec = (reinterpret_cast<uintptr_t>(p) & 7) == 0;
#pragma unroll
                for (int j = 0; j < NTW; ++j) {
                    float2 x, y;
                    if (vec) {
                        x = __ldg(reinterpret_cast<const float2 *>(p + at0 + 8 * j));
                        y = __ldg(reinterpret_cast<const float2 *>(p + at8 + 8 * j));
                    } else {
                        x = make_float2(__ldg(p + at0 + 8 * j), __ldg(p + at0 + 8 * j + 1));
                        y = make_float2(__ldg(p + at8 + 8 * j), __ldg(p + at8 + 8 * j + 1));
                    }
                    lo2[j].x += x.x; lo2[j].y += x.y; hi2[j].x += y.x; hi2[j].y += y.y;
                }
            }
            float *X = fp.out + in.inst * fp.out_stride;
#pragma unroll
            for (int j = 0; j < NTW; ++j) {
                if (masked) {
                    const int cc = c + 8 * j;
                    lo2[j].x = in_structure(st.pout, ra, cc) ? lo2[j].x : 0.f;       lo2[j].y = in_structure(st.pout, ra, cc + 1) ? lo2[j].y : 0.f;
                    hi2[j].x = in_structure(st.pout, ra + 8, cc) ? hi2[j].x : 0.f;   hi2[j].y = in_structure(st.pout, ra + 8, cc + 1) ? hi2[j].y : 0.f;
                }
                *reinterpret_cast<float2 *>(X + at0 + 8 * j) = lo2[j];
                *reinterpret_cast<float2 *>(X + at8 + 8 * j) = hi2[j];
            }
        } else {
#pragma unroll
            for (int j = 0; j < NTW; ++j) {
                store_pair(fp, st, in, r0 + g, c0 + 8 * j + 2 * t, main_acc[j][0] + small_acc[j][0], main_acc[j][1] + small_acc[j][1]);
                store_pair(fp, st, in, r0 + g + 8, c0 + 8 * j + 2 * t, main_acc[j][2] + small_acc[j][2], main_acc[j][3] + small_acc[j][3]);
            }
        }
    }
}

// One product on tensor cores: 16 x 16 output tiles dealt round-robin to the warps.
__device__ void product_mma(const FusedPlan &fp, const FusedStep &st, const Instance &in) {
    if (((st.m | st.n) & 15) == 0 && (st.k & 7) == 0) {
        // 16 x 16 tiles per warp also when that leaves warps idle: the kernel is bound by instruction issue, and a
        // 16 x 16 tile shares the left fragments (and their splits) between its two column halves
        product_mma_whole<2>(fp, st, in);
        return;
    }
    const float *__restrict__ A = at(in, st.a_off);
    const float *__restrict__ B = at(in, st.b_off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int tiles_n = (st.n + 15) >> 4, tiles = ((st.m + 15) >> 4) * tiles_n;
    for (int tile = warp; tile < tiles; tile += WARPS) {
        const int r0 = (tile / tiles_n) << 4, c0 = (tile % tiles_n) << 4;
        int klo, khi;
        tile_k_range(st.pa, st.pb, r0, min(r0 + 16, st.m), c0, min(c0 + 16, st.n), st.k, &klo, &khi);
        klo &= ~7;
        float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        // rows / columns outside the matrix are clamped for the address and zeroed by the flag
        const int ra = min(r0 + g, st.m - 1), rb = min(r0 + g + 8, st.m - 1);
        const float fa = r0 + g < st.m ? 1.f : 0.f, fb = r0 + g + 8 < st.m ? 1.f : 0.f;
        const int n0 = min(c0 + g, st.n - 1), n1 = min(c0 + 8 + g, st.n - 1);
        const float f0 = c0 + g < st.n ? 1.f : 0.f, f1 = c0 + 8 + g < st.n ? 1.f : 0.f;
        for (int l = klo; l < khi; l += 8) {
            const int k0 = min(l + t, st.k - 1), k1 = min(l + t + 4, st.k - 1);
            const float e0 = l + t < st.k ? 1.f : 0.f, e1 = l + t + 4 < st.k ? 1.f : 0.f;
            uint32_t a_hi[4], a_lo[4], b_hi[2], b_lo[2];
            split_tf32(A[ra * st.lda + k0] * (fa * e0), a_hi[0], a_lo[0]);
            split_tf32(A[rb * st.lda + k0] * (fb * e0), a_hi[1], a_lo[1]);
            split_tf32(A[ra * st.lda + k1] * (fa * e1), a_hi[2], a_lo[2]);
            split_tf32(A[rb * st.lda + k1] * (fb * e1), a_hi[3], a_lo[3]);
            split_tf32(B[k0 * st.ldb + n0] * (f0 * e0), b_hi[0], b_lo[0]);
            split_tf32(B[k1 * st.ldb + n0] * (f0 * e1), b_hi[1], b_lo[1]);
            mma_tf32(acc[0], a_lo, b_hi);
            mma_tf32(acc[0], a_hi, b_lo);
            mma_tf32(acc[0], a_hi, b_hi);
            split_tf32(B[k0 * st.ldb + n1] * (f1 * e0), b_hi[0], b_lo[0]);
            split_tf32(B[k1 * st.ldb + n1] * (f1 * e1), b_hi[1], b_lo[1]);
            mma_tf32(acc[1], a_lo, b_hi);
            mma_tf32(acc[1], a_hi, b_lo);
            mma_tf32(acc[1], a_hi, b_hi);
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            store_pair(fp, st, in, r0 + g, c0 + 8 * h + 2 * t, acc[h][0], acc[h][1]);
            store_pair(fp, st, in, r0 + g + 8, c0 + 8 * h + 2 * t, acc[h][2], acc[h][3]);
        }
    }
}

// One product with plain FMA: cells of 2 rows x 4 columns dealt round-robin to the threads.
__device__ void product_ffma(const FusedPlan &fp, const FusedStep &st, const Instance &in) {
    const float *__restrict__ A = at(in, st.a_off);
    const float *__restrict__ B = at(in, st.b_off);
    const int cells_per_row = (st.n + 3) >> 2, row_pairs = (st.m + 1) >> 1;
    for (int cell = threadIdx.x; cell < row_pairs * cells_per_row; cell += THREADS) {
        const int r = (cell / cells_per_row) << 1, c = (cell % cells_per_row) << 2;
        const bool two = r + 1 < st.m;
        int klo, khi;
        tile_k_range(st.pa, st.pb, r, two ? r + 2 : r + 1, c, min(c + 4, st.n), st.k, &klo, &khi);
        float a0[4] = {0.f, 0.f, 0.f, 0.f}, a1[4] = {0.f, 0.f, 0.f, 0.f};
        const float *ar0 = A + r * st.lda, *ar1 = A + (two ? r + 1 : r) * st.lda;
        for (int l = klo; l < khi; ++l) {
            const float4 b = *reinterpret_cast<const float4 *>(B + l * st.ldb + c);   // padded columns hold zeros
            const float x0 = ar0[l], x1 = ar1[l];
            a0[0] = fmaf(x0, b.x, a0[0]); a0[1] = fmaf(x0, b.y, a0[1]); a0[2] = fmaf(x0, b.z, a0[2]); a0[3] = fmaf(x0, b.w, a0[3]);
            a1[0] = fmaf(x1, b.x, a1[0]); a1[1] = fmaf(x1, b.y, a1[1]); a1[2] = fmaf(x1, b.z, a1[2]); a1[3] = fmaf(x1, b.w, a1[3]);
        }
        store_pair(fp, st, in, r, c, a0[0], a0[1]);
        store_pair(fp, st, in, r, c + 2, a0[2], a0[3]);
        if (two) {
            store_pair(fp, st, in, r + 1, c, a1[0], a1[1]);
            store_pair(fp, st, in, r + 1, c + 2, a1[2], a1[3]);
        }
    }
}

template <bool MMA>
__global__ void __launch_bounds__(THREADS, 4)
fused_small_kernel(const FusedPlan fp) {
    extern __shared__ __align__(16) float smem[];
    Instance in;
    in.smem = smem;
    const uint32_t smem_base = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
    for (long long inst = blockIdx.x; inst < fp.batch; inst += gridDim.x) {
        in.inst = inst;
        for (int i = 0; i < fp.n_ops; ++i) {
            const FusedOperand &op = fp.ops[i];
            const float *src = op.ptr + inst * op.stride;
            if (op.tab_end > op.tab_begin) {
                const uint2 *e = fp.copy_table + (size_t)op.tab_begin * THREADS + threadIdx.x;
                for (int row = op.tab_begin; row < op.tab_end; ++row, e += THREADS) {
                    const uint2 c = __ldg(e);
                    if (c.x != FUSED_COPY_NONE)
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_base + (c.x & ~15u)), "l"(src + c.y), "r"((c.x & 1u) ? 16 : 0) : "memory");
                }
            } else {
                load_operand(smem + op.smem_off, src, op.rows, op.cols, op.ld, op.prop, op.transposed);
            }
        }
        cp_async_wait_all();
        __syncthreads();
        for (int s = 0; s < fp.n_steps; ++s) {
            if (MMA) product_mma(fp, fp.steps[s], in);
            else product_ffma(fp, fp.steps[s], in);
            __syncthreads();
        }
    }
}

}  // namespace

int fused_copy_table(int rows, int cols, int prop, int smem_off, int ld, std::vector<uint2> &table) {
    const size_t first = table.size();
    const bool lower = prop == MOM_LOWER_TRI || prop == MOM_DIAGONAL, upper = prop == MOM_UPPER_TRI || prop == MOM_DIAGONAL;
    for (int r = 0; r < rows; ++r) {
        const int block = r & ~15;
        for (int c = 0; c < cols; c += 4) {
            if ((lower && c >= block + 16) || (upper && c + 3 < block)) continue;      // never read by any product
            const bool needed = !((lower && c > r) || (upper && c + 3 < r));
            table.push_back(make_uint2((uint32_t)(smem_off + r * ld + c) * 4u | (needed ? 1u : 0u), (uint32_t)(r * cols + c)));
        }
    }
    while ((table.size() - first) % FUSED_THREADS != 0) table.push_back(make_uint2(FUSED_COPY_NONE, 0));
    return (int)((table.size() - first) / FUSED_THREADS);
}

cudaError_t launch_fused_small(const FusedPlan &fp, size_t smem_bytes, cudaStream_t stream) {
    const int v = fp.use_mma ? 1 : 0;
    int sm_count = 0;
    {
        std::lock_guard<std::mutex> lock(device_info_mutex());
        DeviceInfo *info = current_device_info();
        if (!info) return cudaErrorInvalidDevice;
        sm_count = info->sm_count;
        if ((int)smem_bytes > info->fused_max_smem[v]) {
            cudaError_t e = v ? cudaFuncSetAttribute(fused_small_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes)
                              : cudaFuncSetAttribute(fused_small_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
            if (e != cudaSuccess) return e;
            info->fused_max_smem[v] = (int)smem_bytes;
        }
    }
    // enough CTAs to fill every SM several times over; each walks instances with a grid stride
    long long per_sm = smem_bytes ? (long long)(220 * 1024) / (long long)smem_bytes : 8;
    if (per_sm > 8) per_sm = 8;
    if (per_sm < 1) per_sm = 1;
    long long grid = (long long)sm_count * per_sm;
    if (grid > fp.batch) grid = fp.batch;
    if (v) fused_small_kernel<true><<<(unsigned)grid, THREADS, smem_bytes, stream>>>(fp);
    else fused_small_kernel<false><<<(unsigned)grid, THREADS, smem_bytes, stream>>>(fp);
    return cudaGetLastError();
}

}  // namespace mom
