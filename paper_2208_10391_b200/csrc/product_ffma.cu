// FFMA product kernel: C = A*B (+ Add terms) on CUDA cores in plain f32, for every pair of operand
// properties.  It is the comparison variant of the tensor-core kernel and the fallback for shapes
// TMA cannot address.  One CTA computes one 128x128 output tile over the tile's structural k-range
// (tile_k_range), so all-zero blocks of triangular operands are never read and structurally-zero
// output tiles are only zero-filled.
#include "device_common.cuh"
#include <algorithm>

#include "kernels.h"
#include "packed.cuh"

namespace mom {

namespace {

constexpr int BM = 128, BN = 128, BK = 16, THREADS = 256;     // a k-block is loaded as two halves of 8

__global__ void __launch_bounds__(THREADS, 2)
product_ffma_kernel(ProductArgs a) {
    __shared__ __align__(16) float As[2][BK][BM];     // k-major: As[k][row]
    __shared__ __align__(16) float Bs[2][BK][BN];

    const int tid = threadIdx.x;
    const long long inst = blockIdx.z;
    const float *__restrict__ A = a.A + inst * a.strideA;
    const float *__restrict__ B = a.B + inst * a.strideB;
    float *__restrict__ C = a.C + inst * a.strideC;
    const int m = a.m, n = a.n, k = a.k;
    // tile rows of a lower triangular A get heavier downwards: start them from the bottom, so that the longest tiles
    // are not the last ones to be scheduled
    const int by = a.pa == MOM_LOWER_TRI ? (int)(gridDim.y - 1 - blockIdx.y) : (int)blockIdx.y;
    const int r0 = by * BM, c0 = blockIdx.x * BN;
    const int r1 = min(r0 + BM, m), c1 = min(c0 + BN, n);

    int klo, khi;
    tile_k_range(a.pa, a.pb, r0, r1, c0, c1, k, &klo, &khi);
    klo &= ~(BK - 1);                     // extra leading elements are stored zeros

    // global -> shared mapping
    const int a_row = tid >> 1, a_k = (tid & 1) * 4;          // A tile: 128 rows x 8 k, one float4 along k
    const int b_k = tid >> 5, b_col = (tid & 31) * 4;         // B tile: 8 k x 128 cols, one float4 along n
    const bool a_vec = !a.transA && (k % 4 == 0) && ((reinterpret_cast<uintptr_t>(A) & 15) == 0);
    const bool b_vec = !a.transB && (n % 4 == 0) && ((reinterpret_cast<uintptr_t>(B) & 15) == 0);

    auto load_a = [&](int k0, float (&v)[4]) {
        const int r = r0 + a_row, kk = k0 + a_k;
        v[0] = v[1] = v[2] = v[3] = 0.0f;
        if (r < m && a.transA) {                 // stored k x m: consecutive threads read consecutive rows r
#pragma unroll
            for (int i = 0; i < 4; ++i) if (kk + i < k) v[i] = __ldg(A + (long long)(kk + i) * m + r);
        } else if (r < m) {
            const float *p = A + (long long)r * k + kk;
            if (a_vec && kk + 3 < k) {
                const float4 t = __ldg(reinterpret_cast<const float4 *>(p));
                v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) if (kk + i < k) v[i] = __ldg(p + i);
            }
        }
    };
    auto load_b = [&](int k0, float (&v)[4]) {
        const int kk = k0 + b_k, c = c0 + b_col;
        v[0] = v[1] = v[2] = v[3] = 0.0f;
        if (kk < k && a.transB) {                // stored n x k
#pragma unroll
            for (int i = 0; i < 4; ++i) if (c + i < n) v[i] = __ldg(B + (long long)(c + i) * k + kk);
        } else if (kk < k) {
            const float *p = B + (long long)kk * n + c;
            if (b_vec && c + 3 < n) {
                const float4 t = __ldg(reinterpret_cast<const float4 *>(p));
                v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) if (c + i < n) v[i] = __ldg(p + i);
            }
        }
    };
    auto store_tiles = [&](int buf, int half, const float (&va)[4], const float (&vb)[4]) {
#pragma unroll
        for (int i = 0; i < 4; ++i) As[buf][half * 8 + a_k + i][a_row] = va[i];
        *reinterpret_cast<float4 *>(&Bs[buf][half * 8 + b_k][b_col]) = make_float4(vb[0], vb[1], vb[2], vb[3]);
    };

    // each thread owns rows {ty*4..+3, 64+ty*4..+3} x cols {tx*4..+3, 64+tx*4..+3}
    const int ty = tid >> 4, tx = tid & 15;
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;

    if (klo < khi) {
        float va[4], vb[4], va2[4], vb2[4];
        load_a(klo, va);
        load_b(klo, vb);
        load_a(klo + 8, va2);
        load_b(klo + 8, vb2);
        store_tiles(0, 0, va, vb);
        store_tiles(0, 1, va2, vb2);
        __syncthreads();
        int buf = 0;
        for (int k0 = klo; k0 < khi; k0 += BK) {
            const bool more = k0 + BK < khi;
            if (more) { load_a(k0 + BK, va); load_b(k0 + BK, vb); load_a(k0 + BK + 8, va2); load_b(k0 + BK + 8, vb2); }
#pragma unroll
            for (int kk = 0; kk < BK; ++kk) {
                const float4 a0 = *reinterpret_cast<const float4 *>(&As[buf][kk][ty * 4]);
                const float4 a1 = *reinterpret_cast<const float4 *>(&As[buf][kk][64 + ty * 4]);
                const float4 b0 = *reinterpret_cast<const float4 *>(&Bs[buf][kk][tx * 4]);
                const float4 b1 = *reinterpret_cast<const float4 *>(&Bs[buf][kk][64 + tx * 4]);
                const float ar[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                const float br[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
            }
            if (more) {
                store_tiles(buf ^ 1, 0, va, vb);
                store_tiles(buf ^ 1, 1, va2, vb2);
                __syncthreads();
                buf ^= 1;
            }
        }
    }

    // fused epilogue: Add terms, structure mask (+0.0f outside), vector stores where aligned
    const bool c_vec = (n % 4 == 0) && ((reinterpret_cast<uintptr_t>(C) & 15) == 0);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = r0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (r >= m) continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int c = c0 + h * 64 + tx * 4;
            if (c >= n) continue;
            float v[4] = {acc[i][h * 4], acc[i][h * 4 + 1], acc[i][h * 4 + 2], acc[i][h * 4 + 3]};
            finish_row4(v, a.add, inst, r, c, n, n, a.pout, (n & 3) == 0);     // compact: the epilogue stays small in the instruction cache
            float *p = C + (long long)r * n + c;
            if (c_vec && c + 3 < n) {
                *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) if (c + j < n) p[j] = v[j];
            }
        }
    }
}

// X = src (+ Add terms), masked to the result's structure.  src_mode: 0 pointer, 1 Identity,
// 2 X itself (in place; used to add terms beyond the fused limit), 3 pointer to the transposed matrix.
// Bound by HBM: a thread takes four consecutive columns of four rows per pass (16-byte accesses where
// the layout allows, all loads of a pass issued before its first store).
constexpr int EW_TX = 64, EW_TY = 4, EW_ROWS = 4;

__global__ void __launch_bounds__(EW_TX * EW_TY)
elementwise_kernel(const float *__restrict__ src, long long src_stride, int src_mode, float *X, long long x_stride,
                   int rows, int cols, int out_prop, AddTerms add) {
    const long long inst = blockIdx.z;
    const float *S = src_mode == 2 ? X + inst * x_stride : src + inst * src_stride;
    float *Xi = X + inst * x_stride;
    const bool ld4 = (cols & 3) == 0;
    const bool vec_x = ld4 && (reinterpret_cast<uintptr_t>(Xi) & 15) == 0;
    const bool vec_s = vec_x && (src_mode == 2 || (src_mode == 0 && (reinterpret_cast<uintptr_t>(S) & 15) == 0));
    const int c = (blockIdx.x * EW_TX + threadIdx.x) * 4;
    if (c >= cols) return;
    for (int rb = blockIdx.y * (EW_TY * EW_ROWS) + threadIdx.y; rb < rows; rb += gridDim.y * (EW_TY * EW_ROWS)) {
        float v[EW_ROWS][4];
#pragma unroll
        for (int i = 0; i < EW_ROWS; ++i) {
            const int r = rb + i * EW_TY;
            v[i][0] = v[i][1] = v[i][2] = v[i][3] = 0.f;
            if (r >= rows) continue;
            if (src_mode == 1) {
#pragma unroll
                for (int j = 0; j < 4; ++j) v[i][j] = r == c + j ? 1.0f : 0.0f;
            } else if (vec_s) {
                const float4 *q = reinterpret_cast<const float4 *>(S + (long long)r * cols + c);
                const float4 t = src_mode == 2 ? __ldcg(q) : __ldg(q);      // X itself is never read through the read-only path
                v[i][0] = t.x; v[i][1] = t.y; v[i][2] = t.z; v[i][3] = t.w;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (c + j >= cols) continue;
                    if (src_mode == 3) v[i][j] = __ldg(S + (long long)(c + j) * rows + r);
                    else if (src_mode == 2) v[i][j] = __ldcg(S + (long long)r * cols + c + j);
                    else v[i][j] = __ldg(S + (long long)r * cols + c + j);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < EW_ROWS; ++i) {
            const int r = rb + i * EW_TY;
            if (r >= rows) continue;
            finish_row4(v[i], add, inst, r, c, cols, cols, out_prop, ld4);
            float *p = Xi + (long long)r * cols + c;
            if (vec_x) {
                *reinterpret_cast<float4 *>(p) = make_float4(v[i][0], v[i][1], v[i][2], v[i][3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) if (c + j < cols) p[j] = v[i][j];
            }
        }
    }
}

// The same when the source or an Add term is read through its transposed layout (stored cols x rows).  A
// CTA pass covers 16 rows x 256 columns of X; of a transposed matrix that is, per column, 16 consecutive
// floats.  They are staged through shared memory: thread t fetches column t's 64 bytes (whole sectors),
// then every thread picks its 4 x 4 entries from the tile.  (Read directly, every entry would touch a
// sector of its own: 82 us instead of 40 for a 4096 x 4096 sum.)
__global__ void __launch_bounds__(EW_TX * EW_TY)
elementwise_transposed_kernel(const float *__restrict__ src, long long src_stride, int src_mode, float *X, long long x_stride,
                              int rows, int cols, int out_prop, AddTerms add) {
    constexpr int PASS_ROWS = EW_TY * EW_ROWS, PASS_COLS = EW_TX * 4;
    __shared__ float tile[PASS_COLS][PASS_ROWS + 1];
    const long long inst = blockIdx.z;
    const float *S = src_mode == 2 ? X + inst * x_stride : src + inst * src_stride;
    float *Xi = X + inst * x_stride;
    const bool ld4 = (cols & 3) == 0;
    const bool vec_x = ld4 && (reinterpret_cast<uintptr_t>(Xi) & 15) == 0;
    const int tid = threadIdx.y * EW_TX + threadIdx.x;
    const int cbase = blockIdx.x * PASS_COLS, c = cbase + threadIdx.x * 4;
    // T is stored cols x rows: column cbase + tid of X is row cbase + tid of T
    auto stage = [&](const float *T, int rbase) {
        __syncthreads();                                     // the previous tile has been consumed
        const int tc = cbase + tid;
        if (tc < cols) {
            const float *q = T + (long long)tc * rows + rbase;
            const bool vec = (rows & 3) == 0 && (reinterpret_cast<uintptr_t>(T) & 15) == 0;
#pragma unroll
            for (int g = 0; g < PASS_ROWS / 4; ++g) {
                float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
                if (vec && rbase + 4 * g + 3 < rows) {
                    t = __ldg(reinterpret_cast<const float4 *>(q + 4 * g));
                } else {
                    if (rbase + 4 * g < rows) t.x = __ldg(q + 4 * g);
                    if (rbase + 4 * g + 1 < rows) t.y = __ldg(q + 4 * g + 1);
                    if (rbase + 4 * g + 2 < rows) t.z = __ldg(q + 4 * g + 2);
                    if (rbase + 4 * g + 3 < rows) t.w = __ldg(q + 4 * g + 3);
                }
                tile[tid][4 * g] = t.x; tile[tid][4 * g + 1] = t.y; tile[tid][4 * g + 2] = t.z; tile[tid][4 * g + 3] = t.w;
            }
        }
        __syncthreads();
    };
    for (int rbase = blockIdx.y * PASS_ROWS; rbase < rows; rbase += gridDim.y * PASS_ROWS) {     // the same trip count for the whole CTA
        float v[EW_ROWS][4];
        if (src_mode == 3) stage(S, rbase);
#pragma unroll
        for (int i = 0; i < EW_ROWS; ++i) {
            const int lr = threadIdx.y + i * EW_TY, r = rbase + lr;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float x = 0.f;
                if (r < rows && c + j < cols) {
                    if (src_mode == 3) x = tile[threadIdx.x * 4 + j][lr];
                    else if (src_mode == 1) x = r == c + j ? 1.0f : 0.0f;
                    else if (src_mode == 2) x = __ldcg(S + (long long)r * cols + c + j);
                    else x = __ldg(S + (long long)r * cols + c + j);
                }
                v[i][j] = x;
            }
        }
#pragma unroll 1
        for (int t = 0; t < add.count; ++t) {
            const float *p = add.ptr[t];
            if (p) p += inst * add.stride[t];
            const bool tr = p && ((add.transposed >> t) & 1u);
            if (tr) stage(p, rbase);
#pragma unroll
            for (int i = 0; i < EW_ROWS; ++i) {
                const int lr = threadIdx.y + i * EW_TY, r = rbase + lr;
                if (r >= rows) continue;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (c + j >= cols) continue;
                    if (!p) v[i][j] += r == c + j ? 1.0f : 0.0f;
                    else if (tr) v[i][j] += tile[threadIdx.x * 4 + j][lr];
                    else if ((add.aliases_out >> t) & 1u) v[i][j] += __ldcg(p + (long long)r * cols + c + j);
                    else v[i][j] += __ldg(p + (long long)r * cols + c + j);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < EW_ROWS; ++i) {
            const int r = rbase + threadIdx.y + i * EW_TY;
            if (r >= rows || c >= cols) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) v[i][j] = in_structure(out_prop, r, c + j) ? v[i][j] : 0.0f;
            float *o = Xi + (long long)r * cols + c;
            if (vec_x) {
                *reinterpret_cast<float4 *>(o) = make_float4(v[i][0], v[i][1], v[i][2], v[i][3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) if (c + j < cols) o[j] = v[i][j];
            }
        }
    }
}

// Product with a Diagonal operand: C = D*B scales row r of B by d_r, C = A*D scales column c of A by d_c
// (+ Add terms, structure mask).  One pass over the other operand, bound by HBM: a thread takes four
// consecutive columns of a row (one 16-byte load and store where the layout allows), only the diagonal of
// D and the structural part of the other operand are read.
constexpr int SCALE_TX = 64, SCALE_TY = 4;

__global__ void __launch_bounds__(SCALE_TX * SCALE_TY)
scale_kernel(ProductArgs a) {
    const long long inst = blockIdx.z;
    const bool left = a.pa == MOM_DIAGONAL;                 // D on the left: the other operand is B
    const float *__restrict__ D = (left ? a.A : a.B) + inst * (left ? a.strideA : a.strideB);
    const float *__restrict__ S = (left ? a.B : a.A) + inst * (left ? a.strideB : a.strideA);
    const int ps = left ? a.pb : a.pa;
    const bool trans = left ? a.transB != 0 : a.transA != 0;   // S is stored n x m
    float *__restrict__ C = a.C + inst * a.strideC;
    const int m = a.m, n = a.n;
    const long long dstep = (long long)a.k + 1;             // D is k x k: d_i sits at i * (k + 1)
    const bool vec = !trans && (n & 3) == 0 && ((reinterpret_cast<uintptr_t>(S) | reinterpret_cast<uintptr_t>(C)) & 15) == 0;
    const int c = (blockIdx.x * SCALE_TX + threadIdx.x) * 4;
    if (c >= n) return;
    float dc[4] = {0.f, 0.f, 0.f, 0.f};                     // D on the right: this thread's four columns keep their factors
    if (!left) {
#pragma unroll
        for (int j = 0; j < 4; ++j) if (c + j < n) dc[j] = __ldg(D + (c + j) * dstep);
    }
    // four rows per thread and pass: their loads are all issued before the first store
    constexpr int ROWS = 4;
    for (int rb = blockIdx.y * (SCALE_TY * ROWS) + threadIdx.y; rb < m; rb += gridDim.y * (SCALE_TY * ROWS)) {
        float s[ROWS][4];
        float dr[ROWS];
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
            const int r = rb + i * SCALE_TY;
            s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
            dr[i] = 0.f;
            if (r >= m) continue;
            // the four entries lie inside S's structure?  (outside, the stored zeros need not be read)
            const bool any = ps == MOM_GENERAL || ps == MOM_SYMMETRIC || (ps == MOM_LOWER_TRI && c <= r) || (ps == MOM_UPPER_TRI && c + 3 >= r) ||
                             (ps == MOM_DIAGONAL && c <= r && c + 3 >= r);
            if (any) {
                if (vec) {
                    const float4 t = __ldg(reinterpret_cast<const float4 *>(S + (long long)r * n + c));
                    s[i][0] = t.x; s[i][1] = t.y; s[i][2] = t.z; s[i][3] = t.w;
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (c + j < n) s[i][j] = __ldg(trans ? S + (long long)(c + j) * m + r : S + (long long)r * n + c + j);
                }
            }
            if (left) dr[i] = __ldg(D + r * dstep);
        }
#pragma unroll
        for (int i = 0; i < ROWS; ++i) {
            const int r = rb + i * SCALE_TY;
            if (r >= m) continue;
            float v[4];
#pragma unroll
            // (+ 0.0f: a product with a stored zero is +0 whatever the sign of d, so the diagonal of a strictly
            // triangular result holds +0.0f like every entry outside a structure)
            for (int j = 0; j < 4; ++j) v[j] = fmaf(left ? dr[i] : dc[j], s[i][j], 0.0f);
            finish_row4(v, a.add, inst, r, c, n, n, a.pout, (n & 3) == 0);
            float *p = C + (long long)r * n + c;
            if (vec) {
                *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) if (c + j < n) p[j] = v[j];
            }
        }
    }
}

}  // namespace

cudaError_t launch_scale(const ProductArgs &a, int batch, cudaStream_t stream) {
    const int gx = (a.n + SCALE_TX * 4 - 1) / (SCALE_TX * 4);
    int gy = (a.m + SCALE_TY * 4 - 1) / (SCALE_TY * 4);     // a CTA pass covers 16 rows
    const int want = (148 * 16 + gx - 1) / gx;              // a few CTAs per SM; rows beyond that are looped over
    if (gy > want) gy = want;
    if (gy < 1) gy = 1;
    scale_kernel<<<dim3(gx, gy, batch), dim3(SCALE_TX, SCALE_TY), 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_product_ffma(const ProductArgs &a, int batch, cudaStream_t stream) {
    dim3 grid((a.n + BN - 1) / BN, (a.m + BM - 1) / BM, batch);
    product_ffma_kernel<<<grid, THREADS, 0, stream>>>(a);
    return cudaGetLastError();
}

// Packed triangle <-> dense matrix, one thread per 16-byte group of a row (see packed.cuh for the container).
// unpack: the dense n x n matrix gets the stored entries and zeros everywhere else; pack: the container gets the
// dense matrix's entries of every stored position (zeros beyond the last column).  Bound by HBM; grid.z = instances.
namespace {
__global__ void __launch_bounds__(256)
unpack_kernel(const float *__restrict__ src, long long src_stride, float *__restrict__ dst, long long dst_stride, int n, int lower) {
    const int groups = (n + 3) >> 2;
    src += (long long)blockIdx.z * src_stride;
    dst += (long long)blockIdx.z * dst_stride;
    const bool vec = (n & 3) == 0;                               // dense rows are 16-byte aligned
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < (long long)n * groups; e += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(e / groups), c = (int)(e % groups) << 2;
        const PackedRow row = packed_row(lower != 0, n, r);
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c >= row.first && c < row.end) v = __ldg(reinterpret_cast<const float4 *>(src + row.offset + (c - row.first)));
        float *d = dst + (long long)r * n + c;
        if (vec) {
            *reinterpret_cast<float4 *>(d) = v;
        } else {
            d[0] = v.x;
            if (c + 1 < n) d[1] = v.y;
            if (c + 2 < n) d[2] = v.z;
            if (c + 3 < n) d[3] = v.w;
        }
    }
}

__global__ void __launch_bounds__(256)
pack_kernel(const float *__restrict__ src, long long src_stride, float *__restrict__ dst, long long dst_stride, int n, int lower) {
    const int groups = (n + 3) >> 2;
    src += (long long)blockIdx.z * src_stride;
    dst += (long long)blockIdx.z * dst_stride;
    const bool vec = (n & 3) == 0;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < (long long)n * groups; e += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(e / groups), c = (int)(e % groups) << 2;
        const PackedRow row = packed_row(lower != 0, n, r);
        if (c < row.first || c >= row.end) continue;
        const float *a = src + (long long)r * n + c;
        float4 v;
        if (vec) {
            v = __ldg(reinterpret_cast<const float4 *>(a));
        } else {
            v.x = __ldg(a);
            v.y = c + 1 < n ? __ldg(a + 1) : 0.f;
            v.z = c + 2 < n ? __ldg(a + 2) : 0.f;
            v.w = c + 3 < n ? __ldg(a + 3) : 0.f;
        }
        *reinterpret_cast<float4 *>(dst + row.offset + (c - row.first)) = v;
    }
}
}  // namespace

cudaError_t launch_unpack(const float *src, long long src_stride, float *dst, long long dst_stride, int n, bool lower, int batch,
                          cudaStream_t stream) {
    const long long work = (long long)n * ((n + 3) >> 2);
    const unsigned gx = (unsigned)std::min<long long>((work + 255) / 256, 148 * 16);
    unpack_kernel<<<dim3(gx, 1, batch), 256, 0, stream>>>(src, src_stride, dst, dst_stride, n, lower ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_pack(const float *src, long long src_stride, float *dst, long long dst_stride, int n, bool lower, int batch,
                        cudaStream_t stream) {
    const long long work = (long long)n * ((n + 3) >> 2);
    const unsigned gx = (unsigned)std::min<long long>((work + 255) / 256, 148 * 16);
    pack_kernel<<<dim3(gx, 1, batch), 256, 0, stream>>>(src, src_stride, dst, dst_stride, n, lower ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_elementwise(const float *src, long long src_stride, int src_mode, float *X, long long x_stride,
                               int rows, int cols, int out_prop, const AddTerms &add, int batch, cudaStream_t stream) {
    const int gx = (cols + EW_TX * 4 - 1) / (EW_TX * 4);
    int gy = (rows + EW_TY * EW_ROWS - 1) / (EW_TY * EW_ROWS);
    const int want = (148 * 16 + gx - 1) / gx;              // a few CTAs per SM; rows beyond that are looped over
    if (gy > want) gy = want;
    if (gy < 1) gy = 1;
    const bool transposed = src_mode == 3 || (add.transposed & ((1u << add.count) - 1u)) != 0;
    if (transposed) elementwise_transposed_kernel<<<dim3(gx, gy, batch), dim3(EW_TX, EW_TY), 0, stream>>>(src, src_stride, src_mode, X, x_stride, rows, cols, out_prop, add);
    else elementwise_kernel<<<dim3(gx, gy, batch), dim3(EW_TX, EW_TY), 0, stream>>>(src, src_stride, src_mode, X, x_stride, rows, cols, out_prop, add);
    return cudaGetLastError();
}

}  // namespace mom
