// FFMA product kernel: C = A*B (+ Add terms) on CUDA cores in plain f32, for every pair of operand
// properties.  It is the comparison variant of the tensor-core kernel and the fallback for shapes
// TMA cannot address.  One CTA computes one 128x128 output tile over the tile's structural k-range
// (tile_k_range), so all-zero blocks of triangular operands are never read and structurally-zero
// output tiles are only zero-filled.
#include "device_common.cuh"
#include "kernels.h"

namespace mom {

namespace {

constexpr int BM = 128, BN = 128, BK = 8, THREADS = 256;

__global__ void __launch_bounds__(THREADS)
product_ffma_kernel(ProductArgs a) {
    __shared__ __align__(16) float As[2][BK][BM];     // k-major: As[k][row]
    __shared__ __align__(16) float Bs[2][BK][BN];

    const int tid = threadIdx.x;
    const long long inst = blockIdx.z;
    const float *__restrict__ A = a.A + inst * a.strideA;
    const float *__restrict__ B = a.B + inst * a.strideB;
    float *__restrict__ C = a.C + inst * a.strideC;
    const int m = a.m, n = a.n, k = a.k;
    const int r0 = blockIdx.y * BM, c0 = blockIdx.x * BN;
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
    auto store_tiles = [&](int buf, const float (&va)[4], const float (&vb)[4]) {
#pragma unroll
        for (int i = 0; i < 4; ++i) As[buf][a_k + i][a_row] = va[i];
        *reinterpret_cast<float4 *>(&Bs[buf][b_k][b_col]) = make_float4(vb[0], vb[1], vb[2], vb[3]);
    };

    // each thread owns rows {ty*4..+3, 64+ty*4..+3} x cols {tx*4..+3, 64+tx*4..+3}
    const int ty = tid >> 4, tx = tid & 15;
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;

    if (klo < khi) {
        float va[4], vb[4];
        load_a(klo, va);
        load_b(klo, vb);
        store_tiles(0, va, vb);
        __syncthreads();
        int buf = 0;
        for (int k0 = klo; k0 < khi; k0 += BK) {
            const bool more = k0 + BK < khi;
            if (more) { load_a(k0 + BK, va); load_b(k0 + BK, vb); }
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
                store_tiles(buf ^ 1, va, vb);
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
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                v[j] = (c + j < n) ? finish_entry(acc[i][h * 4 + j], a.add, inst, r, c + j, n, a.pout) : 0.0f;
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
__global__ void __launch_bounds__(256)
elementwise_kernel(const float *__restrict__ src, long long src_stride, int src_mode, float *X, long long x_stride,
                   int rows, int cols, int out_prop, AddTerms add) {
    const long long inst = blockIdx.z;
    const long long total = (long long)rows * cols;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(e / cols), c = (int)(e % cols);
        float v;
        if (src_mode == 0) v = __ldg(src + inst * src_stride + e);
        else if (src_mode == 3) v = __ldg(src + inst * src_stride + (long long)c * rows + r);
        else if (src_mode == 1) v = (r == c) ? 1.0f : 0.0f;
        else v = X[inst * x_stride + e];
        X[inst * x_stride + e] = finish_entry(v, add, inst, r, c, cols, out_prop);
    }
}

}  // namespace

cudaError_t launch_product_ffma(const ProductArgs &a, int batch, cudaStream_t stream) {
    dim3 grid((a.n + BN - 1) / BN, (a.m + BM - 1) / BM, batch);
    product_ffma_kernel<<<grid, THREADS, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_elementwise(const float *src, long long src_stride, int src_mode, float *X, long long x_stride,
                               int rows, int cols, int out_prop, const AddTerms &add, int batch, cudaStream_t stream) {
    const long long total = (long long)rows * cols;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) blocks = 1;
    dim3 grid((unsigned)blocks, 1, batch);
    elementwise_kernel<<<grid, 256, 0, stream>>>(src, src_stride, src_mode, X, x_stride, rows, cols, out_prop, add);
    return cudaGetLastError();
}

}  // namespace mom
