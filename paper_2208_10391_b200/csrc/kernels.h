// Launch interfaces of the CUDA kernels (internal).
#pragma once

#include <cuda_runtime.h>

#include "device_common.cuh"

namespace mom {

// One binary product C(m x n) = A(m x k) * B(k x n) (+ Add terms), dense row-major f32.
struct ProductArgs {
    const float *A;
    const float *B;
    float *C;
    int m, n, k;
    int pa, pb, pout;                       // mom_property_t of A, B (as used) and of what is written to C
    int transA, transB;                     // the operand is stored transposed (k x m resp. n x k)
    long long strideA, strideB, strideC;    // elements between batch instances
    AddTerms add;
    // tensor-core path only: the operand is d * A (rows of A as used scaled, scale_rows != 0) or A * d (columns);
    // d points at a dense Diagonal matrix whose entries are scale_step floats apart; NULL: no scaling
    const float *scaleA, *scaleB;
    long long scaleA_step, scaleB_step;
    int scaleA_rows, scaleB_rows;
    // tensor-core path only: the operand (as stored) / the result is a packed triangle read / written in place
    int packedA, packedB, packedC;
};

cudaError_t launch_product_ffma(const ProductArgs &a, int batch, cudaStream_t stream);

// The same product on the warp-level tensor-core kernel (mma.sync, 3xTF32 split in registers): one launch,
// operands read as stored, contraction split over a thread-block cluster when the output has few tiles.
cudaError_t launch_product_mma(const ProductArgs &a, int batch, cudaStream_t stream);

// The same product when A or B is Diagonal: a row or column scaling of the other operand (one pass).
cudaError_t launch_scale(const ProductArgs &a, int batch, cudaStream_t stream);

// src_mode: 0 pointer, 1 Identity, 2 X itself (in place), 3 pointer to the transposed matrix (cols x rows)
cudaError_t launch_elementwise(const float *src, long long src_stride, int src_mode, float *X, long long x_stride,
                               int rows, int cols, int out_prop, const AddTerms &add, int batch, cudaStream_t stream);

// Packed triangle -> dense n x n matrix (zeros outside the container) and back, `batch` instances.
cudaError_t launch_unpack(const float *src, long long src_stride, float *dst, long long dst_stride, int n, bool lower, int batch,
                          cudaStream_t stream);
cudaError_t launch_pack(const float *src, long long src_stride, float *dst, long long dst_stride, int n, bool lower, int batch,
                        cudaStream_t stream);

}  // namespace mom
