// Device-side pieces shared by the product kernels: the structural k-range of an output tile, the
// structure mask of the result, and the fused Add epilogue.
#pragma once

#include <cstdint>
#include <utility>
#include <cuda_runtime.h>

#include "mom.h"

namespace mom {

// Programmatic dependent launch: a kernel that is launched with the programmatic-stream-serialization attribute may start
// while its predecessor in the stream is still running; it must not touch global memory before grid_dependency_wait(), which
// returns once the predecessor has completed and its writes are visible.  Such a kernel's lifetime overlaps its predecessors'
// writes, so it must not read anything they may have produced through the non-coherent path (ld.global.nc / __ldg promises data
// that is read-only for the kernel's whole lifetime): operands, Add terms and partial sums are read with ld.global.cg (__ldcg).  allow_dependents() lets the NEXT kernel of the stream
// start its own prologue (it becomes resident as resources free up and waits at its grid_dependency_wait()).  Both are no-ops
// in a kernel launched the ordinary way.
__device__ __forceinline__ void allow_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Launch with the attribute that allows the overlap described above (plus, optionally, a cluster dimension).
template <typename... KernelArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KernelArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, unsigned cluster,
                                    Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int n = 0;
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

constexpr int MAX_FUSED_ADD = 8;    // Add terms fused into one launch; more are added by follow-up passes

// Add terms of the equation (paper Table 1, "Add"), applied left to right in f32.
struct AddTerms {
    const float *ptr[MAX_FUSED_ADD];     // NULL for an Identity term
    long long stride[MAX_FUSED_ADD];     // elements between batch instances
    int count;
    unsigned transposed;                 // bit t: term t is stored transposed (cols x rows of X)
    unsigned aliases_out;                // bit t: term t is X itself (a later chain adding to it): read past L1, never
                                         // through the read-only path, and only by the thread that then writes the entry
    int rows;                            // rows of X (leading dimension of a transposed term)
};

// With dense zero-filled storage every product is C[r,c] = sum over l in [klo, khi) of A[r,l]*B[l,c],
// where the range for an output tile rows [r0,r1) x cols [c0,c1) is the intersection of the
// operands' structural ranges:
//   A lowerTri: l < r1      A upperTri: l >= r0      B lowerTri: l >= c0      B upperTri: l < c1
//   A Diagonal: r0 <= l < r1                         B Diagonal: c0 <= l < c1
// An empty range means the tile is structurally zero.
__host__ __device__ inline void tile_k_range(int pa, int pb, int r0, int r1, int c0, int c1, int k,
                                             int *klo, int *khi) {
    int lo = 0, hi = k;
    if ((pa == MOM_UPPER_TRI || pa == MOM_DIAGONAL) && r0 > lo) lo = r0;
    if ((pb == MOM_LOWER_TRI || pb == MOM_DIAGONAL) && c0 > lo) lo = c0;
    if ((pa == MOM_LOWER_TRI || pa == MOM_DIAGONAL) && r1 < hi) hi = r1;
    if ((pb == MOM_UPPER_TRI || pb == MOM_DIAGONAL) && c1 < hi) hi = c1;
    *klo = lo;
    *khi = hi;
}

__host__ __device__ inline bool in_structure(int prop, int r, int c) {
    return prop == MOM_GENERAL || prop == MOM_SYMMETRIC || (prop == MOM_LOWER_TRI && r >= c) || (prop == MOM_UPPER_TRI && r <= c) ||
           ((prop == MOM_IDENTITY || prop == MOM_DIAGONAL) && r == c);
}

// value of the equation at (r, c) given the chain's value `acc` there
__device__ __forceinline__ float finish_entry(float acc, const AddTerms &add, long long batch, int r, int c,
                                               int ld, int out_prop) {
    float v = acc;
#pragma unroll
    for (int t = 0; t < MAX_FUSED_ADD; ++t) {
        if (t < add.count) {
            const float *p = add.ptr[t];
            const long long at = (add.transposed >> t) & 1u ? (long long)c * add.rows + r : (long long)r * ld + c;
            if (!p) v += r == c ? 1.0f : 0.0f;
            else v += __ldcg(p + batch * add.stride[t] + at);
        }
    }
    return in_structure(out_prop, r, c) ? v : 0.0f;
}

// The same with a loop over the terms instead of unrolled code (for kernels whose epilogue runs once per
// thread and should stay small).
__device__ __forceinline__ float finish_entry_compact(float acc, const AddTerms &add, long long batch, int r, int c,
                                                       int ld, int out_prop) {
    float v = acc;
#pragma unroll 1
    for (int t = 0; t < add.count; ++t) {
        const float *p = add.ptr[t];
        if (!p) { v += r == c ? 1.0f : 0.0f; continue; }
        p += batch * add.stride[t] + ((add.transposed >> t) & 1u ? (long long)c * add.rows + r : (long long)r * ld + c);
        v += __ldcg(p);
    }
    return in_structure(out_prop, r, c) ? v : 0.0f;
}

// The same for four consecutive entries (r, c .. c+3) of a row, for the kernels that are bound by memory
// traffic: a compact loop over the terms (no unrolling: these kernels are tiny and must stay in the
// instruction cache), one 16-byte load per term where its layout allows.  `n` is the row length of X
// (entries at or beyond it are left alone), `vec` says that ld is a multiple of 4 (so that a term's
// row segment is 16-byte aligned whenever the term's base is).
__device__ __forceinline__ void finish_row4(float (&v)[4], const AddTerms &add, long long batch, int r, int c,
                                             int ld, int n, int out_prop, bool vec) {
#pragma unroll 1
    for (int t = 0; t < add.count; ++t) {
        const float *p = add.ptr[t];
        if (!p) {                                            // Identity term
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] += r == c + j ? 1.0f : 0.0f;
            continue;
        }
        p += batch * add.stride[t];
        const bool tr = (add.transposed >> t) & 1u;          // (a term that aliases the output is read like any other: every load here is coherent)
        if (!tr && vec && c + 3 < n && (reinterpret_cast<uintptr_t>(p) & 15) == 0) {
            const float4 *q = reinterpret_cast<const float4 *>(p + (long long)r * ld + c);
            const float4 x = __ldcg(q);
            v[0] += x.x; v[1] += x.y; v[2] += x.z; v[3] += x.w;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (c + j >= n) continue;
                const long long at = tr ? (long long)(c + j) * add.rows + r : (long long)r * ld + c + j;
                v[j] += __ldcg(p + at);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = in_structure(out_prop, r, c + j) ? v[j] : 0.0f;
}

}  // namespace mom
