// Fused small-equation kernel: launch interface (internal).
#pragma once

#include <cuda_runtime.h>

#include <vector>

#include "device_common.cuh"

namespace mom {

constexpr int FUSED_MAX_OPERANDS = 8;
constexpr int FUSED_MAX_STEPS = 7;
constexpr size_t FUSED_MAX_SMEM = 100 * 1024;   // per instance: keeps at least two CTAs on an SM

struct FusedOperand {
    const float *ptr;
    long long stride;        // elements between instances
    int rows, cols, prop;
    int smem_off;            // floats
    int ld;                  // leading dimension in shared memory (floats)
    int transposed;          // stored as cols x rows; read transposed into shared memory
    int tab_begin, tab_end;  // rows of the copy table that fetch this operand; empty: the generic loader does it
};

struct FusedStep {
    int a_off, b_off;        // shared-memory offsets (floats) of the operands
    int out_off;             // shared-memory offset of the intermediate, or -1: last step, writes X
    int m, n, k;
    int pa, pb, pout;
    int lda, ldb, ldc;       // shared-memory leading dimensions (ldc unused on the last step)
};

struct FusedPlan {
    int n_ops, n_steps;
    FusedOperand ops[FUSED_MAX_OPERANDS];
    FusedStep steps[FUSED_MAX_STEPS];
    AddTerms add;
    float *out;
    long long out_stride;
    long long batch;
    int use_mma;             // 1: tensor-core mma.sync with the 3xTF32 split, 0: plain FMA
    const uint2 *copy_table; // device: FUSED_THREADS entries per row, see fused_copy_table()
};

constexpr int FUSED_THREADS = 256;
constexpr uint32_t FUSED_COPY_NONE = 0xFFFFFFFFu;

// Copy table of an operand that is read as stored with rows of whole 16-byte pieces: where every 16-byte
// piece of one instance goes, worked out once on the host so that the kernel (bound by instruction issue)
// spends a load and an add per copy instead of index arithmetic.  Entry (row, thread): x = byte offset in
// shared memory | 1 if the piece meets the operand's structure (else it is zero-filled without a read),
// y = offset in floats from the instance's first element; x = FUSED_COPY_NONE: nothing to do.  Pieces that no
// product can read (beyond the 16-column block of a triangular row's diagonal) get no entry.
// Appends whole rows to `table` and returns the number of rows appended.
int fused_copy_table(int rows, int cols, int prop, int smem_off, int ld, std::vector<uint2> &table);

// Leading dimension (floats) of a matrix with `cols` columns held in shared memory.  A value is read
// by exactly one product, as its left or its right operand; the padding makes that product's
// fragment loads bank-conflict free: rows 4 (mod 8) words apart for a left operand (thread (g, t)
// reads row g, column t), 8 (mod 16) apart for a right operand (reads row t, column g).
__host__ __device__ inline int fused_ld(int cols, bool is_rhs) {
    int ld = (cols + 3) & ~3;
    if (is_rhs) { while (ld % 16 != 8) ld += 4; }
    else { while (ld % 8 != 4) ld += 4; }
    return ld;
}

cudaError_t launch_fused_small(const FusedPlan &fp, size_t smem_bytes, cudaStream_t stream);

}  // namespace mom
