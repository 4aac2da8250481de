// Batched right-nested chains with a narrow right end, X_i = M_S * ( ... (M_2 * (M_1 * B_i)) ... ) + terms,
// for thousands of independent instances: launch interface (internal).  See batched_chain.cu.
#pragma once

#include <cuda_runtime.h>

#include "device_common.cuh"

namespace mom {

constexpr int BC_MAX_STEPS = 4;
constexpr int BC_MAX_DIM = 64;       // rows and contraction length of every product
constexpr int BC_MAX_N = 16;         // columns of the right end (and of every intermediate and of X)

struct BatchedChainStep {
    const float *lhs;                // the left factor of this product, m x k, row-major as stored (one instance)
    long long lhs_stride;            // elements between instances
    int m, k;
    int packed;                      // 0: dense; 1 / 2: a packed lower / upper triangle (m == k) read in place
    // work split of the step's 16-row blocks over the two warps of an instance: warp w handles row blocks
    // rb[w][0] and rb[w][1] (-1: none); chunks[w][q] has bit c set when that row block needs columns
    // [16 c, 16 c + 16) of the left factor (blocks wholly outside a triangular factor's structure are skipped)
    signed char rb[2][2];
    unsigned char chunks[2][2];
};

struct BatchedChainPlan {
    int n_steps;
    BatchedChainStep steps[BC_MAX_STEPS];    // innermost product first
    const float *rhs;                // the right end B, k_0 x n, row-major
    long long rhs_stride;
    int n;                           // 8 or 16
    AddTerms add;                    // none of them transposed
    float *out;
    long long out_stride;
    int pout;                        // structure of X (entries outside it are written as +0.0f)
    long long batch;
};

// Splits the row blocks of a product with `row_blocks` blocks of 16 rows over two warps so that both get about
// the same number of 16 x 16 blocks to multiply; needed[rb] is the chunk mask of row block rb.
void batched_chain_assign(const unsigned char *needed, int row_blocks, BatchedChainStep *step);

cudaError_t launch_batched_chain(const BatchedChainPlan &bp, cudaStream_t stream);

}  // namespace mom
