// Internal structures shared by the host planner and the launcher.  Not part of the public ABI.
#pragma once

#include <cstddef>
#include <cstdint>
#include <mutex>
#include <string>
#include <vector>

#include "mom.h"

namespace mom {

// Tile shapes of the tensor-core product kernel (see product_tc.cu).
constexpr int TC_BM = 128;          // output rows per tile   (MMA M)
constexpr int TC_BN = 256;          // output cols per tile   (MMA N)
constexpr int TC_BK = 32;           // f32 elements per k-block = one 128-byte swizzle row
// The operand-split pre-pass works on square blocks of this edge and skips blocks that lie wholly
// outside a triangular operand's structure.  It must be a multiple of both TC_BM and TC_BN so that
// every block a product tile can touch has been written.
constexpr int SPLIT_BLOCK = 256;

// Tile shape of the FFMA product kernel (see product_ffma.cu).
constexpr int FF_BM = 128;
constexpr int FF_BN = 128;

constexpr size_t WS_ALIGN = 256;

// Largest rows / cols a descriptor may have: every kernel indexes rows, columns and k with 32-bit integers.
constexpr int64_t MAX_DIMENSION = 2147483647 - 1024;
// Largest m (and n) of a product on the tcgen05 kernel: a tile-table entry keeps the tile's first row in 24 bits
// and a padding entry sits at row 2^24 - 256, which must lie outside every matrix.
constexpr int64_t TC_MAX_ROWS = (1 << 24) - 1024;

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Type of A^T: lower and upper swap (the inference rule of the paper's Section 2), the kind of diagonal stays.
inline int32_t transpose_property(int32_t p) {
    switch (p) {
        case MOM_LOWER_TRI: return MOM_UPPER_TRI;
        case MOM_UPPER_TRI: return MOM_LOWER_TRI;
        case MOM_STRICT_LOWER: return MOM_STRICT_UPPER;
        case MOM_STRICT_UPPER: return MOM_STRICT_LOWER;
        case MOM_UNIT_LOWER: return MOM_UNIT_UPPER;
        case MOM_UNIT_UPPER: return MOM_UNIT_LOWER;
        default: return p;
    }
}

// The structure the kernels work with: a strict or unit triangle is handled as the ordinary triangle around it
// (its diagonal holds stored zeros or ones; products with them give exact zeros and ones).
inline int32_t kernel_property(int32_t p) {
    if (p == MOM_STRICT_LOWER || p == MOM_UNIT_LOWER) return MOM_LOWER_TRI;
    if (p == MOM_STRICT_UPPER || p == MOM_UNIT_UPPER) return MOM_UPPER_TRI;
    return p;
}

struct StepImpl {
    mom_step_t pub;
    bool is_last = false;           // root of its chain's tree: writes X (the first root also carries the Add terms)
    bool accumulate = false;        // a later chain's root: adds its product to what the sum's buffer already holds
    int sum = -1;                   // roots: index of the sum (mom_plan::sums) whose value they write
    // workspace byte offsets (per instance); SIZE_MAX = not used
    size_t out_off = SIZE_MAX;      // f32 intermediate written by this step (not for the last step)
    size_t a_hi_off = SIZE_MAX, a_lo_off = SIZE_MAX;   // split planes of the operands (tensor-core steps)
    size_t b_hi_off = SIZE_MAX, b_lo_off = SIZE_MAX;
    // When this tensor-core step feeds another tensor-core step, its epilogue writes the consumer's hi/lo
    // planes directly (transposed if the consumer takes it as right operand) and no f32 intermediate exists.
    int planes_out = 0;             // 0: f32 output; 1: planes as stored (consumer's left operand); 2: transposed planes
    size_t planes_hi_off = SIZE_MAX, planes_lo_off = SIZE_MAX;
    bool a_planes_ready = false, b_planes_ready = false;   // this step's operand planes come from the producing step
    // Split-K: products with few output tiles and a long contraction run `split_k` k-slices per tile on
    // different CTAs; the slices' partial sums go to scratch and a small kernel adds them up.
    int split_k = 1;
    size_t partial_off = SIZE_MAX;
    // A scaling step (Diagonal factor) whose only reader is a tensor-core step is folded into that step's
    // operand-split pass: it launches nothing and has no buffer; the reader splits d * S instead of S.
    bool mirror = false;            // Gram product on the tensor-core kernel: lower tiles computed, upper ones mirrored
    bool folded = false;
    int fold_into = -1;             // folded step: the tensor-core step that reads it
    int fold_a = -1, fold_b = -1;   // tensor-core step: the folded scaling step behind its left / right operand
};

// One summand of X = sum of chain values + Add terms, in the order written.
enum SummandKind { SUM_STEP = 0, SUM_FACTOR = 1, SUM_TERM = 2, SUM_IDENTITY = 3 };
struct Summand {
    int kind;       // SUM_STEP: a chain with products (index = its root step); SUM_FACTOR: a chain that reduced to
    int index;      // one factor (index = factor id); SUM_TERM: Add term `index`; SUM_IDENTITY: a chain equal to I
};

// One sum of chains.  The last sum of a plan is the equation's value X; earlier ones are nested sums of an
// expression (a sum inside a product), evaluated into a workspace temporary that is then a factor of a later chain.
struct SumInfo {
    std::vector<Summand> summands;          // what is added up, in the order written
    int step_begin = 0, step_end = 0;       // the products emitted for this sum
    mom_matrix_desc_t desc{};               // type of the value
    size_t out_off = SIZE_MAX;              // workspace byte offset of the temporary (per instance); SIZE_MAX: X
};

struct DeviceState;   // launcher-owned, created on first execute (execute.cu)

}  // namespace mom

struct mom_plan {
    int32_t variant = 0;
    std::vector<mom_matrix_desc_t> chain;      // every factor of every chain as the equation uses it (transposed type where flagged)
    std::vector<int32_t> factor_ptr;           // per factor: index into the caller's pointer array; -1 for a temporary
    std::vector<int32_t> factor_sum;           // per factor: the nested sum whose temporary it is; -1 for a stored matrix
    std::vector<mom_matrix_desc_t> ptr_desc;   // per entry of the caller's pointer array: the matrix as stored
    std::vector<char> slot_used;               // per entry: some factor refers to it (an unused operand may be NULL)
    std::vector<mom_matrix_desc_t> add;
    std::vector<char> chain_t, add_t;          // operand enters transposed: stored shape is (cols x rows) of the entry above
    std::vector<int32_t> chain_begin;          // factors of chain c are [chain_begin[c], chain_begin[c + 1])
    std::vector<int32_t> names;                // per pointer entry: equal names = the same stored matrix (empty: all distinct)
    std::vector<int32_t> kept;                 // factor indices surviving identity simplification
    std::vector<mom::SumInfo> sums;            // nested sums first, X last
    int32_t temporaries = 0;                   // nested sums that are materialized
    int32_t reused = 0;                        // products not emitted because an earlier chain computed them
    std::string paren;
    uint64_t mults = 0;                        // useful multiplications of the chosen tree
    uint64_t add_flops = 0;
    std::vector<mom::StepImpl> steps;
    mom_matrix_desc_t product_desc{};          // chain value before the Add terms
    mom_matrix_desc_t result_desc{};
    size_t workspace_per_instance = 0;
    // fused small-equation kernel: whole plan in shared memory, one instance per CTA (no workspace)
    bool fused_ok = false;
    size_t fused_smem_bytes = 0;
    std::vector<int> fused_value_off;          // shared-memory offset (floats) per value id; -1 = not resident
    std::vector<int> fused_value_ld;           // shared-memory leading dimension (floats) per value id
    // launcher state: created at the first execute on a device, rebuilt when the plan moves to another device;
    // `exec_mutex` serialises the host side of execute calls on one plan (enqueueing only: the kernels of two
    // calls on different streams still overlap on the GPU)
    mutable std::mutex exec_mutex;
    mutable mom::DeviceState *dev = nullptr;
    mutable int32_t last_launches = 0;
    bool step_timing = false;
};

namespace mom {
// defined in execute.cu; releases device-side state of a plan (no-op when none exists)
void destroy_device_state(DeviceState *);
}  // namespace mom
