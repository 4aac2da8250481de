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

// Default variant: where the one-launch tcgen05 kernel (product_tc_inline.cu) is the quickest of the three tensor-core kernels
// (back to back, us, warp-level / plane-fed / one-launch: 256^3 8.6 / 24.9 / 8.2, 448^3 14.5 / 30.9 / 8.8, 512^3 14.8 / 23.8 / 9.0,
// 768^3 31.1 / 30.0 / 14.6, 1024^3 65.2 / 31.3 / 22.0, 1280^3 115 / 48.4 / 41.0, 1536^3 - / 55.7 / 48.3, 2048^3 - / 95 / 116;
// 900 x 1200 x 100 16.6 / 27.1 / 10.9, 4096 x 256 x 64 10.4 / 22.7 / 7.6, 256 x 2048 x 64 10.5 / 23.7 / 10.7, 128 x 4096 x 128 14.8 / 26.8 / 15.5).
// Up to INLINE_SMALL_WORK it is taken whatever the shape; up to INLINE_MAX_WORK while its 128 x 128 tiles fit one wave of CTAs
// (a second wave repeats the whole of the first: 1792^3 93 us against 1536^3 48 us).
// Beyond that, up to INLINE_PAIR_MAX_WORK while its CTA pairs' 256 x 256 tiles fit one wave (1792^3 78.7 against the plane
// kernel's 81.3, 2048^3 84.5 against 92.7, 2048 x 512 x 2048 31.3 against 35.9; 2560^3, 100 pairs, 204 against 187).
constexpr double INLINE_MIN_WORK = 6.0e7, INLINE_SMALL_WORK = 1.0e9, INLINE_MAX_WORK = 4.0e9, INLINE_PAIR_MAX_WORK = 1.0e10,
                 INLINE_MIN_OUTPUT = 65536.0;
constexpr int64_t INLINE_WAVE_TILES = 148, INLINE_WAVE_PAIRS = 74;
// Products below this many multiplications count as small when independent subtrees are put side by side on two streams.
constexpr double SIDE_BY_SIDE_MAX_WORK = 1.0e9;

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
    // storage layer (mom_equation_plan_stored): per caller pointer / Add term / for X; empty vectors: all dense
    std::vector<int32_t> ptr_storage, add_storage;
    int32_t result_storage = 0;
    std::vector<char> slot_native;             // packed slot that every reader addresses in place (no dense copy needed)
    bool result_native = false;                // packed X written in place by the product that writes X
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
    // Two independent subtrees of the parenthesization, both made of small products, run side by side: steps
    // [side_begin, side_end) -- the right subtree of step `side_join` -- go to a second stream the plan owns while the left
    // subtree runs on the caller's stream; side_join waits for both.  side_join < 0: everything runs in order.
    int side_begin = 0, side_end = 0, side_join = -1;
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

// ---- storage layer (packed triangles) ----------------------------------------------------------------------
inline bool is_lower_kind(int32_t p) { return kernel_property(p) == MOM_LOWER_TRI; }
inline bool is_triangular_kind(int32_t p) { return kernel_property(p) == MOM_LOWER_TRI || kernel_property(p) == MOM_UPPER_TRI; }

// f32 entries a matrix occupies as stored
inline int64_t stored_elements(const mom_matrix_desc_t &d, int32_t storage) {
    if (storage != MOM_STORAGE_PACKED) return d.rows * d.cols;
    const int64_t n = d.rows, q = n >> 2, rest = n - 4 * q, n4 = (n + 3) & ~(int64_t)3;
    return is_lower_kind(d.property) ? 8 * q * (q + 1) + rest * 4 * (q + 1) : n * n4 - 8 * q * (q - 1) - 4 * q * rest;
}
inline int32_t slot_storage(const mom_plan &p, int slot) { return p.ptr_storage.empty() ? 0 : p.ptr_storage[slot]; }
inline int32_t term_storage(const mom_plan &p, int term) { return p.add_storage.empty() ? 0 : p.add_storage[term]; }

// Shape test of the batched-chain kernel (batched_chain.cu): a right-nested chain M_S * (... (M_1 * B)) of stored,
// untransposed factors with whole 16-row blocks of at most 64 rows, a right end of 8 or 16 columns, Add terms not
// transposed.  (Whether a call takes that kernel also depends on its batch size.)
constexpr int64_t BATCHED_CHAIN_MIN_BATCH = 256;
inline bool batched_chain_shape(const mom_plan &p) {
    const int S = (int)p.steps.size(), n_chain = (int)p.chain.size();
    if (!p.fused_ok || p.variant == MOM_VARIANT_FFMA || p.sums.size() != 1 || S < 1 || S > 4 || p.add.size() > 8) return false;
    for (const Summand &sm : p.sums[0].summands)
        if (sm.kind != SUM_STEP && sm.kind != SUM_TERM) return false;
    for (char t : p.add_t)
        if (t) return false;
    const int64_t n = p.steps[0].pub.n;
    if ((n != 8 && n != 16) || !p.steps[S - 1].is_last) return false;
    for (int s = 0; s < S; ++s) {
        const mom_step_t &st = p.steps[s].pub;
        if (st.kind == MOM_KIND_SCALE || st.kind == MOM_KIND_GRAM || p.steps[s].folded || p.steps[s].accumulate) return false;
        if (st.lhs < 0 || st.lhs >= n_chain || st.lhs_transposed || p.chain_t[st.lhs] || p.factor_ptr[st.lhs] < 0) return false;
        if (s == 0 ? (st.rhs < 0 || st.rhs >= n_chain || st.rhs_transposed || p.chain_t[st.rhs] || p.factor_ptr[st.rhs] < 0)
                   : st.rhs != p.steps[s - 1].pub.out) return false;
        if (st.m % 16 || st.m > 64 || st.k % 16 || st.k > 64 || st.n != n) return false;
        const int pa = kernel_property(st.lhs_property), pb = kernel_property(st.rhs_property);
        if (pa == MOM_DIAGONAL || pa == MOM_IDENTITY || pb == MOM_DIAGONAL || pb == MOM_IDENTITY) return false;
    }
    return true;
}

// A packed operand that every kernel of a call with `batch` instances reads in place (no dense copy): what the plan
// marked (operands of tcgen05 steps), or a left factor of the batched-chain kernel when the call qualifies for it.
inline bool storage_in_place(const mom_plan &p, int slot, int64_t batch) {
    if (slot_storage(p, slot) != MOM_STORAGE_PACKED || !p.slot_used[slot]) return false;
    if (p.slot_native[slot]) return true;
    if (batch < BATCHED_CHAIN_MIN_BATCH || p.result_storage != MOM_STORAGE_DENSE || !batched_chain_shape(p)) return false;
    for (size_t i = 0; i < p.add.size(); ++i)
        if (term_storage(p, (int)i) != MOM_STORAGE_DENSE) return false;
    return slot != p.factor_ptr[p.steps[0].pub.rhs];         // the right end is read dense
}

// elements between the instances of a dense copy the storage layer makes (a multiple of 4: rows stay 16-byte addressable)
inline int64_t dense_copy_stride(const mom_matrix_desc_t &d) { return (d.rows * d.cols + 3) & ~(int64_t)3; }

// Room behind the plan's own workspace for the storage layer: a dense copy of every packed operand that some kernel
// cannot read in place, of every packed Add term, and a dense X when the packed X is not written in place.  Offsets
// are in bytes from the start of that region (SIZE_MAX: none); returns the region's size.
struct StorageLayout {
    std::vector<size_t> slot_off, add_off;
    size_t x_off = SIZE_MAX;
    size_t bytes = 0;
};
inline StorageLayout storage_layout(const mom_plan &p, int64_t batch) {
    StorageLayout l;
    l.slot_off.assign(p.ptr_desc.size(), SIZE_MAX);
    l.add_off.assign(p.add.size(), SIZE_MAX);
    auto take = [&](const mom_matrix_desc_t &d) {
        const size_t at = l.bytes;
        l.bytes += align_up((size_t)dense_copy_stride(d) * sizeof(float) * (size_t)batch, WS_ALIGN);
        return at;
    };
    for (size_t i = 0; i < p.ptr_desc.size(); ++i)
        if (slot_storage(p, (int)i) == MOM_STORAGE_PACKED && p.slot_used[i] && !storage_in_place(p, (int)i, batch)) l.slot_off[i] = take(p.ptr_desc[i]);
    for (size_t i = 0; i < p.add.size(); ++i)
        if (term_storage(p, (int)i) == MOM_STORAGE_PACKED) l.add_off[i] = take(p.add[i]);
    if (p.result_storage == MOM_STORAGE_PACKED && !p.result_native) l.x_off = take(p.result_desc);
    return l;
}

// defined in execute.cu; releases device-side state of a plan (no-op when none exists)
void destroy_device_state(DeviceState *);
}  // namespace mom
