// Host planner: identity simplification, property-aware matrix-chain dynamic program, property
// propagation, step emission and workspace layout (paper Section 2, "Transformations").
// Pure host code: no CUDA call is made here.
#include <algorithm>
#include <cstring>
#include <map>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include "fused_small.h"
#include "mom_internal.h"
#include "product_tc.h"

namespace {

using u128 = unsigned __int128;
constexpr uint64_t COST_LIMIT = (uint64_t)1 << 63;

bool is_lower(int32_t p) { return p == MOM_LOWER_TRI || p == MOM_STRICT_LOWER || p == MOM_UNIT_LOWER; }
bool is_upper(int32_t p) { return p == MOM_UPPER_TRI || p == MOM_STRICT_UPPER || p == MOM_UNIT_UPPER; }
bool is_tri(int32_t p) { return is_lower(p) || is_upper(p); }

// What a type states about its diagonal.
enum Diag { DIAG_DATA = 0, DIAG_ZERO = 1, DIAG_ONE = 2 };
Diag diag_of(int32_t p) {
    if (p == MOM_STRICT_LOWER || p == MOM_STRICT_UPPER) return DIAG_ZERO;
    if (p == MOM_UNIT_LOWER || p == MOM_UNIT_UPPER || p == MOM_IDENTITY) return DIAG_ONE;
    return DIAG_DATA;
}
int32_t triangle(bool lower, Diag d) {
    if (d == DIAG_ZERO) return lower ? MOM_STRICT_LOWER : MOM_STRICT_UPPER;
    if (d == DIAG_ONE) return lower ? MOM_UNIT_LOWER : MOM_UNIT_UPPER;
    return lower ? MOM_LOWER_TRI : MOM_UPPER_TRI;
}

// Least upper bound in  Identity < Diagonal < {lowerTri, upperTri} < general  (paper Listing 3 types L*L as lowerTri).
// Inside one orientation the product's diagonal is the entrywise product of the factors' diagonals.
int32_t join_property(int32_t p, int32_t q) {
    if (p == MOM_IDENTITY) return q;
    if (q == MOM_IDENTITY) return p;
    if (p == MOM_SYMMETRIC || q == MOM_SYMMETRIC) return (int32_t)MOM_GENERAL;   // S*S, D*S, ... are not symmetric in general
    if (p == MOM_GENERAL || q == MOM_GENERAL) return (int32_t)MOM_GENERAL;
    if (p == MOM_DIAGONAL && q == MOM_DIAGONAL) return (int32_t)MOM_DIAGONAL;
    const bool lower = is_lower(p) || is_lower(q), upper = is_upper(p) || is_upper(q);
    if (lower && upper) return (int32_t)MOM_GENERAL;
    const Diag dp = diag_of(p), dq = diag_of(q);
    return triangle(lower, dp == DIAG_ZERO || dq == DIAG_ZERO ? DIAG_ZERO : dp == DIAG_ONE && dq == DIAG_ONE ? DIAG_ONE : DIAG_DATA);
}

// structural non-zeros of an r x c matrix with property p (every property but general is square)
unsigned __int128 structural_entries(int32_t p, int64_t r, int64_t c) {
    const unsigned __int128 R = (unsigned __int128)r, C = (unsigned __int128)c;
    if (p == MOM_GENERAL || p == MOM_SYMMETRIC) return R * C;
    if (diag_of(p) == DIAG_ZERO) return R * (R - 1) / 2;
    if (is_tri(p)) return R * (R + 1) / 2;
    return R;
}

// of those, the entries that are not known to be 1 (the ones a multiplication needs)
unsigned __int128 multiplying_entries(int32_t p, int64_t r, int64_t c) {
    if (p == MOM_IDENTITY) return 0;
    if (p == MOM_UNIT_LOWER || p == MOM_UNIT_UPPER) return (unsigned __int128)r * (unsigned __int128)(r - 1) / 2;
    return structural_entries(p, r, c);
}

// Multiplications of the lower triangle (i >= j) of Y * Y^T, Y m x k: k m(m+1)/2 for a full Y, n(n+1)(n+2)/6 for a
// triangular one.  Returns false on overflow.
bool gram_mults(int32_t py, int64_t m, int64_t k, uint64_t *out);

// Scalar multiplications a_il * b_lj of an (m x k)(k x n) product in which both factors are structurally
// non-zero and neither is known to be 1.  Triangular operands are square.  Returns false on overflow.
bool useful_mults(int32_t pa, int32_t pb, int64_t m, int64_t k, int64_t n, uint64_t *out) {
    u128 v;
    const u128 M = (u128)m, K = (u128)k, N = (u128)n;
    // a strict or unit triangle takes part with the entries off its diagonal only: e of its K diagonal entries drop out
    const u128 ea = pa == MOM_LOWER_TRI || pa == MOM_UPPER_TRI ? 0 : 1, eb = pb == MOM_LOWER_TRI || pb == MOM_UPPER_TRI ? 0 : 1;
    if (pa == MOM_DIAGONAL) {
        v = multiplying_entries(pb, k, n);         // D*B scales the rows of B: one multiplication per entry of B
    } else if (pb == MOM_DIAGONAL) {
        v = multiplying_entries(pa, m, k);         // A*D scales the columns of A
    } else if (!is_tri(pa) && !is_tri(pb)) {
        v = M * K * N;
    } else if (is_tri(pa) && !is_tri(pb)) {
        v = N * (K * (K + 1) / 2 - ea * K);        // row i of A has i+1 (or k-i) non-zeros, one fewer without the diagonal
    } else if (!is_tri(pa) && is_tri(pb)) {
        v = M * (K * (K + 1) / 2 - eb * K);
    } else if (is_lower(pa) == is_lower(pb)) {
        // sum_l (k - l - ea)(l + 1 - eb), l = 0..k-1; with ea = eb = 0 this is k(k+1)(k+2)/6
        const u128 s1 = K * (K - 1) / 2, s2 = (K - 1) * K * (2 * K - 1) / 6;        // sum of l and of l^2
        // (K - ea)(1 - eb) K + ((K - ea) - (1 - eb)) s1 - s2
        const u128 c0 = K - ea, c1 = 1 - eb;
        v = c0 * c1 * K + c0 * s1 - s2 - c1 * s1;
    } else {
        // sum_t (t - ea)(t - eb), t = 1..k; with ea = eb = 0 the sum of squares k(k+1)(2k+1)/6
        v = K * (K + 1) * (2 * K + 1) / 6 + ea * eb * K - (ea + eb) * (K * (K + 1) / 2);
    }
    if (v >= (u128)COST_LIMIT) return false;
    *out = (uint64_t)v;
    return true;
}

bool gram_mults(int32_t py, int64_t m, int64_t k, uint64_t *out) {
    const u128 M = (u128)m, K = (u128)k;
    // triangular Y: triples i >= j >= l (lower) of a shared column l; without the diagonal i >= j > l
    const u128 v = !is_tri(py) ? K * (M * (M + 1) / 2)
                   : py == MOM_LOWER_TRI || py == MOM_UPPER_TRI ? M * (M + 1) * (M + 2) / 6 : (M + 1) * M * (M - 1) / 6;
    if (v >= (u128)COST_LIMIT) return false;
    *out = (uint64_t)v;
    return true;
}

mom_status_t check_desc(const mom_matrix_desc_t &d) {
    if (d.rows < 1 || d.cols < 1) return MOM_ERR_INVALID_ARG;
    if (d.property < MOM_GENERAL || d.property > MOM_UNIT_UPPER) return MOM_ERR_INVALID_ARG;
    if (d.dtype != MOM_F32) return MOM_ERR_DTYPE;
    if (d.property != MOM_GENERAL && d.rows != d.cols) return MOM_ERR_PROPERTY;
    if (d.rows > mom::MAX_DIMENSION || d.cols > mom::MAX_DIMENSION) return MOM_ERR_LIMIT;   // the kernels index with 32-bit integers
    return MOM_OK;
}

uint64_t nnz(const mom_matrix_desc_t &d) { return (uint64_t)structural_entries(d.property, d.rows, d.cols); }

// Property of a sum of summands (chain values and Add terms).  A sum of two or more is never Identity: an
// Identity summand contributes its diagonal footprint and is joined as a Diagonal matrix.
int32_t sum_property(const std::vector<int32_t> &props) {
    if (props.size() == 1) return props[0];
    bool any_symmetric = false, only_symmetric_like = true;      // Symmetric + (Symmetric | Diagonal | Identity) is Symmetric
    for (int32_t p : props) {
        any_symmetric |= p == MOM_SYMMETRIC;
        only_symmetric_like &= p == MOM_SYMMETRIC || p == MOM_DIAGONAL || p == MOM_IDENTITY;
    }
    if (any_symmetric) return only_symmetric_like ? (int32_t)MOM_SYMMETRIC : (int32_t)MOM_GENERAL;
    bool lower = false, upper = false;
    Diag d = DIAG_ZERO;                             // the diagonals add up: 0 + x = x, anything else is data
    for (int32_t p : props) {
        if (p == MOM_GENERAL) return (int32_t)MOM_GENERAL;
        lower |= is_lower(p);
        upper |= is_upper(p);
        const Diag dp = diag_of(p);
        d = d == DIAG_ZERO ? dp : dp == DIAG_ZERO ? d : DIAG_DATA;
    }
    if (lower && upper) return (int32_t)MOM_GENERAL;
    if (!lower && !upper) return (int32_t)MOM_DIAGONAL;
    return triangle(lower, d);
}

struct Node { int64_t rows, cols; int32_t prop; };

struct Interval { size_t bytes; int first, last; size_t *slot; size_t off; };

// First-fit offsets such that buffers whose live ranges [first, last] intersect never overlap.
size_t pack(std::vector<Interval> &items) {
    size_t total = 0;
    std::vector<Interval *> placed;
    std::vector<Interval *> order;
    for (auto &it : items) order.push_back(&it);
    std::stable_sort(order.begin(), order.end(), [](Interval *a, Interval *b) { return a->bytes > b->bytes; });
    for (Interval *it : order) {
        size_t off = 0;
        bool moved = true;
        while (moved) {
            moved = false;
            for (Interval *p : placed) {
                const bool live = !(p->last < it->first || it->last < p->first);
                const bool overlap = off < p->off + p->bytes && p->off < off + it->bytes;
                if (live && overlap) { off = mom::align_up(p->off + p->bytes, mom::WS_ALIGN); moved = true; }
            }
        }
        it->off = off;
        *it->slot = off;
        placed.push_back(it);
        total = std::max(total, off + it->bytes);
    }
    return mom::align_up(total, mom::WS_ALIGN);
}

}  // namespace

extern "C" {

mom_status_t mom_matrix_desc(int64_t rows, int64_t cols, mom_property_t property, mom_dtype_t dtype,
                             mom_matrix_desc_t *out) {
    if (!out) return MOM_ERR_INVALID_ARG;
    mom_matrix_desc_t d{rows, cols, (int32_t)property, (int32_t)dtype};
    mom_status_t st = check_desc(d);
    if (st != MOM_OK) return st;
    *out = d;
    return MOM_OK;
}

mom_status_t mom_column_slab(int64_t cols, int32_t rank, int32_t world, int64_t multiple, int64_t *begin, int64_t *end) {
    if (!begin || !end || cols < 1 || world < 1 || rank < 0 || rank >= world || multiple < 1) return MOM_ERR_INVALID_ARG;
    const unsigned __int128 units = ((unsigned __int128)cols + (unsigned __int128)multiple - 1) / (unsigned __int128)multiple;
    const unsigned __int128 u0 = units * (unsigned __int128)rank / (unsigned __int128)world;
    const unsigned __int128 u1 = units * (unsigned __int128)(rank + 1) / (unsigned __int128)world;
    const unsigned __int128 b = u0 * (unsigned __int128)multiple, e = u1 * (unsigned __int128)multiple;
    *begin = (int64_t)std::min<unsigned __int128>(b, (unsigned __int128)cols);
    *end = (int64_t)std::min<unsigned __int128>(e, (unsigned __int128)cols);
    return MOM_OK;
}

mom_status_t mom_column_slab_desc(const mom_matrix_desc_t *stored, int32_t transposed, int64_t begin, int64_t end,
                                  mom_matrix_desc_t *slab) {
    if (!stored || !slab) return MOM_ERR_INVALID_ARG;
    mom_status_t st = check_desc(*stored);
    if (st != MOM_OK) return st;
    const int64_t used_cols = transposed ? stored->rows : stored->cols;
    if (begin < 0 || end <= begin || end > used_cols) return MOM_ERR_INVALID_ARG;
    if (begin == 0 && end == used_cols) { *slab = *stored; return MOM_OK; }
    *slab = transposed ? mom_matrix_desc_t{end - begin, stored->cols, MOM_GENERAL, stored->dtype}
                       : mom_matrix_desc_t{stored->rows, end - begin, MOM_GENERAL, stored->dtype};
    return MOM_OK;
}

// What the planning entry points hand to the shared planner: sums of chains in dependency order (a nested sum
// before the sum that uses it; the last one is X).  A factor is a stored matrix (an entry of the caller's pointer
// array, possibly transposed) or the temporary of an earlier sum.
struct FactorIn {
    int32_t ptr;        // entry of the pointer array, or -1
    int32_t sub;        // earlier sum, or -1
    bool t;             // enters transposed (stored matrices only)
    int64_t name;       // equal names = the same value; -1: nothing known
    std::string label;  // how a stored matrix prints in the parenthesization string
};
struct SumIn { std::vector<std::vector<FactorIn>> chains; };

static mom_status_t plan_sums(const std::vector<mom_matrix_desc_t> &slots, const std::vector<SumIn> &sums_in,
                              const int32_t *slot_names, const mom_matrix_desc_t *stored_add,
                              const int32_t *add_transposed, int32_t n_add, mom_variant_t variant, mom_plan_t **out_plan,
                              bool packed_storage = false) {
    if (!out_plan || sums_in.empty() || n_add < 0 || (n_add > 0 && !stored_add)) return MOM_ERR_INVALID_ARG;
    if ((int)variant < 0 || (int)variant > 4) return MOM_ERR_INVALID_ARG;
    int64_t total = 0;
    int n_chains = 0;
    for (const SumIn &si : sums_in) {
        if (si.chains.empty()) return MOM_ERR_INVALID_ARG;
        for (const auto &c : si.chains) {
            if (c.empty()) return MOM_ERR_INVALID_ARG;
            total += (int64_t)c.size();
            ++n_chains;
            if (total > (1 << 20)) return MOM_ERR_INVALID_ARG;
        }
    }
    const int n_chain = (int)total;                         // factors over all chains of all sums
    for (const auto &d : slots) {
        mom_status_t st = check_desc(d);
        if (st != MOM_OK) return st;
    }
    for (int i = 0; i < n_add; ++i) {
        mom_status_t st = check_desc(stored_add[i]);
        if (st != MOM_OK) return st;
    }
    // A transposed operand takes part with its transposed type: shape swapped, lowerTri <-> upperTri
    // (the inference rule of the paper's Section 2); `chain` / `add_terms` hold the types as used.
    auto as_used = [](const mom_matrix_desc_t &d, bool t) {
        if (!t) return d;
        return mom_matrix_desc_t{d.cols, d.rows, mom::transpose_property(d.property), d.dtype};
    };
    if (slot_names) {                                       // one name, one stored type
        try {
            std::map<int32_t, size_t> first;
            for (size_t i = 0; i < slots.size(); ++i) {
                auto it = first.emplace(slot_names[i], i).first;
                const mom_matrix_desc_t &a = slots[it->second], &b = slots[i];
                if (a.rows != b.rows || a.cols != b.cols || a.property != b.property) return MOM_ERR_INVALID_ARG;
            }
        } catch (const std::bad_alloc &) {
            return MOM_ERR_ALLOC;
        }
    }

    mom_plan *p = new (std::nothrow) mom_plan();
    if (!p) return MOM_ERR_ALLOC;
    try {
        p->variant = (int32_t)variant;
        p->ptr_desc = slots;
        if (slot_names) p->names.assign(slot_names, slot_names + slots.size());
        for (int i = 0; i < n_add; ++i) {
            p->add_t.push_back(add_transposed && add_transposed[i] != 0);
            p->add.push_back(as_used(stored_add[i], p->add_t.back() != 0));
        }
        p->chain_begin.push_back(0);

        int32_t next_id = n_chain;
        std::vector<std::string> sum_text(sums_in.size());
        std::vector<int64_t> factor_name;                   // per factor, over all sums

        for (size_t si = 0; si < sums_in.size(); ++si) {
            const SumIn &in = sums_in[si];
            const bool top = si + 1 == sums_in.size();
            mom::SumInfo info;
            info.step_begin = (int)p->steps.size();
            std::map<std::vector<int64_t>, int32_t> seen;   // run of (name, transposed) -> id of its product
            std::vector<int32_t> summand_props;
            std::string &text = sum_text[si];
            int64_t rows = 0, cols = 0;

            for (size_t c = 0; c < in.chains.size(); ++c) {
                if (c) text += "+";
                // this chain's factors as used
                const int begin = (int)p->chain.size();
                std::vector<int64_t> fname;
                std::vector<std::string> flabel;
                for (const FactorIn &f : in.chains[c]) {
                    if (f.sub >= 0) {
                        if ((size_t)f.sub >= si) { delete p; return MOM_ERR_INVALID_ARG; }
                        p->chain.push_back(p->sums[f.sub].desc);
                        p->chain_t.push_back(0);
                        flabel.push_back("[" + sum_text[f.sub] + "]");
                    } else {
                        if (f.ptr < 0 || (size_t)f.ptr >= slots.size()) { delete p; return MOM_ERR_INVALID_ARG; }
                        p->chain.push_back(as_used(slots[f.ptr], f.t));
                        p->chain_t.push_back(f.t ? 1 : 0);
                        flabel.push_back(f.label);
                    }
                    p->factor_ptr.push_back(f.sub >= 0 ? -1 : f.ptr);
                    p->factor_sum.push_back(f.sub);
                    fname.push_back(f.name);
                    factor_name.push_back(f.name);
                }
                const int end = (int)p->chain.size();
                p->chain_begin.push_back(end);
                const mom_matrix_desc_t *chain = p->chain.data();
                for (int i = begin; i + 1 < end; ++i)
                    if (chain[i].cols != chain[i + 1].rows) { delete p; return MOM_ERR_SHAPE_MISMATCH; }
                if (c == 0) { rows = chain[begin].rows; cols = chain[end - 1].cols; }
                else if (chain[begin].rows != rows || chain[end - 1].cols != cols) { delete p; return MOM_ERR_SHAPE_MISMATCH; }

                // identity simplification: A*I -> A, I*A -> A, I*I -> I
                std::vector<int32_t> kept;
                for (int i = begin; i < end; ++i)
                    if (chain[i].property != MOM_IDENTITY) kept.push_back(i);
                p->kept.insert(p->kept.end(), kept.begin(), kept.end());
                const int r = (int)kept.size();
                mom_matrix_desc_t value_desc;

                if (r == 0) {
                    text += "I";
                    value_desc = mom_matrix_desc_t{rows, cols, MOM_IDENTITY, MOM_F32};
                    info.summands.push_back(mom::Summand{mom::SUM_IDENTITY, 0});
                } else {
                    // dynamic program over the reduced chain
                    std::vector<Node> node((size_t)r * r);
                    std::vector<uint64_t> cost((size_t)r * r, 0);
                    std::vector<int> split((size_t)r * r, -1);
                    auto at = [r](int i, int j) { return (size_t)i * r + j; };
                    for (int i = 0; i < r; ++i) {
                        const auto &d = chain[kept[i]];
                        node[at(i, i)] = Node{d.rows, d.cols, d.property};
                    }
                    // Does the reduced run [i, j] read Y * Y^T factor by factor?  Factor j - q must be the transpose of
                    // factor i + q: the same named matrix with the other flag, or with any flag when it is its own
                    // transpose (Symmetric, Diagonal).
                    auto reads_as_gram = [&](int i, int j) {
                        if ((j - i + 1) % 2) return false;
                        for (int q = 0; q < (j - i + 1) / 2; ++q) {
                            const int a = kept[i + q], b = kept[j - q];
                            if (fname[a - begin] < 0 || fname[a - begin] != fname[b - begin]) return false;
                            const int32_t pa = chain[a].property;
                            if (p->chain_t[a] == p->chain_t[b] && pa != MOM_SYMMETRIC && pa != MOM_DIAGONAL) return false;
                        }
                        return true;
                    };
                    std::vector<char> gram((size_t)r * r, 0);       // [i, j] is a Gram product (typed Symmetric whatever its tree)
                    for (int len = 2; len <= r; ++len) {
                        for (int i = 0; i + len - 1 < r; ++i) {
                            const int j = i + len - 1;
                            // the type of [i, j] does not depend on its tree: join of the factors' types, Symmetric for a Gram run
                            int32_t prop = node[at(i, i)].prop;
                            for (int q = i + 1; q <= j; ++q) prop = join_property(prop, node[at(q, q)].prop);
                            const bool is_gram = prop == MOM_GENERAL && reads_as_gram(i, j);
                            gram[at(i, j)] = is_gram;
                            bool have = false;
                            uint64_t best = 0;
                            int best_k = -1;
                            for (int k = i; k < j; ++k) {
                                const Node &a = node[at(i, k)], &b = node[at(k + 1, j)];
                                uint64_t m;
                                u128 cst;
                                if (is_gram && 2 * k == i + j - 1) {            // split in the middle: the right half is never computed
                                    if (!gram_mults(a.prop, a.rows, a.cols, &m)) { delete p; return MOM_ERR_OVERFLOW; }
                                    cst = (u128)cost[at(i, k)] + m;
                                } else {
                                    if (!useful_mults(a.prop, b.prop, a.rows, a.cols, b.cols, &m)) { delete p; return MOM_ERR_OVERFLOW; }
                                    cst = (u128)cost[at(i, k)] + cost[at(k + 1, j)] + m;
                                }
                                if (cst >= (u128)COST_LIMIT) { delete p; return MOM_ERR_OVERFLOW; }
                                if (!have || (uint64_t)cst < best) { best = (uint64_t)cst; best_k = k; have = true; }
                            }
                            cost[at(i, j)] = best;
                            split[at(i, j)] = best_k;
                            const Node &a = node[at(i, best_k)], &b = node[at(best_k + 1, j)];
                            node[at(i, j)] = Node{a.rows, b.cols, is_gram ? (int32_t)MOM_SYMMETRIC : prop};
                        }
                    }

                    // Post-order emission of the binary products; returns the id of the value of [i, j].  A product
                    // below the root whose run of named factors an earlier chain of this sum already multiplied (also
                    // below its root) is not emitted again: its id is reused and only its text is written.
                    struct Emit {
                        mom_plan *p; const std::vector<Node> &node; const std::vector<int> &split; int r; int32_t &next_id;
                        const std::vector<int32_t> &kept; std::map<std::vector<int64_t>, int32_t> &seen;
                        const std::vector<int64_t> &fname; const std::vector<std::string> &flabel; int begin; int n_factors;
                        int sum_index; std::string &s; const std::vector<char> &gram;
                        // `key` receives the run of (name, transposed) factors the value multiplies (empty when a factor has
                        // no name); the right half of a Gram product Y * Y^T is Y's run reversed with every flag flipped
                        int32_t run(int i, int j, bool emit, std::vector<int64_t> &key) {
                            key.clear();
                            if (i == j) {
                                s += flabel[kept[i] - begin];
                                if (p->chain_t[kept[i]]) s += "^T";
                                if (fname[kept[i] - begin] >= 0) key.push_back(fname[kept[i] - begin] * 2 + (p->chain_t[kept[i]] ? 1 : 0));
                                return kept[i];
                            }
                            const bool root = i == 0 && j == r - 1;
                            const int k = split[(size_t)i * r + j];
                            const bool is_gram = gram[(size_t)i * r + j] && 2 * k == i + j - 1;
                            bool named = true;
                            for (int q = i; q <= j; ++q) named &= fname[kept[q] - begin] >= 0;
                            // text first (both halves as written), with nothing emitted; then the products
                            const size_t text_at = s.size();
                            std::vector<int64_t> kl, kr;
                            s += "(";
                            run(i, k, false, kl);
                            s += "*";
                            if (is_gram) right_nested(k + 1, j);  // never multiplied: every tree costs the same, the first in the tie order is written
                            else run(k + 1, j, false, kr);
                            s += ")";
                            if (!emit) {
                                if (named) {
                                    key = kl;
                                    if (is_gram) for (size_t q = kl.size(); q-- > 0;) key.push_back(kl[q] ^ 1);
                                    else key.insert(key.end(), kr.begin(), kr.end());
                                }
                                return -1;
                            }
                            const std::string text = s.substr(text_at);
                            s.resize(text_at);
                            std::string scratch;
                            std::swap(s, scratch);                // emission below must not write the text twice
                            int32_t l, rr;
                            {
                                std::vector<int64_t> k2;
                                if (named) {
                                    key = kl;
                                    if (is_gram) for (size_t q = kl.size(); q-- > 0;) key.push_back(kl[q] ^ 1);
                                    else key.insert(key.end(), kr.begin(), kr.end());
                                }
                                int32_t shared = -1;
                                if (named && !root) {
                                    auto it = seen.find(key);
                                    if (it != seen.end()) { shared = it->second; p->reused += count_products(i, j); }
                                }
                                if (shared >= 0) {
                                    std::swap(s, scratch);
                                    s += text;
                                    return shared;
                                }
                                l = run(i, k, true, k2);
                                rr = is_gram ? l : run(k + 1, j, true, k2);
                            }
                            std::swap(s, scratch);
                            s += text;
                            const Node &a = node[(size_t)i * r + k], &b = node[(size_t)(k + 1) * r + j], &o = node[(size_t)i * r + j];
                            mom::StepImpl st;
                            std::memset(&st.pub, 0, sizeof(st.pub));
                            st.pub.lhs = l; st.pub.rhs = rr; st.pub.out = next_id++;
                            st.pub.lhs_property = a.prop; st.pub.out_property = o.prop;
                            st.pub.lhs_transposed = l < n_factors && p->chain_t[l];
                            st.pub.m = a.rows; st.pub.k = a.cols;
                            if (is_gram) {
                                // Y * Y^T: the right operand is the left one read transposed
                                st.pub.rhs_property = mom::transpose_property(a.prop);
                                st.pub.rhs_transposed = l < n_factors ? !p->chain_t[l] : 1;
                                st.pub.n = a.rows;
                                gram_mults(a.prop, a.rows, a.cols, &st.pub.useful_mults);
                                st.pub.kind = MOM_KIND_GRAM;
                            } else {
                                st.pub.rhs_property = b.prop;
                                st.pub.rhs_transposed = rr < n_factors && p->chain_t[rr];
                                st.pub.n = b.cols;
                                useful_mults(a.prop, b.prop, a.rows, a.cols, b.cols, &st.pub.useful_mults);
                                const bool ta = is_tri(a.prop), tb = is_tri(b.prop);
                                st.pub.kind = a.prop == MOM_DIAGONAL || b.prop == MOM_DIAGONAL ? MOM_KIND_SCALE
                                              : !ta && !tb ? MOM_KIND_GG : ta && !tb ? MOM_KIND_TG : !ta && tb ? MOM_KIND_GT
                                              : is_lower(a.prop) == is_lower(b.prop) ? MOM_KIND_TT : MOM_KIND_TTMIX;
                            }
                            st.is_last = root;
                            if (root) st.sum = sum_index;
                            p->steps.push_back(st);
                            if (named && !root) seen.emplace(key, st.pub.out);
                            return st.pub.out;
                        }
                        void right_nested(int i, int j) {
                            if (i < j) s += "(";
                            s += flabel[kept[i] - begin];
                            if (p->chain_t[kept[i]]) s += "^T";
                            if (i < j) { s += "*"; right_nested(i + 1, j); s += ")"; }
                        }
                        // binary products in the chosen tree of [i, j] (a Gram node's right half has none)
                        int count_products(int i, int j) const {
                            if (i == j) return 0;
                            const int k = split[(size_t)i * r + j];
                            const bool is_gram = gram[(size_t)i * r + j] && 2 * k == i + j - 1;
                            return 1 + count_products(i, k) + (is_gram ? 0 : count_products(k + 1, j));
                        }
                    } emit{p, node, split, r, next_id, kept, seen, fname, flabel, begin, n_chain, (int)si, text, gram};
                    std::vector<int64_t> root_key;
                    emit.run(0, r - 1, true, root_key);
                    const Node &root = node[at(0, r - 1)];
                    value_desc = mom_matrix_desc_t{root.rows, root.cols, root.prop, MOM_F32};
                    if (r == 1) info.summands.push_back(mom::Summand{mom::SUM_FACTOR, kept[0]});
                    else info.summands.push_back(mom::Summand{mom::SUM_STEP, (int)p->steps.size() - 1});
                }
                if (c == 0) { if (top) p->product_desc = value_desc; }
                else p->add_flops += nnz(value_desc);
                summand_props.push_back(value_desc.property);
            }
            if (top) {
                for (int i = 0; i < n_add; ++i) {
                    if (p->add[i].rows != rows || p->add[i].cols != cols) { delete p; return MOM_ERR_SHAPE_MISMATCH; }
                    p->add_flops += nnz(p->add[i]);
                    info.summands.push_back(mom::Summand{mom::SUM_TERM, i});
                    summand_props.push_back(p->add[i].property);
                }
            }
            info.step_end = (int)p->steps.size();
            info.desc = mom_matrix_desc_t{rows, cols, sum_property(summand_props), MOM_F32};
            {                                           // every root after the first adds to what the sum's buffer holds
                bool first = true;
                for (int s = info.step_begin; s < info.step_end; ++s)
                    if (p->steps[s].is_last) { p->steps[s].accumulate = !first; first = false; }
            }
            p->sums.push_back(std::move(info));
        }
        p->slot_used.assign(slots.size(), 0);
        for (int32_t f : p->factor_ptr)
            if (f >= 0) p->slot_used[f] = 1;
        p->paren = sum_text.back();
        p->result_desc = p->sums.back().desc;
        p->temporaries = (int32_t)p->sums.size() - 1;
        for (const auto &st : p->steps) {
            const u128 sum = (u128)p->mults + st.pub.useful_mults;
            if (sum >= (u128)COST_LIMIT) { delete p; return MOM_ERR_OVERFLOW; }
            p->mults = (uint64_t)sum;
        }
        const bool single_chain = sums_in.size() == 1 && n_chains == 1;

        // kernel choice and workspace layout
        const int ns = (int)p->steps.size();
        std::vector<Interval> items;
        items.reserve((size_t)ns * 6);
        for (int s = 0; s < ns; ++s) {
            mom::StepImpl &st = p->steps[s];
            const int64_t m = st.pub.m, n = st.pub.n, k = st.pub.k;
            // what TMA can address (16-byte row pitch) and the tile table can hold (first row of a tile in 24 bits)
            const bool addressable = (k % 4 == 0) && (n % 4 == 0) && m <= mom::TC_MAX_ROWS && n <= mom::TC_MAX_ROWS;
            // below this size the tcgen05 path's extra launches (operand splits, split-K reduction) cost more
            // than its faster mainloop saves; the warp-level kernel is one launch
            const bool large = (double)m * (double)n * (double)k >= 6.0 * (double)(1 << 26);
            // in between: the tcgen05 kernel that reads the operands as stored and splits them in shared memory (one launch);
            // it takes operands (transposed ones as stored) whose rows TMA can address
            // (a Gram product Y * Y^T goes there only below the plane kernel's range: that one computes half of the tiles and mirrors them)
            const bool inline_ok = (st.pub.kind != MOM_KIND_GRAM || !large) &&
                                   mom::product_tc_inline_takes(m, n, k, st.pub.lhs_transposed, st.pub.rhs_transposed,
                                                                mom::kernel_property(st.pub.lhs_property), mom::kernel_property(st.pub.rhs_property));
            // ... and it pays between the two (measured, see the constants): from about 400^3 on it beats the warp-level kernel, and
            // its single launch beats the plane kernel's two up to 1000^3 whatever the shape and up to about 1600^3 while its
            // 128 x 128 tiles fit one wave of CTAs, and to 2000^3 while its CTA pairs' 256 x 256 tiles do; a result of fewer than four 128 x 128 tiles would leave each CTA a long
            // contraction even when split over a cluster, and the warp-level kernel is quicker there
            const double work = (double)m * (double)n * (double)k;
            const bool one_wave = ((m + 127) / 128) * ((n + 127) / 128) <= mom::INLINE_WAVE_TILES;
            // (only for an equation of one product: in a chain the plane kernel's steps hand each other their planes, which
            // saves the split passes that make it the slower one here: L*A*U*B at 2048 249 us against 263 us mixed)
            const bool one_wave_of_pairs = ns == 1 && ((m + 255) / 256) * ((n + 255) / 256) <= mom::INLINE_WAVE_PAIRS;
            const bool inline_pays = work >= mom::INLINE_MIN_WORK && (double)m * (double)n >= mom::INLINE_MIN_OUTPUT &&
                                     (work < mom::INLINE_SMALL_WORK || (work < mom::INLINE_MAX_WORK && one_wave) ||
                                      (work < mom::INLINE_PAIR_MAX_WORK && one_wave_of_pairs));
            if (st.pub.kind == MOM_KIND_SCALE) st.pub.uses_tensor_cores = 0;       // a Diagonal operand: one scaling pass, bound by HBM
            // operands or a result in packed storage: the plane kernel addresses the containers in place, the one-launch
            // kernel would need them unpacked first
            else if (variant == MOM_VARIANT_3XTF32 && packed_storage && addressable && large) st.pub.uses_tensor_cores = 1;
            else if (variant == MOM_VARIANT_3XTF32) st.pub.uses_tensor_cores = inline_ok && inline_pays ? 3 : addressable && large ? 1 : 2;
            else if (variant == MOM_VARIANT_3XTF32_FORCE) st.pub.uses_tensor_cores = addressable ? 1 : 0;
            else if (variant == MOM_VARIANT_3XTF32_WARP) st.pub.uses_tensor_cores = 2;
            else if (variant == MOM_VARIANT_3XTF32_INLINE) st.pub.uses_tensor_cores = inline_ok ? 3 : 2;
            else st.pub.uses_tensor_cores = 0;
            if (st.pub.uses_tensor_cores == 1) {
                // few output tiles, long contraction: split k over otherwise idle SMs
                const int64_t tiles = ((m + mom::TC_BM - 1) / mom::TC_BM) * ((n + mom::TC_BN - 1) / mom::TC_BN);
                if ((tiles <= 37 && k >= 512) || (tiles <= 74 && k >= 1024)) {      // up to half of the SMs busy otherwise
                    int64_t split = std::min<int64_t>(std::min<int64_t>(148 / tiles, k / 128), 32);
                    if (split >= 2) st.split_k = (int)split;
                }
            }
        }
        // A scaling step read by exactly one tensor-core step is folded into that step's operand-split pass.
        for (int s = 0; s < ns; ++s) {
            mom::StepImpl &st = p->steps[s];
            if (st.pub.kind != MOM_KIND_SCALE || st.is_last) continue;
            if (st.pub.lhs_property == MOM_DIAGONAL && st.pub.rhs_property == MOM_DIAGONAL) continue;
            int readers = 0, reader = -1;
            for (int t = s + 1; t < ns; ++t)
                if (p->steps[t].pub.lhs == st.pub.out || p->steps[t].pub.rhs == st.pub.out) { ++readers; reader = t; }
            if (readers != 1 || p->steps[reader].pub.uses_tensor_cores != 1) continue;
            if (p->steps[reader].pub.lhs == st.pub.out && p->steps[reader].pub.rhs == st.pub.out) continue;
            st.folded = true;
            st.fold_into = reader;
            (p->steps[reader].pub.lhs == st.pub.out ? p->steps[reader].fold_a : p->steps[reader].fold_b) = s;
        }
        // the step at which a reader really reads its operands: a folded step's operands are read by its target
        auto read_at = [&](int t) { return p->steps[t].folded ? p->steps[t].fold_into : t; };
        // f32 intermediates, or planes written by the producer: a tensor-core producer writes its consumers' operand
        // planes itself when every consumer is a tensor-core step that takes the value on the same side
        for (int s = 0; s < ns; ++s) {
            mom::StepImpl &st = p->steps[s];
            const int64_t m = st.pub.m, n = st.pub.n;
            int last_consumer = -1, as_lhs = 0, as_rhs = 0;   // a product shared between chains has several consumers
            bool all_tc = true;
            for (int t = s + 1; t < ns; ++t) {
                const mom::StepImpl &c = p->steps[t];
                if (c.pub.lhs != st.pub.out && c.pub.rhs != st.pub.out) continue;
                last_consumer = std::max(last_consumer, read_at(t));
                (c.pub.lhs == st.pub.out ? as_lhs : as_rhs)++;
                all_tc &= c.pub.uses_tensor_cores == 1;
            }
            // (a Gram product keeps its f32 output: its epilogue mirrors the lower triangle into the upper one)
            const bool fused_planes = last_consumer >= 0 && all_tc && (as_lhs == 0 || as_rhs == 0) &&
                                      st.pub.uses_tensor_cores == 1 && st.split_k == 1 && st.pub.kind != MOM_KIND_GRAM;
            // mirrored Gram product: only the tiles on and below the diagonal are computed, the others are written as
            // mirror images; needs a plain f32 result, and as a root a Symmetric sum (then every fused summand is
            // Symmetric, Diagonal or Identity, so the mirror image of entry (i, j) is the value of entry (j, i))
            st.mirror = st.pub.kind == MOM_KIND_GRAM && st.pub.uses_tensor_cores == 1 && st.split_k == 1 &&
                        (!st.is_last || (!st.accumulate && p->sums[st.sum].desc.property == MOM_SYMMETRIC));
            if (fused_planes) {
                st.planes_out = as_lhs ? 1 : 2;
            } else if (!st.is_last && !st.folded) {
                items.push_back(Interval{mom::align_up((size_t)m * n * sizeof(float), mom::WS_ALIGN), s,
                                         last_consumer < 0 ? ns - 1 : last_consumer, &st.out_off, 0});
            }
        }
        // temporaries of nested sums: written by their roots (or by one elementwise pass just before the next
        // sum's first product), read as a factor by later products or as a summand of a later sum
        for (size_t si = 0; si + 1 < p->sums.size(); ++si) {
            mom::SumInfo &sum = p->sums[si];
            const int last_step = ns > 0 ? ns - 1 : 0;
            int last = std::min(sum.step_begin, last_step);
            for (int t = 0; t < ns; ++t) {
                const mom_step_t &c = p->steps[t].pub;
                const bool reads = (c.lhs < n_chain && p->factor_sum[c.lhs] == (int)si) || (c.rhs < n_chain && p->factor_sum[c.rhs] == (int)si);
                if (reads) last = std::max(last, read_at(t));
            }
            for (size_t sj = si + 1; sj < p->sums.size(); ++sj)
                for (const mom::Summand &sm : p->sums[sj].summands)
                    if (sm.kind == mom::SUM_FACTOR && p->factor_sum[sm.index] == (int)si)
                        last = std::max(last, std::min(p->sums[sj].step_end, last_step));
            items.push_back(Interval{mom::align_up((size_t)sum.desc.rows * sum.desc.cols * sizeof(float), mom::WS_ALIGN),
                                     std::min(sum.step_begin, last_step), last, &sum.out_off, 0});
        }
        // Operand planes of the tensor-core steps.  Steps that take the same value on the same side (a shared
        // product; a named factor with the same transposition) read one set of planes: the first of them owns
        // the buffers, which then live until the last, and the others skip their split pass.
        struct Shared { int owner; size_t hi_item, lo_item; };
        std::map<std::pair<int64_t, int>, Shared> plane_sets;       // (value, side) -> owner
        struct Copy { int step, side, owner; };
        std::vector<Copy> copies;
        for (int s = 0; s < ns; ++s) {
            mom::StepImpl &st = p->steps[s];
            if (st.pub.uses_tensor_cores != 1) continue;
            const int64_t m = st.pub.m, n = st.pub.n, k = st.pub.k;
            for (int side = 0; side < 2; ++side) {
                if (side == 1 && st.pub.kind == MOM_KIND_GRAM) {
                    // Y * Y^T: the right operand's planes (n x k, K-major) are the left operand's
                    copies.push_back(Copy{s, 1, -1});
                    st.b_planes_ready = true;
                    continue;
                }
                const int32_t v = side == 0 ? st.pub.lhs : st.pub.rhs;
                const size_t bytes = mom::align_up((size_t)(side == 0 ? m * k : k * n) * sizeof(float), mom::WS_ALIGN);
                size_t *hi = side == 0 ? &st.a_hi_off : &st.b_hi_off, *lo = side == 0 ? &st.a_lo_off : &st.b_lo_off;
                bool &ready = side == 0 ? st.a_planes_ready : st.b_planes_ready;
                int from = s;
                int64_t key = -1;                                    // -1: nothing to share with
                if (v >= n_chain) {
                    const int producer = v - n_chain;
                    key = (int64_t)v << 1;
                    if (p->steps[producer].planes_out) { from = producer; ready = true; }
                } else if (factor_name[v] >= 0) {
                    key = ((factor_name[v] << 1) | (p->chain_t[v] ? 1 : 0)) | ((int64_t)1 << 62);
                }
                auto it = key >= 0 ? plane_sets.find({key, side}) : plane_sets.end();
                if (it != plane_sets.end()) {
                    items[it->second.hi_item].last = s;
                    items[it->second.lo_item].last = s;
                    copies.push_back(Copy{s, side, it->second.owner});
                    ready = true;
                    continue;
                }
                items.push_back(Interval{bytes, from, s, hi, 0});
                items.push_back(Interval{bytes, from, s, lo, 0});
                if (key >= 0) plane_sets[{key, side}] = Shared{s, items.size() - 2, items.size() - 1};
            }
            if (st.split_k > 1) {
                const size_t slab_rows = (size_t)((m + mom::TC_BM - 1) / mom::TC_BM * mom::TC_BM);
                items.push_back(Interval{mom::align_up((size_t)st.split_k * slab_rows * n * sizeof(float), mom::WS_ALIGN), s, s, &st.partial_off, 0});
            }
        }
        // Small products leave most of the GPU idle (a launch of a few microseconds on a few dozen SMs), so two subtrees of the tree that
        // do not depend on each other run side by side on two streams: the five-matrix chain ((0*(1*2))*(3*4)) computes (3*4) while
        // (0*(1*2)) is under way.  One such pair per plan: the node whose smaller subtree is the largest.  Every buffer either subtree
        // touches is kept for the whole of both (their steps no longer run one after the other).
        if (single_chain && variant != MOM_VARIANT_FFMA) {
            std::vector<int> first(ns, 0);                   // first step of the subtree that ends at step s (post-order: contiguous)
            std::vector<double> work(ns, 0.0);
            std::vector<char> small(ns, 1);
            for (int s = 0; s < ns; ++s) {
                const mom_step_t &st = p->steps[s].pub;
                first[s] = s;
                work[s] = (double)st.m * (double)st.n * (double)st.k;
                small[s] = st.uses_tensor_cores != 1 && st.kind != MOM_KIND_SCALE && work[s] < mom::SIDE_BY_SIDE_MAX_WORK && !p->steps[s].folded;
                for (int32_t v : {st.lhs, st.rhs})
                    if (v >= n_chain) {
                        const int c = v - n_chain;
                        first[s] = std::min(first[s], first[c]);
                        work[s] += work[c];
                        small[s] = small[s] && small[c];
                    }
            }
            double best = 0.0;
            for (int s = 0; s < ns; ++s) {
                const mom_step_t &st = p->steps[s].pub;
                if (st.lhs < n_chain || st.rhs < n_chain || st.lhs == st.rhs) continue;
                const int l = st.lhs - n_chain, r = st.rhs - n_chain;
                if (!small[l] || !small[r] || r != s - 1 || l != first[r] - 1) continue;      // left subtree, then right subtree, then s
                const double gain = std::min(work[l], work[r]);
                if (gain > best) { best = gain; p->side_begin = first[r]; p->side_end = r + 1; p->side_join = s; }
            }
            if (p->side_join >= 0) {
                const int lo = first[p->steps[p->side_join].pub.lhs - n_chain], hi = p->side_join;
                for (Interval &it : items)
                    if (!(it.last < lo || it.first > hi)) { it.first = std::min(it.first, lo); it.last = std::max(it.last, hi); }
            }
        }
        p->workspace_per_instance = pack(items);
        for (const Copy &c : copies) {
            if (c.owner < 0) continue;
            mom::StepImpl &st = p->steps[c.step];
            const mom::StepImpl &o = p->steps[c.owner];
            if (c.side == 0) { st.a_hi_off = o.a_hi_off; st.a_lo_off = o.a_lo_off; }
            else { st.b_hi_off = o.b_hi_off; st.b_lo_off = o.b_lo_off; }
        }
        for (const Copy &c : copies) {                  // Gram products: right planes = left planes (set above by now)
            if (c.owner >= 0) continue;
            mom::StepImpl &st = p->steps[c.step];
            st.b_hi_off = st.a_hi_off;
            st.b_lo_off = st.a_lo_off;
        }
        for (int s = 0; s < ns; ++s) {                  // a producer's plane targets are its consumers' operand planes
            mom::StepImpl &st = p->steps[s];
            if (!st.planes_out) continue;
            for (int t = s + 1; t < ns; ++t) {
                const mom::StepImpl &c = p->steps[t];
                if (st.planes_out == 1 && c.pub.lhs == st.pub.out) { st.planes_hi_off = c.a_hi_off; st.planes_lo_off = c.a_lo_off; }
                if (st.planes_out == 2 && c.pub.rhs == st.pub.out) { st.planes_hi_off = c.b_hi_off; st.planes_lo_off = c.b_lo_off; }
            }
        }

        // Small equations run as one fused kernel with every operand and intermediate in shared memory.
        {
            bool any_tc = false, any_gram = false;      // (a Gram product reads one value on both sides: the layout below gives a value one side)
            for (const auto &st : p->steps) { any_tc |= st.pub.uses_tensor_cores == 1; any_gram |= st.pub.kind == MOM_KIND_GRAM; }
            const int values = n_chain + ns;
            p->fused_value_off.assign(values, -1);
            size_t floats = 0;
            bool ok = single_chain && ns >= 1 && ns <= mom::FUSED_MAX_STEPS && (int)p->kept.size() <= mom::FUSED_MAX_OPERANDS &&
                      n_add <= mom::MAX_FUSED_ADD && !any_tc && variant != MOM_VARIANT_3XTF32_WARP && variant != MOM_VARIANT_3XTF32_INLINE && !any_gram;
            // every value feeds exactly one product: remember on which side
            std::vector<char> is_rhs(values, 0);
            for (const auto &st : p->steps) is_rhs[st.pub.rhs] = 1;
            p->fused_value_ld.assign(values, 0);
            if (ok) {
                for (int id : p->kept) {
                    p->fused_value_off[id] = (int)floats;
                    p->fused_value_ld[id] = mom::fused_ld((int)p->chain[id].cols, is_rhs[id] != 0);
                    floats += (size_t)p->chain[id].rows * p->fused_value_ld[id];
                    if (floats * sizeof(float) > mom::FUSED_MAX_SMEM) { ok = false; break; }
                }
            }
            if (ok) {
                for (int s = 0; s + 1 < ns; ++s) {
                    const int id = n_chain + s;
                    p->fused_value_off[id] = (int)floats;
                    p->fused_value_ld[id] = mom::fused_ld((int)p->steps[s].pub.n, is_rhs[id] != 0);
                    floats += (size_t)p->steps[s].pub.m * p->fused_value_ld[id];
                    if (floats * sizeof(float) > mom::FUSED_MAX_SMEM) { ok = false; break; }
                }
            }
            p->fused_ok = ok;
            p->fused_smem_bytes = ok ? floats * sizeof(float) : 0;
            if (ok) p->workspace_per_instance = 0;
        }
    } catch (const std::bad_alloc &) {
        delete p;
        return MOM_ERR_ALLOC;
    }
    *out_plan = p;
    return MOM_OK;
}

mom_status_t mom_equation_plan(const mom_matrix_desc_t *chain, int32_t n_chain,
                               const mom_matrix_desc_t *add_terms, int32_t n_add,
                               mom_variant_t variant, mom_plan_t **out_plan) {
    return mom_equation_plan_transposed(chain, nullptr, n_chain, add_terms, nullptr, n_add, variant, out_plan);
}

// one sum whose factors are the caller's array entries in order
static mom_status_t plan_flat(const mom_matrix_desc_t *stored, const int32_t *transposed, const int32_t *names,
                              const int32_t *chain_len, int32_t n_chains, const mom_matrix_desc_t *stored_add,
                              const int32_t *add_transposed, int32_t n_add, mom_variant_t variant, mom_plan_t **out_plan,
                              bool packed_storage = false) {
    if (!out_plan || !stored || !chain_len || n_chains < 1) return MOM_ERR_INVALID_ARG;
    try {
        std::vector<SumIn> sums(1);
        int64_t total = 0;
        for (int c = 0; c < n_chains; ++c) {
            if (chain_len[c] < 1 || total + chain_len[c] > (1 << 20)) return MOM_ERR_INVALID_ARG;
            std::vector<FactorIn> chain;
            for (int i = 0; i < chain_len[c]; ++i, ++total) {
                const int32_t f = (int32_t)total;
                chain.push_back(FactorIn{f, -1, transposed && transposed[f] != 0, names ? (int64_t)(uint32_t)names[f] : -1,
                                         std::to_string(f)});
            }
            sums[0].chains.push_back(std::move(chain));
        }
        std::vector<mom_matrix_desc_t> slots(stored, stored + total);
        return plan_sums(slots, sums, names, stored_add, add_transposed, n_add, variant, out_plan, packed_storage);
    } catch (const std::bad_alloc &) {
        return MOM_ERR_ALLOC;
    }
}

mom_status_t mom_equation_plan_transposed(const mom_matrix_desc_t *stored_chain, const int32_t *chain_transposed, int32_t n_chain,
                                          const mom_matrix_desc_t *stored_add, const int32_t *add_transposed, int32_t n_add,
                                          mom_variant_t variant, mom_plan_t **out_plan) {
    return plan_flat(stored_chain, chain_transposed, nullptr, &n_chain, 1, stored_add, add_transposed, n_add, variant, out_plan);
}

mom_status_t mom_packed_elements(int64_t rows, mom_property_t property, int64_t *elements) {
    if (!elements || rows < 1) return MOM_ERR_INVALID_ARG;
    if (property < MOM_GENERAL || property > MOM_UNIT_UPPER) return MOM_ERR_INVALID_ARG;
    if (!mom::is_triangular_kind(property)) return MOM_ERR_PROPERTY;
    if (rows > mom::MAX_DIMENSION) return MOM_ERR_LIMIT;
    const mom_matrix_desc_t d{rows, rows, (int32_t)property, MOM_F32};
    *elements = mom::stored_elements(d, MOM_STORAGE_PACKED);
    return MOM_OK;
}

mom_status_t mom_packed_row(int64_t rows, mom_property_t property, int64_t row, int64_t *offset, int64_t *first_col, int64_t *end_col) {
    if (!offset || !first_col || !end_col || rows < 1 || row < 0 || row >= rows) return MOM_ERR_INVALID_ARG;
    if (property < MOM_GENERAL || property > MOM_UNIT_UPPER) return MOM_ERR_INVALID_ARG;
    if (!mom::is_triangular_kind(property)) return MOM_ERR_PROPERTY;
    if (rows > mom::MAX_DIMENSION) return MOM_ERR_LIMIT;
    // the rows before `row` are the container of a `row`-row matrix whose rows have the same lengths: for a lower
    // triangle that is the packed `row` x `row` triangle; for an upper one the lengths depend on `rows` (n4 below)
    const int64_t q = row >> 2, rest = row - 4 * q, n4 = (rows + 3) & ~(int64_t)3;
    if (mom::is_lower_kind(property)) {
        *first_col = 0;
        *end_col = 4 * (q + 1);
        *offset = 8 * q * (q + 1) + rest * 4 * (q + 1);
    } else {
        *first_col = 4 * q;
        *end_col = n4;
        *offset = row * n4 - 8 * q * (q - 1) - 4 * q * rest;
    }
    return MOM_OK;
}

mom_status_t mom_plan_result_elements(const mom_plan_t *plan, int64_t *elements) {
    if (!plan || !elements) return MOM_ERR_INVALID_ARG;
    *elements = mom::stored_elements(plan->result_desc, plan->result_storage);
    return MOM_OK;
}

mom_status_t mom_equation_plan_stored(const mom_matrix_desc_t *chain, const int32_t *chain_transposed, const int32_t *chain_storage,
                                      int32_t n_chain, const mom_matrix_desc_t *add_terms, const int32_t *add_transposed,
                                      const int32_t *add_storage, int32_t n_add, mom_storage_t result_storage,
                                      mom_variant_t variant, mom_plan_t **out_plan) {
    if (result_storage != MOM_STORAGE_DENSE && result_storage != MOM_STORAGE_PACKED) return MOM_ERR_INVALID_ARG;
    mom_plan_t *p = nullptr;
    bool any_packed = result_storage == MOM_STORAGE_PACKED;
    for (int i = 0; chain_storage && i < n_chain; ++i) any_packed |= chain_storage[i] == MOM_STORAGE_PACKED;
    const mom_status_t st = plan_flat(chain, chain_transposed, nullptr, &n_chain, 1, add_terms, add_transposed, n_add, variant, &p, any_packed);
    if (st != MOM_OK) return st;
    auto fail = [&](mom_status_t e) { mom_plan_destroy(p); return e; };
    try {
        for (int i = 0; i < n_chain; ++i) {
            const int32_t sto = chain_storage ? chain_storage[i] : 0;
            if (sto != MOM_STORAGE_DENSE && sto != MOM_STORAGE_PACKED) return fail(MOM_ERR_INVALID_ARG);
            if (sto == MOM_STORAGE_PACKED && !mom::is_triangular_kind(chain[i].property)) return fail(MOM_ERR_PROPERTY);
            p->ptr_storage.push_back(sto);
        }
        for (int i = 0; i < n_add; ++i) {
            const int32_t sto = add_storage ? add_storage[i] : 0;
            if (sto != MOM_STORAGE_DENSE && sto != MOM_STORAGE_PACKED) return fail(MOM_ERR_INVALID_ARG);
            if (sto == MOM_STORAGE_PACKED && !mom::is_triangular_kind(add_terms[i].property)) return fail(MOM_ERR_PROPERTY);
            p->add_storage.push_back(sto);
        }
        if (result_storage == MOM_STORAGE_PACKED && !mom::is_triangular_kind(p->result_desc.property)) return fail(MOM_ERR_PROPERTY);
        p->result_storage = result_storage;
        // which packed operands every reader addresses in place: factors read only as operands of tcgen05 steps (their
        // operand-split pass has a packed addressing mode), as stored, not through a folded scaling, not as summands
        const int nf = (int)p->chain.size();
        p->slot_native.assign(p->ptr_desc.size(), 0);
        for (size_t slot = 0; slot < p->ptr_desc.size(); ++slot) {
            if (p->ptr_storage[slot] != MOM_STORAGE_PACKED || p->fused_ok) continue;
            bool native = true, read = false;
            for (int f = 0; f < nf; ++f) {
                if (p->factor_ptr[f] != (int)slot) continue;
                if (p->chain_t[f]) native = false;
                for (const auto &sp : p->steps) {
                    if (sp.pub.lhs != f && sp.pub.rhs != f) continue;
                    read = true;
                    if (sp.pub.uses_tensor_cores != 1 || sp.folded || sp.pub.kind == MOM_KIND_GRAM || sp.pub.kind == MOM_KIND_SCALE) native = false;
                }
                for (const auto &sum : p->sums)
                    for (const auto &sm : sum.summands)
                        if (sm.kind == mom::SUM_FACTOR && sm.index == f) native = false;
            }
            p->slot_native[slot] = native && read;
        }
        // a packed X is written in place when one tcgen05 product writes it, whole, with every summand fused
        if (result_storage == MOM_STORAGE_PACKED) {
            const mom::SumInfo &top = p->sums.back();
            int roots = 0, root = -1, simple = 0;
            for (const auto &sm : top.summands) {
                if (sm.kind == mom::SUM_STEP) { ++roots; root = sm.index; }
                else ++simple;
            }
            if (roots == 1 && simple <= mom::MAX_FUSED_ADD && !p->fused_ok) {
                const mom::StepImpl &r = p->steps[root];
                p->result_native = r.pub.uses_tensor_cores == 1 && r.split_k == 1 && !r.mirror && r.planes_out == 0 && !r.accumulate;
            }
        }
    } catch (const std::bad_alloc &) {
        return fail(MOM_ERR_ALLOC);
    }
    *out_plan = p;
    return MOM_OK;
}

mom_status_t mom_equation_plan_sum(const mom_matrix_desc_t *factors, const int32_t *factor_transposed,
                                   const int32_t *factor_names, const int32_t *chain_lengths, int32_t n_chains,
                                   mom_variant_t variant, mom_plan_t **out_plan) {
    return plan_flat(factors, factor_transposed, factor_names, chain_lengths, n_chains, nullptr, nullptr, 0, variant, out_plan);
}

// ---- nested expressions ------------------------------------------------------------------------------------
namespace {

// Normal form of an expression: transposes pushed down to the operands, products inside products and sums
// inside sums flattened, and every sum inside a product registered as a sum of its own (identical ones once).
struct Normalizer {
    const mom_expr_node_t *nodes; int32_t n_nodes; const int32_t *children; int32_t n_children; int32_t n_operands;
    std::vector<SumIn> sums;                          // registered nested sums, in dependency order
    std::map<std::string, int32_t> known;             // serialized normal form -> index in `sums`
    int64_t factors = 0;
    mom_status_t err = MOM_OK;

    static std::string serialize(const SumIn &s) {
        std::string out;
        for (const auto &c : s.chains) {
            out += "(";
            for (const FactorIn &f : c)
                out += f.sub >= 0 ? "S" + std::to_string(f.sub) + ";" : "L" + std::to_string(f.ptr) + (f.t ? "t;" : ";");
            out += ")";
        }
        return out;
    }

    SumIn run(int32_t node, bool t, int depth) {
        SumIn out;
        if (err != MOM_OK) return out;
        if (node < 0 || node >= n_nodes || depth > n_nodes) { err = MOM_ERR_INVALID_ARG; return out; }
        const mom_expr_node_t &nd = nodes[node];
        if (nd.kind == MOM_EXPR_OPERAND) {
            if (nd.operand < 0 || nd.operand >= n_operands) { err = MOM_ERR_INVALID_ARG; return out; }
            if (++factors > (1 << 20)) { err = MOM_ERR_INVALID_ARG; return out; }
            out.chains.push_back({FactorIn{nd.operand, -1, t, nd.operand, std::to_string(nd.operand)}});
            return out;
        }
        if (nd.n_children < 1 || nd.first_child < 0 || (int64_t)nd.first_child + nd.n_children > n_children) {
            err = MOM_ERR_INVALID_ARG;
            return out;
        }
        const int32_t *ch = children + nd.first_child;
        if (nd.kind == MOM_EXPR_TRANSPOSE) {
            if (nd.n_children != 1) { err = MOM_ERR_INVALID_ARG; return out; }
            return run(ch[0], !t, depth + 1);
        }
        if (nd.kind == MOM_EXPR_ADD) {
            for (int i = 0; i < nd.n_children && err == MOM_OK; ++i) {
                SumIn s = run(ch[i], t, depth + 1);
                for (auto &c : s.chains) out.chains.push_back(std::move(c));
            }
            return out;
        }
        if (nd.kind != MOM_EXPR_MUL) { err = MOM_ERR_INVALID_ARG; return out; }
        std::vector<FactorIn> chain;
        for (int i = 0; i < nd.n_children && err == MOM_OK; ++i) {
            SumIn s = run(ch[t ? nd.n_children - 1 - i : i], t, depth + 1);     // (e1*e2)^T = e2^T*e1^T
            if (err != MOM_OK) break;
            if (s.chains.size() == 1) {
                for (auto &f : s.chains[0]) chain.push_back(std::move(f));
            } else {
                const std::string key = serialize(s);
                auto it = known.find(key);
                int32_t index;
                if (it != known.end()) index = it->second;
                else {
                    index = (int32_t)sums.size();
                    sums.push_back(std::move(s));
                    known.emplace(key, index);
                }
                chain.push_back(FactorIn{-1, index, false, (int64_t)n_operands + index, std::string()});
            }
        }
        out.chains.push_back(std::move(chain));
        return out;
    }
};

}  // namespace

mom_status_t mom_expression_plan(const mom_matrix_desc_t *operands, int32_t n_operands,
                                 const mom_expr_node_t *nodes, int32_t n_nodes,
                                 const int32_t *children, int32_t n_children, int32_t root,
                                 mom_variant_t variant, mom_plan_t **out_plan) {
    if (!out_plan || !operands || n_operands < 1 || !nodes || n_nodes < 1 || n_children < 0 || (n_children > 0 && !children))
        return MOM_ERR_INVALID_ARG;
    try {
        Normalizer nz{nodes, n_nodes, children, n_children, n_operands, {}, {}, 0, MOM_OK};
        SumIn top = nz.run(root, false, 0);
        if (nz.err != MOM_OK) return nz.err;
        nz.sums.push_back(std::move(top));
        std::vector<mom_matrix_desc_t> slots(operands, operands + n_operands);
        return plan_sums(slots, nz.sums, nullptr, nullptr, nullptr, 0, variant, out_plan);
    } catch (const std::bad_alloc &) {
        return MOM_ERR_ALLOC;
    }
}

mom_status_t mom_plan_temporaries(const mom_plan_t *plan, int32_t *temporaries) {
    if (!plan || !temporaries) return MOM_ERR_INVALID_ARG;
    *temporaries = plan->temporaries;
    return MOM_OK;
}

mom_status_t mom_plan_reused_products(const mom_plan_t *plan, int32_t *reused) {
    if (!plan || !reused) return MOM_ERR_INVALID_ARG;
    *reused = plan->reused;
    return MOM_OK;
}

mom_status_t mom_plan_flops(const mom_plan_t *plan, uint64_t *mul_flops, uint64_t *add_flops) {
    if (!plan) return MOM_ERR_INVALID_ARG;
    if (mul_flops) *mul_flops = 2 * plan->mults;
    if (add_flops) *add_flops = plan->add_flops;
    return MOM_OK;
}

mom_status_t mom_plan_parenthesization(const mom_plan_t *plan, char *buf, size_t cap, size_t *needed) {
    if (!plan) return MOM_ERR_INVALID_ARG;
    const size_t need = plan->paren.size() + 1;
    if (needed) *needed = need;
    if (!buf || cap < need) return buf || needed ? MOM_ERR_BUFFER_TOO_SMALL : MOM_ERR_INVALID_ARG;
    std::memcpy(buf, plan->paren.c_str(), need);
    return MOM_OK;
}

mom_status_t mom_plan_num_steps(const mom_plan_t *plan, int32_t *n) {
    if (!plan || !n) return MOM_ERR_INVALID_ARG;
    *n = (int32_t)plan->steps.size();
    return MOM_OK;
}

mom_status_t mom_plan_step(const mom_plan_t *plan, int32_t i, mom_step_t *out) {
    if (!plan || !out || i < 0 || i >= (int32_t)plan->steps.size()) return MOM_ERR_INVALID_ARG;
    *out = plan->steps[i].pub;
    return MOM_OK;
}

mom_status_t mom_plan_result_desc(const mom_plan_t *plan, mom_matrix_desc_t *out) {
    if (!plan || !out) return MOM_ERR_INVALID_ARG;
    *out = plan->result_desc;
    return MOM_OK;
}

mom_status_t mom_plan_workspace_bytes(const mom_plan_t *plan, int64_t batch, size_t *bytes) {
    if (!plan || !bytes || batch < 1) return MOM_ERR_INVALID_ARG;
    // Plans with a tensor-core step walk the instances one after the other through one instance's
    // workspace; all-FFMA plans run up to 65535 instances per launch and keep one copy of each
    // intermediate per instance.
    bool any_tc = false;
    for (const auto &s : plan->steps) any_tc |= s.pub.uses_tensor_cores == 1;
    const int64_t group = any_tc ? 1 : (batch < 65535 ? batch : 65535);
    *bytes = plan->workspace_per_instance * (size_t)group;
    if (!plan->ptr_storage.empty() || plan->result_storage != MOM_STORAGE_DENSE) {
        // packed storage: dense copies for the kernels that cannot address a packed matrix, behind the plan's own room
        const size_t extra = mom::storage_layout(*plan, batch).bytes;
        if (extra) *bytes = mom::align_up(*bytes, mom::WS_ALIGN) + extra;
    }
    return MOM_OK;
}

mom_status_t mom_plan_host_staging_bytes(const mom_plan_t *plan, int64_t batch, size_t *bytes) {
    if (!plan || !bytes || batch < 1) return MOM_ERR_INVALID_ARG;
    size_t total = 0;
    for (size_t i = 0; i < plan->ptr_desc.size(); ++i) {
        const auto &d = plan->ptr_desc[i];
        if (d.property != MOM_IDENTITY) total += mom::align_up((size_t)mom::stored_elements(d, mom::slot_storage(*plan, (int)i)) * sizeof(float) * batch, mom::WS_ALIGN);
    }
    for (size_t i = 0; i < plan->add.size(); ++i) {
        const auto &d = plan->add[i];
        if (d.property != MOM_IDENTITY) total += mom::align_up((size_t)mom::stored_elements(d, mom::term_storage(*plan, (int)i)) * sizeof(float) * batch, mom::WS_ALIGN);
    }
    total += mom::align_up((size_t)mom::stored_elements(plan->result_desc, plan->result_storage) * sizeof(float) * batch, mom::WS_ALIGN);
    size_t ws = 0;
    mom_plan_workspace_bytes(plan, batch, &ws);
    total += ws;
    *bytes = total;
    return MOM_OK;
}

mom_status_t mom_plan_concurrent_steps(const mom_plan_t *plan, int32_t *begin, int32_t *end, int32_t *join) {
    if (!plan || !begin || !end || !join) return MOM_ERR_INVALID_ARG;
    *begin = plan->side_join >= 0 ? plan->side_begin : 0;
    *end = plan->side_join >= 0 ? plan->side_end : 0;
    *join = plan->side_join;
    return MOM_OK;
}

mom_status_t mom_plan_last_launch_count(const mom_plan_t *plan, int32_t *launches) {
    if (!plan || !launches) return MOM_ERR_INVALID_ARG;
    *launches = plan->last_launches;
    return MOM_OK;
}

mom_status_t mom_plan_destroy(mom_plan_t *plan) {
    if (!plan) return MOM_OK;
    mom::destroy_device_state(plan->dev);
    delete plan;
    return MOM_OK;
}

const char *mom_status_string(mom_status_t s) {
    switch (s) {
        case MOM_OK: return "ok";
        case MOM_ERR_INVALID_ARG: return "invalid argument";
        case MOM_ERR_PROPERTY: return "triangular, Diagonal, Symmetric and Identity matrices must be square";
        case MOM_ERR_DTYPE: return "unsupported element type";
        case MOM_ERR_SHAPE_MISMATCH: return "shape mismatch";
        case MOM_ERR_OVERFLOW: return "multiplication count overflows 63 bits";
        case MOM_ERR_ALLOC: return "allocation failed";
        case MOM_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case MOM_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
        case MOM_ERR_ARCH: return "device is not sm_100";
        case MOM_ERR_CUDA: return "CUDA call failed";
        case MOM_ERR_DEVICE_TIMEOUT: return "bounded device-side wait expired";
        case MOM_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case MOM_ERR_LIMIT: return "size beyond a fixed maximum";
    }
    return "unknown status";
}

}  // extern "C"
