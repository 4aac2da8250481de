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

namespace {

using u128 = unsigned __int128;
constexpr uint64_t COST_LIMIT = (uint64_t)1 << 63;

bool is_tri(int32_t p) { return p == MOM_LOWER_TRI || p == MOM_UPPER_TRI; }

// Least upper bound in  Identity < {lowerTri, upperTri} < general  (paper Listing 3 types L*L as lowerTri).
int32_t join_property(int32_t p, int32_t q) {
    if (p == MOM_IDENTITY) return q;
    if (q == MOM_IDENTITY) return p;
    return p == q ? p : (int32_t)MOM_GENERAL;
}

// Scalar multiplications a_il * b_lj of an (m x k)(k x n) product in which both factors are
// structurally non-zero.  Triangular operands are square.  Returns false on overflow.
bool useful_mults(int32_t pa, int32_t pb, int64_t m, int64_t k, int64_t n, uint64_t *out) {
    u128 v;
    const u128 M = (u128)m, K = (u128)k, N = (u128)n;
    if (!is_tri(pa) && !is_tri(pb)) {
        v = M * K * N;
    } else if (is_tri(pa) && !is_tri(pb)) {
        v = N * (K * (K + 1) / 2);                 // row i of A has i+1 (or k-i) non-zeros
    } else if (!is_tri(pa) && is_tri(pb)) {
        v = M * (K * (K + 1) / 2);
    } else if (pa == pb) {
        v = K * (K + 1) * (K + 2) / 6;             // sum_l (l+1)(k-l) over the shared triangle
    } else {
        v = K * (K + 1) * (2 * K + 1) / 6;         // sum_l (l+1)^2 : opposite triangles
    }
    if (v >= (u128)COST_LIMIT) return false;
    *out = (uint64_t)v;
    return true;
}

mom_status_t check_desc(const mom_matrix_desc_t &d) {
    if (d.rows < 1 || d.cols < 1) return MOM_ERR_INVALID_ARG;
    if (d.property < MOM_GENERAL || d.property > MOM_IDENTITY) return MOM_ERR_INVALID_ARG;
    if (d.dtype != MOM_F32) return MOM_ERR_DTYPE;
    if (d.property != MOM_GENERAL && d.rows != d.cols) return MOM_ERR_PROPERTY;
    return MOM_OK;
}

uint64_t nnz(const mom_matrix_desc_t &d) {
    if (d.property == MOM_GENERAL) return (uint64_t)d.rows * (uint64_t)d.cols;
    if (d.property == MOM_IDENTITY) return (uint64_t)d.rows;
    return (uint64_t)d.rows * ((uint64_t)d.rows + 1) / 2;
}

// Property of a sum of summands (chain values and Add terms).  A sum of two or more is never Identity: an
// Identity summand only contributes its diagonal footprint, which fits inside either triangle.
int32_t sum_property(const std::vector<int32_t> &props) {
    if (props.size() == 1) return props[0];
    bool seen = false;
    int32_t acc = MOM_GENERAL;
    for (int32_t p : props) {
        if (p == MOM_IDENTITY) continue;
        if (!seen) { acc = p; seen = true; }
        else if (acc != p) acc = MOM_GENERAL;
    }
    return seen ? acc : (int32_t)MOM_LOWER_TRI;
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

// Shared body of the planning entry points.  `factors` are all chains' stored factors one after the other,
// `chain_len[c]` of them belong to chain c; `names` (optional) tells which factors are the same stored matrix.
static mom_status_t plan_equation(const mom_matrix_desc_t *stored_chain, const int32_t *chain_transposed,
                                  const int32_t *names, const int32_t *chain_len, int32_t n_chains,
                                  const mom_matrix_desc_t *stored_add, const int32_t *add_transposed, int32_t n_add,
                                  mom_variant_t variant, mom_plan_t **out_plan) {
    if (!out_plan || !stored_chain || !chain_len || n_chains < 1 || n_add < 0 || (n_add > 0 && !stored_add))
        return MOM_ERR_INVALID_ARG;
    if ((int)variant < 0 || (int)variant > 2) return MOM_ERR_INVALID_ARG;
    int64_t total = 0;
    for (int c = 0; c < n_chains; ++c) {
        if (chain_len[c] < 1) return MOM_ERR_INVALID_ARG;
        total += chain_len[c];
        if (total > (1 << 20)) return MOM_ERR_INVALID_ARG;
    }
    const int n_chain = (int)total;
    for (int i = 0; i < n_chain; ++i) {
        mom_status_t st = check_desc(stored_chain[i]);
        if (st != MOM_OK) return st;
    }
    for (int i = 0; i < n_add; ++i) {
        mom_status_t st = check_desc(stored_add[i]);
        if (st != MOM_OK) return st;
    }
    // A transposed operand takes part with its transposed type: shape swapped, lowerTri <-> upperTri
    // (the inference rule of the paper's Section 2); from here on `chain` / `add_terms` are the types as used.
    auto as_used = [](const mom_matrix_desc_t &d, bool t) {
        if (!t) return d;
        const int32_t prop = d.property == MOM_LOWER_TRI ? (int32_t)MOM_UPPER_TRI
                             : d.property == MOM_UPPER_TRI ? (int32_t)MOM_LOWER_TRI : d.property;
        return mom_matrix_desc_t{d.cols, d.rows, prop, d.dtype};
    };
    std::vector<mom_matrix_desc_t> chain_v, add_v;
    std::vector<char> chain_t((size_t)n_chain, 0), add_t((size_t)n_add, 0);
    std::vector<int32_t> begin;
    try {
        for (int i = 0; i < n_chain; ++i) {
            chain_t[i] = chain_transposed && chain_transposed[i] != 0;
            chain_v.push_back(as_used(stored_chain[i], chain_t[i] != 0));
        }
        for (int i = 0; i < n_add; ++i) {
            add_t[i] = add_transposed && add_transposed[i] != 0;
            add_v.push_back(as_used(stored_add[i], add_t[i] != 0));
        }
        begin.push_back(0);
        for (int c = 0; c < n_chains; ++c) begin.push_back(begin.back() + chain_len[c]);
        if (names) {                                   // one name, one stored type
            std::map<int32_t, int> first;
            for (int i = 0; i < n_chain; ++i) {
                auto it = first.emplace(names[i], i).first;
                const mom_matrix_desc_t &a = stored_chain[it->second], &b = stored_chain[i];
                if (a.rows != b.rows || a.cols != b.cols || a.property != b.property) return MOM_ERR_INVALID_ARG;
            }
        }
    } catch (const std::bad_alloc &) {
        return MOM_ERR_ALLOC;
    }
    const mom_matrix_desc_t *chain = chain_v.data(), *add_terms = add_v.data();
    for (int c = 0; c < n_chains; ++c)
        for (int i = begin[c]; i + 1 < begin[c + 1]; ++i)
            if (chain[i].cols != chain[i + 1].rows) return MOM_ERR_SHAPE_MISMATCH;
    const int64_t rows = chain[0].rows, cols = chain[begin[1] - 1].cols;
    for (int c = 1; c < n_chains; ++c)
        if (chain[begin[c]].rows != rows || chain[begin[c + 1] - 1].cols != cols) return MOM_ERR_SHAPE_MISMATCH;
    for (int i = 0; i < n_add; ++i)
        if (add_terms[i].rows != rows || add_terms[i].cols != cols) return MOM_ERR_SHAPE_MISMATCH;

    mom_plan *p = new (std::nothrow) mom_plan();
    if (!p) return MOM_ERR_ALLOC;
    try {
        p->variant = (int32_t)variant;
        p->chain.assign(chain, chain + n_chain);
        if (n_add) p->add.assign(add_terms, add_terms + n_add);
        p->chain_t = chain_t;
        p->add_t = add_t;
        p->chain_begin = begin;
        if (names) p->names.assign(names, names + n_chain);
        for (int i = 0; i < n_add; ++i) p->add_flops += nnz(add_terms[i]);

        int32_t next_id = n_chain;
        std::map<std::vector<int64_t>, int32_t> seen;       // run of (name, transposed) -> id of its product
        std::vector<int32_t> summand_props;

        for (int c = 0; c < n_chains; ++c) {
            if (c) p->paren += "+";
            // identity simplification: A*I -> A, I*A -> A, I*I -> I
            std::vector<int32_t> kept;
            for (int i = begin[c]; i < begin[c + 1]; ++i)
                if (chain[i].property != MOM_IDENTITY) kept.push_back(i);
            p->kept.insert(p->kept.end(), kept.begin(), kept.end());
            const int r = (int)kept.size();
            mom_matrix_desc_t value_desc;

            if (r == 0) {
                p->paren += "I";
                value_desc = mom_matrix_desc_t{rows, cols, MOM_IDENTITY, MOM_F32};
                p->summands.push_back(mom::Summand{mom::SUM_IDENTITY, 0});
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
                for (int len = 2; len <= r; ++len) {
                    for (int i = 0; i + len - 1 < r; ++i) {
                        const int j = i + len - 1;
                        bool have = false;
                        uint64_t best = 0;
                        int best_k = -1;
                        for (int k = i; k < j; ++k) {
                            const Node &a = node[at(i, k)], &b = node[at(k + 1, j)];
                            uint64_t m;
                            if (!useful_mults(a.prop, b.prop, a.rows, a.cols, b.cols, &m)) { delete p; return MOM_ERR_OVERFLOW; }
                            const u128 cst = (u128)cost[at(i, k)] + cost[at(k + 1, j)] + m;
                            if (cst >= (u128)COST_LIMIT) { delete p; return MOM_ERR_OVERFLOW; }
                            if (!have || (uint64_t)cst < best) { best = (uint64_t)cst; best_k = k; have = true; }
                        }
                        cost[at(i, j)] = best;
                        split[at(i, j)] = best_k;
                        const Node &a = node[at(i, best_k)], &b = node[at(best_k + 1, j)];
                        node[at(i, j)] = Node{a.rows, b.cols, join_property(a.prop, b.prop)};
                    }
                }

                // Post-order emission of the binary products; returns the id of the value of [i, j].  A product
                // below the root whose run of named factors an earlier chain already multiplied (also below its
                // root) is not emitted again: its id is reused and only its text is written.
                struct Emit {
                    mom_plan *p; const std::vector<Node> &node; const std::vector<int> &split; int r; int32_t &next_id;
                    const std::vector<int32_t> &kept; std::map<std::vector<int64_t>, int32_t> &seen; bool named;
                    std::string &s;
                    int32_t run(int i, int j, bool emit) {
                        if (i == j) {
                            s += std::to_string(kept[i]);
                            if (p->chain_t[kept[i]]) s += "^T";
                            return kept[i];
                        }
                        const bool root = i == 0 && j == r - 1;
                        std::vector<int64_t> key;
                        int32_t shared = -1;
                        if (emit && named && !root) {
                            for (int q = i; q <= j; ++q) key.push_back((int64_t)p->names[kept[q]] * 2 + (p->chain_t[kept[q]] ? 1 : 0));
                            auto it = seen.find(key);
                            if (it != seen.end()) { shared = it->second; p->reused += j - i; }
                        }
                        const bool emit_here = emit && shared < 0;
                        const int k = split[(size_t)i * r + j];
                        s += "(";
                        const int32_t l = run(i, k, emit_here);
                        s += "*";
                        const int32_t rr = run(k + 1, j, emit_here);
                        s += ")";
                        if (!emit) return -1;
                        if (shared >= 0) return shared;
                        const Node &a = node[(size_t)i * r + k], &b = node[(size_t)(k + 1) * r + j], &o = node[(size_t)i * r + j];
                        mom::StepImpl st;
                        std::memset(&st.pub, 0, sizeof(st.pub));
                        st.pub.lhs = l; st.pub.rhs = rr; st.pub.out = next_id++;
                        st.pub.lhs_property = a.prop; st.pub.rhs_property = b.prop; st.pub.out_property = o.prop;
                        st.pub.lhs_transposed = l < (int32_t)p->chain.size() && p->chain_t[l];
                        st.pub.rhs_transposed = rr < (int32_t)p->chain.size() && p->chain_t[rr];
                        st.pub.m = a.rows; st.pub.k = a.cols; st.pub.n = b.cols;
                        useful_mults(a.prop, b.prop, a.rows, a.cols, b.cols, &st.pub.useful_mults);
                        const bool ta = is_tri(a.prop), tb = is_tri(b.prop);
                        st.pub.kind = !ta && !tb ? MOM_KIND_GG : ta && !tb ? MOM_KIND_TG : !ta && tb ? MOM_KIND_GT
                                      : a.prop == b.prop ? MOM_KIND_TT : MOM_KIND_TTMIX;
                        st.is_last = root;
                        p->steps.push_back(st);
                        if (named && !root) seen.emplace(std::move(key), st.pub.out);
                        return st.pub.out;
                    }
                } emit{p, node, split, r, next_id, kept, seen, names != nullptr, p->paren};
                emit.run(0, r - 1, true);
                const Node &root = node[at(0, r - 1)];
                value_desc = mom_matrix_desc_t{root.rows, root.cols, root.prop, MOM_F32};
                if (r == 1) p->summands.push_back(mom::Summand{mom::SUM_FACTOR, kept[0]});
                else p->summands.push_back(mom::Summand{mom::SUM_STEP, (int)p->steps.size() - 1});
            }
            if (c == 0) p->product_desc = value_desc;
            else p->add_flops += nnz(value_desc);
            summand_props.push_back(value_desc.property);
        }
        for (const auto &st : p->steps) {
            const u128 sum = (u128)p->mults + st.pub.useful_mults;
            if (sum >= (u128)COST_LIMIT) { delete p; return MOM_ERR_OVERFLOW; }
            p->mults = (uint64_t)sum;
        }
        for (int i = 0; i < n_add; ++i) {
            p->summands.push_back(mom::Summand{mom::SUM_TERM, i});
            summand_props.push_back(add_terms[i].property);
        }
        p->result_desc = mom_matrix_desc_t{rows, cols, sum_property(summand_props), MOM_F32};
        {                                               // every root after the first adds to what X holds
            bool first = true;
            for (auto &st : p->steps)
                if (st.is_last) { st.accumulate = !first; first = false; }
        }

        // kernel choice and workspace layout
        const int ns = (int)p->steps.size();
        std::vector<Interval> items;
        items.reserve((size_t)ns * 6);
        for (int s = 0; s < ns; ++s) {
            mom::StepImpl &st = p->steps[s];
            const int64_t m = st.pub.m, n = st.pub.n, k = st.pub.k;
            const bool addressable = (k % 4 == 0) && (n % 4 == 0);
            const bool worth_it = (double)m * (double)n * (double)k >= (double)(1 << 23);
            st.pub.uses_tensor_cores =
                (variant == MOM_VARIANT_3XTF32 && addressable && worth_it) || ((int)variant == 2 && addressable);
            if (st.pub.uses_tensor_cores) {
                // few output tiles, long contraction: split k over otherwise idle SMs
                const int64_t tiles = ((m + mom::TC_BM - 1) / mom::TC_BM) * ((n + mom::TC_BN - 1) / mom::TC_BN);
                if (tiles <= 37 && k >= 512) {
                    int64_t split = std::min<int64_t>(std::min<int64_t>(148 / tiles, k / 128), 32);
                    if (split >= 2) st.split_k = (int)split;
                }
            }
        }
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
                last_consumer = t;
                (c.pub.lhs == st.pub.out ? as_lhs : as_rhs)++;
                all_tc &= c.pub.uses_tensor_cores != 0;
            }
            const bool fused_planes = last_consumer >= 0 && all_tc && (as_lhs == 0 || as_rhs == 0) &&
                                      st.pub.uses_tensor_cores && st.split_k == 1;
            if (fused_planes) {
                st.planes_out = as_lhs ? 1 : 2;
            } else if (!st.is_last) {
                items.push_back(Interval{mom::align_up((size_t)m * n * sizeof(float), mom::WS_ALIGN), s,
                                         last_consumer < 0 ? ns - 1 : last_consumer, &st.out_off, 0});
            }
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
            if (!st.pub.uses_tensor_cores) continue;
            const int64_t m = st.pub.m, n = st.pub.n, k = st.pub.k;
            for (int side = 0; side < 2; ++side) {
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
                } else if (names) {
                    key = (((int64_t)names[v] << 1) | (chain_t[v] ? 1 : 0)) | ((int64_t)1 << 62);
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
        p->workspace_per_instance = pack(items);
        for (const Copy &c : copies) {
            mom::StepImpl &st = p->steps[c.step];
            const mom::StepImpl &o = p->steps[c.owner];
            if (c.side == 0) { st.a_hi_off = o.a_hi_off; st.a_lo_off = o.a_lo_off; }
            else { st.b_hi_off = o.b_hi_off; st.b_lo_off = o.b_lo_off; }
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
            bool any_tc = false;
            for (const auto &st : p->steps) any_tc |= st.pub.uses_tensor_cores != 0;
            const int values = n_chain + ns;
            p->fused_value_off.assign(values, -1);
            size_t floats = 0;
            bool ok = n_chains == 1 && ns >= 1 && ns <= mom::FUSED_MAX_STEPS && (int)p->kept.size() <= mom::FUSED_MAX_OPERANDS &&
                      n_add <= mom::MAX_FUSED_ADD && !any_tc;
            // every value feeds exactly one product: remember on which side
            std::vector<char> is_rhs(values, 0);
            for (const auto &st : p->steps) is_rhs[st.pub.rhs] = 1;
            p->fused_value_ld.assign(values, 0);
            if (ok) {
                for (int id : p->kept) {
                    p->fused_value_off[id] = (int)floats;
                    p->fused_value_ld[id] = mom::fused_ld((int)chain[id].cols, is_rhs[id] != 0);
                    floats += (size_t)chain[id].rows * p->fused_value_ld[id];
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

mom_status_t mom_equation_plan_transposed(const mom_matrix_desc_t *stored_chain, const int32_t *chain_transposed, int32_t n_chain,
                                          const mom_matrix_desc_t *stored_add, const int32_t *add_transposed, int32_t n_add,
                                          mom_variant_t variant, mom_plan_t **out_plan) {
    return plan_equation(stored_chain, chain_transposed, nullptr, &n_chain, 1, stored_add, add_transposed, n_add, variant, out_plan);
}

mom_status_t mom_equation_plan_sum(const mom_matrix_desc_t *factors, const int32_t *factor_transposed,
                                   const int32_t *factor_names, const int32_t *chain_lengths, int32_t n_chains,
                                   mom_variant_t variant, mom_plan_t **out_plan) {
    return plan_equation(factors, factor_transposed, factor_names, chain_lengths, n_chains, nullptr, nullptr, 0, variant, out_plan);
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
    for (const auto &s : plan->steps) any_tc |= s.pub.uses_tensor_cores != 0;
    const int64_t group = any_tc ? 1 : (batch < 65535 ? batch : 65535);
    *bytes = plan->workspace_per_instance * (size_t)group;
    return MOM_OK;
}

mom_status_t mom_plan_host_staging_bytes(const mom_plan_t *plan, int64_t batch, size_t *bytes) {
    if (!plan || !bytes || batch < 1) return MOM_ERR_INVALID_ARG;
    size_t total = 0;
    for (const auto &d : plan->chain)
        if (d.property != MOM_IDENTITY) total += mom::align_up((size_t)d.rows * d.cols * sizeof(float) * batch, mom::WS_ALIGN);
    for (const auto &d : plan->add)
        if (d.property != MOM_IDENTITY) total += mom::align_up((size_t)d.rows * d.cols * sizeof(float) * batch, mom::WS_ALIGN);
    total += mom::align_up((size_t)plan->result_desc.rows * plan->result_desc.cols * sizeof(float) * batch, mom::WS_ALIGN);
    size_t ws = 0;
    mom_plan_workspace_bytes(plan, batch, &ws);
    total += ws;
    *bytes = total;
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
        case MOM_ERR_PROPERTY: return "triangular and Identity matrices must be square";
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
