// Launcher: walks a plan's steps and enqueues the kernels on the caller's stream.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "batched_chain.h"
#include "fused_small.h"
#include "kernels.h"
#include "mom_internal.h"
#include "product_tc.h"

namespace mom {

struct DeviceState {
    int device = -1;
    int32_t *status = nullptr;          // device: {code, detail, 0, 0}
    TcPlanState tc;                     // tile tables of tensor-core steps
    uint2 *fused_table = nullptr;       // copy table of the fused small-equation kernel
    std::vector<int> fused_tab_begin, fused_tab_end;    // per kept operand: its rows of the table
    // step timing: a ring of TIMING_SLOTS executes, 3 events per step (before pre-pass, before product, after)
    std::vector<cudaEvent_t> events;
    long long timed_executes = 0;       // executes recorded since timing was enabled
    // host-staging entry point: uploads run on a stream of their own, one event per operand, so that the first
    // products start while later operands are still on their way
    // two independent subtrees of small products run side by side: the right one on this stream (see mom_plan::side_join)
    cudaStream_t side_stream = nullptr;
    cudaEvent_t side_fork = nullptr, side_done = nullptr;
    cudaStream_t copy_stream = nullptr, back_stream = nullptr;
    cudaEvent_t call_start = nullptr, first_rows_done = nullptr, back_done = nullptr;
    std::vector<cudaEvent_t> slot_ready, add_ready, slot_head;
};

// events the launcher has to wait for before it first uses an operand (host-staging entry point only)
// and, the other way, an event the launcher records once the first rows of X are final (first_rows is set to their
// number, 0 when X is only final at the end)
struct StageEvents {
    const cudaEvent_t *slot; const cudaEvent_t *add; cudaEvent_t first_rows_done; int *first_rows;
    // operands uploaded in two pieces: slot_head[i] is recorded once rows [0, slot_head_rows[i]) have arrived (0: one piece)
    const cudaEvent_t *slot_head; const int *slot_head_rows;
};

constexpr int TIMING_SLOTS = 32;

// host-staging entry point: triangular operands of at least UPLOAD_MIN rows are uploaded in blocks of UPLOAD_BLOCK rows
constexpr int64_t UPLOAD_BLOCK = 256, UPLOAD_MIN = 1024;
inline bool triangular_upload(const mom_matrix_desc_t &d, int64_t batch, int32_t storage = MOM_STORAGE_DENSE) {
    if (storage != MOM_STORAGE_DENSE) return false;          // a packed triangle crosses the bus as it is
    const int32_t kp = kernel_property(d.property);        // strict and unit triangles lie inside the ordinary one
    return batch == 1 && d.rows >= UPLOAD_MIN && (kp == MOM_LOWER_TRI || kp == MOM_UPPER_TRI);
}
inline size_t upload_bytes(const mom_matrix_desc_t &d, int64_t batch, int32_t storage = MOM_STORAGE_DENSE) {
    if (!triangular_upload(d, batch, storage)) return (size_t)stored_elements(d, storage) * sizeof(float) * batch;
    size_t total = 0;
    for (int64_t r0 = 0; r0 < d.rows; r0 += UPLOAD_BLOCK) {
        const int64_t r1 = std::min<int64_t>(d.rows, r0 + UPLOAD_BLOCK);
        total += (size_t)(r1 - r0) * (size_t)(kernel_property(d.property) == MOM_LOWER_TRI ? r1 : d.rows - r0) * sizeof(float);
    }
    return total;
}

void destroy_device_state(DeviceState *d) {
    if (!d) return;
    int prev = -1;
    cudaGetDevice(&prev);
    if (d->device >= 0) cudaSetDevice(d->device);
    tc_release(d->tc);
    for (cudaEvent_t e : d->events) cudaEventDestroy(e);
    for (cudaEvent_t e : d->slot_ready) cudaEventDestroy(e);
    for (cudaEvent_t e : d->slot_head) cudaEventDestroy(e);
    for (cudaEvent_t e : d->add_ready) cudaEventDestroy(e);
    if (d->call_start) cudaEventDestroy(d->call_start);
    if (d->first_rows_done) cudaEventDestroy(d->first_rows_done);
    if (d->back_done) cudaEventDestroy(d->back_done);
    if (d->side_fork) cudaEventDestroy(d->side_fork);
    if (d->side_done) cudaEventDestroy(d->side_done);
    if (d->side_stream) cudaStreamDestroy(d->side_stream);
    if (d->copy_stream) cudaStreamDestroy(d->copy_stream);
    if (d->back_stream) cudaStreamDestroy(d->back_stream);
    if (d->status) cudaFree(d->status);
    if (d->fused_table) cudaFree(d->fused_table);
    if (prev >= 0) cudaSetDevice(prev);
    delete d;
}

namespace {

mom_status_t check_arch(int *device_out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MOM_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return MOM_ERR_CUDA;
    if (major != 10) return MOM_ERR_ARCH;
    *device_out = dev;
    return MOM_OK;
}

mom_status_t ensure_device_state(const mom_plan *p, int device) {
    if (p->dev && p->dev->device == device) return MOM_OK;
    if (p->dev) { destroy_device_state(p->dev); p->dev = nullptr; }
    DeviceState *d = new (std::nothrow) DeviceState();
    if (!d) return MOM_ERR_ALLOC;
    d->device = device;
    if (cudaMalloc(&d->status, 4 * sizeof(int32_t)) != cudaSuccess) { delete d; return MOM_ERR_ALLOC; }
    if (cudaMemset(d->status, 0, 4 * sizeof(int32_t)) != cudaSuccess) { cudaFree(d->status); delete d; return MOM_ERR_CUDA; }
    p->dev = d;
    return MOM_OK;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Per call: which of the caller's pointers are packed triangles that the kernels read (or write) in place.
struct StorageCall {
    std::vector<char> slot_packed;
    bool out_packed = false;
};

// A plan the batched-chain kernel can run: a right-nested chain M_S * (... (M_1 * B)) of stored, untransposed
// factors with whole 16-row blocks and a right end of 8 or 16 columns, Add terms not transposed, many instances.
bool batched_chain_plan(const mom_plan *p, int64_t batch, const float *const *chain_ptrs, const int64_t *chain_strides,
                        const float *const *add_ptrs, const int64_t *add_strides, float *out, int64_t out_stride,
                        BatchedChainPlan *bp, const StorageCall *sc = nullptr) {
    if (sc && sc->out_packed) return false;
    if (batch < BATCHED_CHAIN_MIN_BATCH || !batched_chain_shape(*p)) return false;
    const int S = (int)p->steps.size(), n_add = (int)p->add.size();
    const int n = (int)p->steps[0].pub.n;
    std::memset(bp, 0, sizeof(*bp));
    for (int s = 0; s < S; ++s) {
        const mom_step_t &st = p->steps[s].pub;
        const int pa = kernel_property(st.lhs_property), pb = kernel_property(st.rhs_property);
        BatchedChainStep &b = bp->steps[s];
        const int slot = p->factor_ptr[st.lhs];
        b.lhs = chain_ptrs[slot];
        b.lhs_stride = chain_strides ? chain_strides[slot] : 0;
        b.m = (int)st.m;
        b.k = (int)st.k;
        b.packed = sc && sc->slot_packed[slot] ? (pa == MOM_LOWER_TRI ? 1 : 2) : 0;
        unsigned char needed[4] = {0, 0, 0, 0};
        for (int rb = 0; rb < b.m / 16; ++rb) {
            int klo, khi;
            tile_k_range(pa, pb, 16 * rb, 16 * rb + 16, 0, n, b.k, &klo, &khi);
            for (int c = klo / 16; c < (khi + 15) / 16; ++c) needed[rb] |= (unsigned char)(1u << c);
        }
        batched_chain_assign(needed, b.m / 16, &b);
    }
    const int rslot = p->factor_ptr[p->steps[0].pub.rhs];
    if (sc && sc->slot_packed[rslot]) return false;          // the right end is read dense
    bp->n_steps = S;
    bp->rhs = chain_ptrs[rslot];
    bp->rhs_stride = chain_strides ? chain_strides[rslot] : 0;
    bp->n = n;
    bp->add.count = n_add;
    bp->add.rows = (int)p->result_desc.rows;
    for (int i = 0; i < n_add; ++i) {
        bp->add.ptr[i] = p->add[i].property == MOM_IDENTITY ? nullptr : add_ptrs[i];
        bp->add.stride[i] = add_strides ? add_strides[i] : 0;
    }
    bp->out = out;
    bp->out_stride = out_stride;
    bp->pout = kernel_property(p->result_desc.property);
    bp->batch = batch;
    return true;
}

struct Operand { const float *ptr; long long stride; };

mom_status_t execute_core(const mom_plan *p, const float *const *chain_ptrs, const int64_t *chain_strides,
                          const float *const *add_ptrs, const int64_t *add_strides, float *out, int64_t out_stride,
                          int64_t batch, void *workspace, size_t workspace_bytes, cudaStream_t stream,
                          const StageEvents *staged = nullptr, const StorageCall *sc = nullptr) {
    if (!p || !chain_ptrs || !out || batch < 1) return MOM_ERR_INVALID_ARG;
    const int n_chain = (int)p->chain.size(), n_add = (int)p->add.size(), n_ptrs = (int)p->ptr_desc.size();
    if (n_add > 0 && !add_ptrs) return MOM_ERR_INVALID_ARG;
    if (batch > 1 && (!chain_strides || (n_add > 0 && !add_strides))) return MOM_ERR_INVALID_ARG;
    const int64_t rows = p->result_desc.rows, cols = p->result_desc.cols;

    for (int i = 0; i < n_ptrs; ++i) {
        if (p->ptr_desc[i].property == MOM_IDENTITY || !p->slot_used[i]) continue;
        if (!chain_ptrs[i]) return MOM_ERR_INVALID_ARG;
        if (!aligned16(chain_ptrs[i])) return MOM_ERR_ALIGNMENT;
        const bool in_place = sc && sc->slot_packed[i];
        if (batch > 1 && (chain_strides[i] % 4 != 0 || chain_strides[i] < stored_elements(p->ptr_desc[i], in_place ? MOM_STORAGE_PACKED : MOM_STORAGE_DENSE)))
            return MOM_ERR_INVALID_ARG;
    }
    if (!p->names.empty()) {          // entries with one name are one matrix: a product shared between chains relies on it
        for (int i = 0; i < n_ptrs; ++i)
            for (int j = 0; j < i; ++j)
                if (p->names[i] == p->names[j] && p->ptr_desc[i].property != MOM_IDENTITY && p->slot_used[i] && p->slot_used[j] &&
                    (chain_ptrs[i] != chain_ptrs[j] || (batch > 1 && chain_strides[i] != chain_strides[j])))
                    return MOM_ERR_INVALID_ARG;
    }
    for (int i = 0; i < n_add; ++i) {
        if (p->add[i].property == MOM_IDENTITY) continue;
        if (!add_ptrs[i]) return MOM_ERR_INVALID_ARG;
        if (!aligned16(add_ptrs[i])) return MOM_ERR_ALIGNMENT;
        if (batch > 1 && (add_strides[i] % 4 != 0 || add_strides[i] < rows * cols)) return MOM_ERR_INVALID_ARG;
    }
    if (!aligned16(out)) return MOM_ERR_ALIGNMENT;
    if (batch > 1 && (out_stride % 4 != 0 || out_stride < stored_elements(p->result_desc, sc && sc->out_packed ? MOM_STORAGE_PACKED : MOM_STORAGE_DENSE)))
        return MOM_ERR_INVALID_ARG;

    size_t need = 0;
    mom_plan_workspace_bytes(p, batch, &need);
    if (need > 0) {
        if (!workspace || workspace_bytes < need) return MOM_ERR_WORKSPACE_TOO_SMALL;
        if (reinterpret_cast<uintptr_t>(workspace) % WS_ALIGN != 0) return MOM_ERR_ALIGNMENT;
    }

    int device = 0;
    mom_status_t st = check_arch(&device);
    if (st != MOM_OK) return st;
    st = ensure_device_state(p, device);
    if (st != MOM_OK) return st;

    bool any_tc = false;
    for (const auto &s : p->steps) any_tc |= s.pub.uses_tensor_cores == 1;
    if (any_tc) {
        st = tc_prepare(*p, p->dev->tc);
        if (st != MOM_OK) return st;
    }

    // operands that are still being uploaded: wait (on the stream) before the first launch that reads them
    std::vector<char> slot_waited(n_ptrs, 0), add_waited(n_add, 0);
    auto need_slot = [&](int slot) {
        if (!staged || slot < 0 || slot_waited[slot] || p->ptr_desc[slot].property == MOM_IDENTITY || !p->slot_used[slot]) return;
        slot_waited[slot] = 1;
        cudaStreamWaitEvent(stream, staged->slot[slot], 0);
    };
    auto need_value = [&](int id) { if (id < n_chain) need_slot(p->factor_ptr[id]); };
    auto need_summands = [&](const SumInfo &sum) {
        if (!staged) return;
        for (const Summand &sm : sum.summands) {
            if (sm.kind == SUM_FACTOR) need_value(sm.index);
            if (sm.kind == SUM_TERM && !add_waited[sm.index] && p->add[sm.index].property != MOM_IDENTITY) {
                add_waited[sm.index] = 1;
                cudaStreamWaitEvent(stream, staged->add[sm.index], 0);
            }
        }
    };

    if (p->fused_ok) {
        for (int i = 0; i < n_ptrs; ++i) need_slot(i);
        need_summands(p->sums.back());
        BatchedChainPlan bp;
        if (batched_chain_plan(p, batch, chain_ptrs, chain_strides, add_ptrs, add_strides, out, out_stride, &bp, sc)) {
            // many instances of a right-nested chain: two warps per instance, operands streamed through registers
            if (launch_batched_chain(bp, stream) != cudaSuccess) return MOM_ERR_CUDA;
            p->last_launches = 1;
            return MOM_OK;
        }
        if (sc)                                               // the shared-memory kernel below reads dense operands only
            for (char in_place : sc->slot_packed)
                if (in_place) return MOM_ERR_INVALID_ARG;
        FusedPlan fp;
        std::memset(&fp, 0, sizeof(fp));
        fp.n_ops = (int)p->kept.size();
        DeviceState *dev = p->dev;
        if (dev->fused_tab_begin.empty()) {
            // first execute: the copy table of every operand that is read as stored in whole 16-byte pieces
            // (operand pointers and instance strides are 16-byte aligned, checked above)
            std::vector<uint2> table;
            dev->fused_tab_begin.assign(fp.n_ops, 0);
            dev->fused_tab_end.assign(fp.n_ops, 0);
            for (int i = 0; i < fp.n_ops; ++i) {
                const int id = p->kept[i];
                if (p->chain_t[id] || p->chain[id].cols % 4 != 0) continue;
                dev->fused_tab_begin[i] = (int)(table.size() / FUSED_THREADS);
                dev->fused_tab_end[i] = dev->fused_tab_begin[i] + fused_copy_table((int)p->chain[id].rows, (int)p->chain[id].cols, kernel_property(p->chain[id].property),
                                                                                    p->fused_value_off[id], p->fused_value_ld[id], table);
            }
            if (!table.empty()) {
                if (cudaMalloc(&dev->fused_table, table.size() * sizeof(uint2)) != cudaSuccess) return MOM_ERR_ALLOC;
                if (cudaMemcpy(dev->fused_table, table.data(), table.size() * sizeof(uint2), cudaMemcpyHostToDevice) != cudaSuccess) return MOM_ERR_CUDA;
            }
        }
        fp.copy_table = dev->fused_table;
        for (int i = 0; i < fp.n_ops; ++i) {
            const int id = p->kept[i], slot = p->factor_ptr[id];
            fp.ops[i] = FusedOperand{chain_ptrs[slot], chain_strides ? chain_strides[slot] : 0, (int)p->chain[id].rows,
                                     (int)p->chain[id].cols, kernel_property(p->chain[id].property), p->fused_value_off[id], p->fused_value_ld[id],
                                     (int)p->chain_t[id], dev->fused_tab_begin[i], dev->fused_tab_end[i]};
        }
        fp.n_steps = (int)p->steps.size();
        for (int s = 0; s < fp.n_steps; ++s) {
            const StepImpl &stp = p->steps[s];
            fp.steps[s] = FusedStep{p->fused_value_off[stp.pub.lhs], p->fused_value_off[stp.pub.rhs],
                                    stp.is_last ? -1 : p->fused_value_off[stp.pub.out], (int)stp.pub.m, (int)stp.pub.n,
                                    (int)stp.pub.k, kernel_property(stp.pub.lhs_property), kernel_property(stp.pub.rhs_property),
                                    kernel_property(stp.is_last ? p->result_desc.property : stp.pub.out_property),
                                    p->fused_value_ld[stp.pub.lhs], p->fused_value_ld[stp.pub.rhs],
                                    stp.is_last ? 0 : p->fused_value_ld[stp.pub.out]};
        }
        fp.add.count = n_add;
        fp.add.transposed = 0;
        fp.add.rows = (int)rows;
        for (int i = 0; i < n_add; ++i) {
            fp.add.ptr[i] = p->add[i].property == MOM_IDENTITY ? nullptr : add_ptrs[i];
            fp.add.stride[i] = add_strides ? add_strides[i] : 0;
            if (p->add_t[i]) fp.add.transposed |= 1u << i;
        }
        fp.out = out;
        fp.out_stride = out_stride;
        fp.batch = batch;
        fp.use_mma = p->variant != MOM_VARIANT_FFMA;
        if (launch_fused_small(fp, p->fused_smem_bytes, stream) != cudaSuccess) return MOM_ERR_CUDA;
        p->last_launches = 1;
        return MOM_OK;
    }

    int launches = 0;
    const int ns = (int)p->steps.size();
    const bool timing = p->step_timing && batch == 1;
    if (timing && p->dev->events.size() != (size_t)ns * 3 * TIMING_SLOTS) {
        for (cudaEvent_t e : p->dev->events) cudaEventDestroy(e);
        p->dev->timed_executes = 0;
        p->dev->events.assign((size_t)ns * 3 * TIMING_SLOTS, nullptr);
        for (auto &e : p->dev->events)
            if (cudaEventCreate(&e) != cudaSuccess) return MOM_ERR_CUDA;
    }
    // instances per pass: all of them when every step can take grid.z batching, else one at a time
    const int64_t group = any_tc ? 1 : (batch < 65535 ? batch : 65535);
    char *const ws = static_cast<char *>(workspace);

    for (int64_t b0 = 0; b0 < batch; b0 += group) {
        const int nb = (int)((batch - b0 < group) ? batch - b0 : group);
        // a factor: a stored matrix of the caller, or the temporary of a nested sum (instance-major in the workspace)
        auto chain_op = [&](int id) {
            if (p->factor_sum[id] >= 0) {
                const SumInfo &t = p->sums[p->factor_sum[id]];
                return Operand{reinterpret_cast<const float *>(ws + t.out_off * (size_t)nb), (long long)(t.desc.rows * t.desc.cols)};
            }
            const int slot = p->factor_ptr[id];
            const long long s = chain_strides ? chain_strides[slot] : 0;
            return Operand{chain_ptrs[slot] ? chain_ptrs[slot] + b0 * s : nullptr, s};
        };

        for (size_t si = 0; si < p->sums.size(); ++si) {
            const SumInfo &sum = p->sums[si];
            const bool top = si + 1 == p->sums.size();
            const int srows = (int)sum.desc.rows, scols = (int)sum.desc.cols;
            // where this sum's value goes: X, or the temporary
            float *x = top ? out + b0 * out_stride : reinterpret_cast<float *>(ws + sum.out_off * (size_t)nb);
            const long long x_stride = top ? out_stride : (long long)srows * scols;

            std::vector<const Summand *> simple;     // summands that are not products, in the order written
            bool has_products = false;
            for (const Summand &sm : sum.summands) {
                if (sm.kind == SUM_STEP) has_products = true;
                else simple.push_back(&sm);
            }
            const int n_simple = (int)simple.size();
            auto is_identity = [&](const Summand &sm) {
                return sm.kind == SUM_IDENTITY || (sm.kind == SUM_TERM && p->add[sm.index].property == MOM_IDENTITY);
            };
            // `simple[first..]` go into `t`, at most MAX_FUSED_ADD of them; returns the next index
            auto add_terms = [&](int first, AddTerms *t) {
                t->count = 0;
                t->transposed = 0;
                t->aliases_out = 0;
                t->rows = srows;
                int i = first;
                for (; i < n_simple && t->count < MAX_FUSED_ADD; ++i, ++t->count) {
                    const Summand &sm = *simple[i];
                    if (is_identity(sm)) {
                        t->ptr[t->count] = nullptr;
                        t->stride[t->count] = 0;
                    } else if (sm.kind == SUM_TERM) {
                        const long long s = add_strides ? add_strides[sm.index] : 0;
                        t->ptr[t->count] = add_ptrs[sm.index] + b0 * s;
                        t->stride[t->count] = s;
                        if (p->add_t[sm.index]) t->transposed |= 1u << t->count;
                    } else {
                        const Operand o = chain_op(sm.index);
                        t->ptr[t->count] = o.ptr;
                        t->stride[t->count] = o.stride;
                        if (p->chain_t[sm.index]) t->transposed |= 1u << t->count;
                    }
                }
                return i;
            };
            int added = 0;

            if (!has_products) {
                need_summands(sum);
                // value = first summand + the following ones
                const Summand &sm = *simple[0];
                AddTerms t;
                added = add_terms(1, &t);
                cudaError_t e;
                if (is_identity(sm)) {
                    e = launch_elementwise(nullptr, 0, 1, x, x_stride, srows, scols, kernel_property(sum.desc.property), t, nb, stream);
                } else if (sm.kind == SUM_FACTOR) {
                    const Operand src = chain_op(sm.index);
                    e = launch_elementwise(src.ptr, src.stride, p->chain_t[sm.index] ? 3 : 0, x, x_stride, srows, scols, kernel_property(sum.desc.property), t, nb, stream);
                } else {
                    const long long ss = add_strides ? add_strides[sm.index] : 0;
                    e = launch_elementwise(add_ptrs[sm.index] + b0 * ss, ss, p->add_t[sm.index] ? 3 : 0, x, x_stride, srows, scols, kernel_property(sum.desc.property), t, nb, stream);
                }
                if (e != cudaSuccess) return MOM_ERR_CUDA;
                ++launches;
            }

            // the order in which the steps are enqueued, and on which stream: normally as planned, all on the caller's stream; with two
            // independent subtrees of small products the right one goes first, onto the plan's side stream, and the step that needs both
            // waits for it (one instance, device operands, no per-step timing: the other cases keep the plain order)
            const bool side_by_side = p->side_join >= sum.step_begin && p->side_join < sum.step_end && batch == 1 && !staged && !timing;
            std::vector<int> order;
            for (int s = sum.step_begin; s < sum.step_end; ++s)
                if (side_by_side && s >= p->side_begin && s < p->side_end) order.push_back(s);
            for (int s = sum.step_begin; s < sum.step_end; ++s)
                if (!(side_by_side && s >= p->side_begin && s < p->side_end)) order.push_back(s);
            if (side_by_side) {
                DeviceState *dev = p->dev;
                if (!dev->side_stream) {
                    if (cudaStreamCreateWithFlags(&dev->side_stream, cudaStreamNonBlocking) != cudaSuccess) return MOM_ERR_CUDA;
                    if (cudaEventCreateWithFlags(&dev->side_fork, cudaEventDisableTiming) != cudaSuccess) return MOM_ERR_CUDA;
                    if (cudaEventCreateWithFlags(&dev->side_done, cudaEventDisableTiming) != cudaSuccess) return MOM_ERR_CUDA;
                }
                // the side stream starts where the caller's stream stands now (earlier work may still use the workspace)
                if (cudaEventRecord(dev->side_fork, stream) != cudaSuccess || cudaStreamWaitEvent(dev->side_stream, dev->side_fork, 0) != cudaSuccess)
                    return MOM_ERR_CUDA;
            }
            cudaStream_t const caller_stream = stream;
            for (int s : order) {
                const StepImpl &stp = p->steps[s];
                const bool on_side = side_by_side && s >= p->side_begin && s < p->side_end;
                cudaStream_t const stream = on_side ? p->dev->side_stream : caller_stream;      // shadows the caller's stream inside the step
                if (side_by_side && s == p->side_join && cudaStreamWaitEvent(caller_stream, p->dev->side_done, 0) != cudaSuccess) return MOM_ERR_CUDA;
                if (stp.folded) {                        // a scaling done by its reader's operand-split pass: nothing to launch
                    if (timing) {
                        cudaEvent_t *fe = &p->dev->events[((size_t)(p->dev->timed_executes % TIMING_SLOTS) * ns + s) * 3];
                        for (int q = 0; q < 3; ++q) cudaEventRecord(fe[q], stream);
                    }
                    continue;
                }
                auto value = [&](int id) {
                    if (id < n_chain) return chain_op(id);
                    const StepImpl &prod = p->steps[id - n_chain];
                    const long long elems = (long long)prod.pub.m * prod.pub.n;
                    // grid.z batching keeps one copy of each intermediate per instance, instance-major
                    // (a tensor-core step that feeds another one leaves no f32 intermediate: its consumer reads planes)
                    if (prod.out_off == SIZE_MAX) return Operand{nullptr, elems};
                    return Operand{reinterpret_cast<const float *>(ws + prod.out_off * (size_t)nb), elems};
                };
                if (stp.is_last && !stp.accumulate) need_summands(sum);
                ProductArgs a;
                std::memset(&a, 0, sizeof(a));
                a.m = (int)stp.pub.m; a.n = (int)stp.pub.n; a.k = (int)stp.pub.k;
                a.pa = kernel_property(stp.pub.lhs_property); a.pb = kernel_property(stp.pub.rhs_property);
                // an operand: the value itself, or d * S / S * d of a folded scaling step (S read as stored, d handed
                // to the split pass)
                // a left operand that arrives in two pieces: the first launch waits for its first rows only
                const int lhs_slot = stp.pub.lhs < n_chain ? p->factor_ptr[stp.pub.lhs] : -1;
                const bool lhs_in_pieces = staged && batch == 1 && stp.pub.uses_tensor_cores == 1 && lhs_slot >= 0 && !slot_waited[lhs_slot] &&
                                           stp.pub.rhs != stp.pub.lhs &&
                                           p->dev->tc.steps[s].split_a_by_part && staged->slot_head_rows[lhs_slot] == p->dev->tc.steps[s].part_row;
                auto operand = [&](int id, int fold, const float **ptr, long long *stride, int *trans, int own_trans,
                                   const float **scale, long long *scale_step, int *scale_rows, int *packed) {
                    if (fold < 0) {
                        if (!(lhs_in_pieces && id == stp.pub.lhs)) need_value(id);
                        const Operand o = value(id);
                        *ptr = o.ptr; *stride = o.stride; *trans = own_trans;
                        *packed = sc && id < n_chain && p->factor_ptr[id] >= 0 && sc->slot_packed[p->factor_ptr[id]];
                        return;
                    }
                    const mom_step_t &sc = p->steps[fold].pub;
                    const bool left = sc.lhs_property == MOM_DIAGONAL;          // d * S
                    const int s_id = left ? sc.rhs : sc.lhs, d_id = left ? sc.lhs : sc.rhs;
                    need_value(s_id);
                    need_value(d_id);
                    const Operand o = value(s_id), d = value(d_id);
                    *ptr = o.ptr; *stride = o.stride;
                    *trans = left ? sc.rhs_transposed : sc.lhs_transposed;
                    *scale = d.ptr; *scale_step = sc.k + 1; *scale_rows = left ? 1 : 0;
                };
                operand(stp.pub.lhs, stp.fold_a, &a.A, &a.strideA, &a.transA, stp.pub.lhs_transposed, &a.scaleA, &a.scaleA_step, &a.scaleA_rows, &a.packedA);
                operand(stp.pub.rhs, stp.fold_b, &a.B, &a.strideB, &a.transB, stp.pub.rhs_transposed, &a.scaleB, &a.scaleB_step, &a.scaleB_rows, &a.packedB);
                if ((a.packedA || a.packedB) && stp.pub.uses_tensor_cores != 1) return MOM_ERR_INVALID_ARG;   // only the split pass reads packed operands in place
                if (stp.is_last && stp.accumulate) {
                    // a later chain's product is added to what the earlier ones left in the sum's buffer
                    a.C = x; a.strideC = x_stride;
                    a.pout = kernel_property(sum.desc.property);
                    a.add.count = 1;
                    a.add.ptr[0] = x;
                    a.add.stride[0] = x_stride;
                    a.add.transposed = 0;
                    a.add.aliases_out = 1u;
                    a.add.rows = srows;
                } else if (stp.is_last) {
                    a.C = x; a.strideC = x_stride;
                    a.pout = kernel_property(sum.desc.property);
                    a.packedC = top && sc && sc->out_packed;
                    added = add_terms(0, &a.add);
                } else {
                    a.C = stp.out_off == SIZE_MAX ? nullptr : reinterpret_cast<float *>(ws + stp.out_off * (size_t)nb);
                    a.strideC = (long long)stp.pub.m * stp.pub.n;
                    a.pout = kernel_property(stp.pub.out_property);
                    a.add.count = 0;
                    a.add.transposed = 0;
                    a.add.aliases_out = 0;
                    a.add.rows = (int)stp.pub.m;
                }
                cudaEvent_t *ev = timing ? &p->dev->events[((size_t)(p->dev->timed_executes % TIMING_SLOTS) * ns + s) * 3] : nullptr;
                if (ev) cudaEventRecord(ev[0], stream);
                if (stp.pub.uses_tensor_cores == 1) {
                    int used = 0;
                    // the host-staging entry point copies the first rows of X back while the rest is still computed:
                    // the product that writes X then runs as two launches (only when nothing is added to X afterwards)
                    bool later_root = false;          // another chain's product is added to X after this one
                    for (int t = s + 1; t < sum.step_end; ++t) later_root |= p->steps[t].is_last;
                    const bool two_parts = staged && staged->first_rows && !a.packedC && top && stp.is_last && !stp.accumulate && !later_root &&
                                           added >= n_simple && batch == 1 && p->dev->tc.steps[s].part_row > 0;
                    if (lhs_in_pieces) {
                        if (cudaStreamWaitEvent(stream, staged->slot_head[lhs_slot], 0) != cudaSuccess) return MOM_ERR_CUDA;
                        st = tc_launch_step(*p, p->dev->tc, s, a, ws, p->dev->status, stream, &used, ev ? ev[1] : nullptr, 1);
                        if (st != MOM_OK) return st;
                        launches += used;
                        need_slot(lhs_slot);                                               // the whole operand
                        st = tc_launch_step(*p, p->dev->tc, s, a, ws, p->dev->status, stream, &used, nullptr, 2);
                    } else if (two_parts) {
                        st = tc_launch_step(*p, p->dev->tc, s, a, ws, p->dev->status, stream, &used, ev ? ev[1] : nullptr, 1);
                        if (st != MOM_OK) return st;
                        launches += used;
                        if (cudaEventRecord(staged->first_rows_done, stream) != cudaSuccess) return MOM_ERR_CUDA;
                        *staged->first_rows = p->dev->tc.steps[s].part_row;
                        st = tc_launch_step(*p, p->dev->tc, s, a, ws, p->dev->status, stream, &used, nullptr, 2);
                    } else {
                        st = tc_launch_step(*p, p->dev->tc, s, a, ws, p->dev->status, stream, &used, ev ? ev[1] : nullptr);
                    }
                    if (st != MOM_OK) return st;
                    launches += used;
                } else {
                    if (ev) cudaEventRecord(ev[1], stream);
                    cudaError_t e = cudaErrorNotSupported;
                    if (stp.pub.kind == MOM_KIND_SCALE) {
                        e = launch_scale(a, nb, stream);
                    } else if (stp.pub.uses_tensor_cores == 3 || stp.pub.uses_tensor_cores == 2) {
                        // the one-launch tcgen05 kernel takes one instance and 16-byte aligned operands; otherwise (and for
                        // batches) the warp-level kernel
                        if (stp.pub.uses_tensor_cores == 3 && nb == 1) e = launch_product_tc_inline(a, p->dev->status, stream);
                        if (e == cudaErrorNotSupported) e = launch_product_mma(a, nb, stream);
                    } else {
                        e = launch_product_ffma(a, nb, stream);
                    }
                    if (e != cudaSuccess) return MOM_ERR_CUDA;
                    ++launches;
                }
                if (ev) cudaEventRecord(ev[2], stream);
                if (on_side && s + 1 == p->side_end && cudaEventRecord(p->dev->side_done, stream) != cudaSuccess) return MOM_ERR_CUDA;
            }

            // summands beyond the fused limit: value += T, a few at a time, in place
            while (added < n_simple) {
                AddTerms t;
                const int first = added;
                added = add_terms(first, &t);
                if (launch_elementwise(nullptr, 0, 2, x, x_stride, srows, scols, kernel_property(sum.desc.property), t, nb, stream) != cudaSuccess)
                    return MOM_ERR_CUDA;
                ++launches;
            }
        }
    }
    if (timing) ++p->dev->timed_executes;
    p->last_launches = launches;
    return MOM_OK;
}


// The storage layer around execute_core: packed operands that no kernel of this plan reads in place are unpacked into
// dense copies behind the plan's own workspace, a packed X that is not written in place is computed dense there and
// packed at the end; everything else goes through untouched.
mom_status_t execute_impl(const mom_plan *p, const float *const *chain_ptrs, const int64_t *chain_strides,
                          const float *const *add_ptrs, const int64_t *add_strides, float *out, int64_t out_stride,
                          int64_t batch, void *workspace, size_t workspace_bytes, cudaStream_t stream,
                          const StageEvents *staged = nullptr) {
    if (!p) return MOM_ERR_INVALID_ARG;
    if (p->ptr_storage.empty() && p->result_storage == MOM_STORAGE_DENSE)
        return execute_core(p, chain_ptrs, chain_strides, add_ptrs, add_strides, out, out_stride, batch, workspace, workspace_bytes, stream, staged);
    if (!chain_ptrs || !out || batch < 1) return MOM_ERR_INVALID_ARG;
    const int n_ptrs = (int)p->ptr_desc.size(), n_add = (int)p->add.size();
    if (n_add > 0 && !add_ptrs) return MOM_ERR_INVALID_ARG;
    if (batch > 1 && (!chain_strides || (n_add > 0 && !add_strides))) return MOM_ERR_INVALID_ARG;
    if (batch > 65535) return MOM_ERR_LIMIT;                 // the packing passes take the instances in grid.z

    // every argument is checked before the first unpacking pass is enqueued
    auto packed_size = [](const mom_matrix_desc_t &d) { return stored_elements(d, MOM_STORAGE_PACKED); };
    for (int i = 0; i < n_ptrs; ++i) {
        if (slot_storage(*p, i) != MOM_STORAGE_PACKED || !p->slot_used[i]) continue;
        if (!chain_ptrs[i]) return MOM_ERR_INVALID_ARG;
        if (!aligned16(chain_ptrs[i])) return MOM_ERR_ALIGNMENT;
        if (batch > 1 && (chain_strides[i] % 4 != 0 || chain_strides[i] < packed_size(p->ptr_desc[i]))) return MOM_ERR_INVALID_ARG;
    }
    for (int i = 0; i < n_add; ++i) {
        if (term_storage(*p, i) != MOM_STORAGE_PACKED) continue;
        if (!add_ptrs[i]) return MOM_ERR_INVALID_ARG;
        if (!aligned16(add_ptrs[i])) return MOM_ERR_ALIGNMENT;
        if (batch > 1 && (add_strides[i] % 4 != 0 || add_strides[i] < packed_size(p->add[i]))) return MOM_ERR_INVALID_ARG;
    }
    if (!aligned16(out)) return MOM_ERR_ALIGNMENT;
    if (p->result_storage == MOM_STORAGE_PACKED && batch > 1 && (out_stride % 4 != 0 || out_stride < packed_size(p->result_desc)))
        return MOM_ERR_INVALID_ARG;
    size_t need = 0;
    mom_plan_workspace_bytes(p, batch, &need);
    if (need > 0) {
        if (!workspace || workspace_bytes < need) return MOM_ERR_WORKSPACE_TOO_SMALL;
        if (reinterpret_cast<uintptr_t>(workspace) % WS_ALIGN != 0) return MOM_ERR_ALIGNMENT;
    }
    int device = 0;
    mom_status_t st = check_arch(&device);
    if (st != MOM_OK) return st;

    const StorageLayout layout = storage_layout(*p, batch);
    char *const region = static_cast<char *>(workspace) + (need - layout.bytes);
    StorageCall sc;
    sc.slot_packed.assign(n_ptrs, 0);
    std::vector<const float *> cptr(chain_ptrs, chain_ptrs + n_ptrs), aptr(n_add, nullptr);
    std::vector<int64_t> cstride(n_ptrs, 0), astride(n_add, 0);
    for (int i = 0; i < n_ptrs; ++i) cstride[i] = chain_strides ? chain_strides[i] : 0;
    for (int i = 0; i < n_add; ++i) { aptr[i] = add_ptrs[i]; astride[i] = add_strides ? add_strides[i] : 0; }

    // which packed operands are read in place (the same rule that sized the workspace)
    for (int i = 0; i < n_ptrs; ++i) sc.slot_packed[i] = storage_in_place(*p, i, batch);

    int extra_launches = 0;
    for (int i = 0; i < n_ptrs; ++i) {
        if (slot_storage(*p, i) != MOM_STORAGE_PACKED || !p->slot_used[i] || sc.slot_packed[i]) continue;
        if (layout.slot_off[i] == SIZE_MAX) return MOM_ERR_INVALID_ARG;
        if (staged && cudaStreamWaitEvent(stream, staged->slot[i], 0) != cudaSuccess) return MOM_ERR_CUDA;
        const mom_matrix_desc_t &d = p->ptr_desc[i];
        float *dense = reinterpret_cast<float *>(region + layout.slot_off[i]);
        if (launch_unpack(cptr[i], cstride[i], dense, dense_copy_stride(d), (int)d.rows, is_lower_kind(d.property), (int)batch, stream) != cudaSuccess)
            return MOM_ERR_CUDA;
        ++extra_launches;
        cptr[i] = dense;
        cstride[i] = dense_copy_stride(d);
    }
    if (!p->names.empty())                                   // entries with one name stay one matrix after the substitution
        for (int i = 0; i < n_ptrs; ++i)
            for (int j = 0; j < i; ++j)
                if (p->names[i] == p->names[j] && chain_ptrs[i] == chain_ptrs[j] && p->slot_used[i] && p->slot_used[j]) { cptr[i] = cptr[j]; cstride[i] = cstride[j]; }
    for (int i = 0; i < n_add; ++i) {
        if (term_storage(*p, i) != MOM_STORAGE_PACKED) continue;
        if (staged && cudaStreamWaitEvent(stream, staged->add[i], 0) != cudaSuccess) return MOM_ERR_CUDA;
        const mom_matrix_desc_t &d = p->add[i];
        float *dense = reinterpret_cast<float *>(region + layout.add_off[i]);
        if (launch_unpack(aptr[i], astride[i], dense, dense_copy_stride(d), (int)d.rows, is_lower_kind(d.property), (int)batch, stream) != cudaSuccess)
            return MOM_ERR_CUDA;
        ++extra_launches;
        aptr[i] = dense;
        astride[i] = dense_copy_stride(d);
    }
    float *x = out;
    int64_t x_stride = out_stride;
    const mom_matrix_desc_t &rd = p->result_desc;
    if (p->result_storage == MOM_STORAGE_PACKED) {
        if (p->result_native) {
            sc.out_packed = true;
        } else {
            x = reinterpret_cast<float *>(region + layout.x_off);
            x_stride = dense_copy_stride(rd);
        }
    }
    st = execute_core(p, cptr.data(), cstride.data(), aptr.data(), astride.data(), x, x_stride, batch, workspace, workspace_bytes, stream, staged, &sc);
    if (st != MOM_OK) return st;
    if (x != out) {
        if (launch_pack(x, x_stride, out, out_stride, (int)rd.rows, is_lower_kind(rd.property), (int)batch, stream) != cudaSuccess) return MOM_ERR_CUDA;
        ++extra_launches;
    }
    p->last_launches += extra_launches;
    return MOM_OK;
}

}  // namespace
}  // namespace mom

extern "C" {

mom_status_t mom_equation_execute(const mom_plan_t *plan, const float *const *chain_ptrs,
                                  const float *const *add_ptrs, float *out,
                                  void *workspace, size_t workspace_bytes, mom_stream_t stream) {
    if (!plan) return MOM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(plan->exec_mutex);
    return mom::execute_impl(plan, chain_ptrs, nullptr, add_ptrs, nullptr, out, 0, 1, workspace, workspace_bytes,
                             reinterpret_cast<cudaStream_t>(stream));
}

mom_status_t mom_equation_execute_batched(const mom_plan_t *plan, const float *const *chain_ptrs,
                                          const int64_t *chain_strides, const float *const *add_ptrs,
                                          const int64_t *add_strides, float *out, int64_t out_stride,
                                          int64_t batch, void *workspace, size_t workspace_bytes,
                                          mom_stream_t stream) {
    if (!plan) return MOM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(plan->exec_mutex);
    return mom::execute_impl(plan, chain_ptrs, chain_strides, add_ptrs, add_strides, out, out_stride, batch,
                             workspace, workspace_bytes, reinterpret_cast<cudaStream_t>(stream));
}

mom_status_t mom_equation_execute_host(const mom_plan_t *plan, const float *const *chain_host,
                                       const float *const *add_host, float *out_host, int64_t batch,
                                       void *staging, size_t staging_bytes, mom_stream_t stream_) {
    if (!plan || !chain_host || !out_host || batch < 1) return MOM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(plan->exec_mutex);
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    size_t need = 0;
    mom_plan_host_staging_bytes(plan, batch, &need);
    if (!staging || staging_bytes < need) return MOM_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(staging) % mom::WS_ALIGN != 0) return MOM_ERR_ALIGNMENT;
    const int n_chain = (int)plan->ptr_desc.size(), n_add = (int)plan->add.size();
    if (n_add > 0 && !add_host) return MOM_ERR_INVALID_ARG;
    // every argument error is found here, before the first copy is enqueued
    std::vector<int> same_as(n_chain, -1);
    bool strides_ok = mom::stored_elements(plan->result_desc, plan->result_storage) % 4 == 0;
    for (int i = 0; i < n_chain; ++i) {
        const mom_matrix_desc_t &d = plan->ptr_desc[i];
        if (d.property == MOM_IDENTITY) continue;
        if (!plan->names.empty())                        // a named matrix is one buffer, copied once
            for (int j = 0; j < i && same_as[i] < 0; ++j)
                if (plan->names[j] == plan->names[i]) same_as[i] = j;
        if (same_as[i] >= 0) {
            if (chain_host[i] != chain_host[same_as[i]]) return MOM_ERR_INVALID_ARG;
            continue;
        }
        if (!plan->slot_used[i]) continue;
        if (!chain_host[i]) return MOM_ERR_INVALID_ARG;
        strides_ok &= mom::stored_elements(d, mom::slot_storage(*plan, i)) % 4 == 0;
    }
    for (int i = 0; i < n_add; ++i) {
        if (plan->add[i].property == MOM_IDENTITY) continue;
        if (!add_host[i]) return MOM_ERR_INVALID_ARG;
        strides_ok &= mom::stored_elements(plan->add[i], mom::term_storage(*plan, i)) % 4 == 0;
    }
    // instance strides that are not multiples of 4 elements cannot be batched in place
    if (batch > 1 && !strides_ok) return MOM_ERR_ALIGNMENT;

    int device = 0;
    mom_status_t est = mom::check_arch(&device);
    if (est != MOM_OK) return est;
    est = mom::ensure_device_state(plan, device);
    if (est != MOM_OK) return est;
    mom::DeviceState *dev = plan->dev;
    if (!dev->copy_stream) {
        if (cudaStreamCreateWithFlags(&dev->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return MOM_ERR_CUDA;
        if (cudaStreamCreateWithFlags(&dev->back_stream, cudaStreamNonBlocking) != cudaSuccess) return MOM_ERR_CUDA;
        if (cudaEventCreateWithFlags(&dev->call_start, cudaEventDisableTiming) != cudaSuccess) return MOM_ERR_CUDA;
        if (cudaEventCreateWithFlags(&dev->first_rows_done, cudaEventDisableTiming) != cudaSuccess) return MOM_ERR_CUDA;
        if (cudaEventCreateWithFlags(&dev->back_done, cudaEventDisableTiming) != cudaSuccess) return MOM_ERR_CUDA;
    }
    bool any_tc = false;
    for (const auto &s : plan->steps) any_tc |= s.pub.uses_tensor_cores == 1;
    if (any_tc) {
        est = mom::tc_prepare(*plan, dev->tc);
        if (est != MOM_OK) return est;
    }
    while ((int)dev->slot_head.size() < n_chain) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return MOM_ERR_CUDA;
        dev->slot_head.push_back(e);
    }
    while ((int)dev->slot_ready.size() < n_chain || (int)dev->add_ready.size() < n_add) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return MOM_ERR_CUDA;
        ((int)dev->slot_ready.size() < n_chain ? dev->slot_ready : dev->add_ready).push_back(e);
    }
    // From here on copies from the caller's host buffers may be in flight: an error return first waits for them, so
    // that the caller may free or reuse those buffers (and the staging area) as soon as the call has returned.
    auto enqueue = [&]() -> mom_status_t {
        // uploads start once the caller's stream has reached this call (the staging area may still be in use before)
        if (cudaEventRecord(dev->call_start, stream) != cudaSuccess) return MOM_ERR_CUDA;
        if (cudaStreamWaitEvent(dev->copy_stream, dev->call_start, 0) != cudaSuccess) return MOM_ERR_CUDA;

        char *cur = static_cast<char *>(staging);
        std::vector<const float *> cptr(n_chain, nullptr), aptr(n_add, nullptr);
        std::vector<int64_t> cstride(n_chain, 0), astride(n_add, 0);
        std::vector<size_t> cbytes(n_chain, 0);
        for (int i = 0; i < n_chain; ++i) {                  // addresses in the staging area, in the order given
            const mom_matrix_desc_t &d = plan->ptr_desc[i];
            if (d.property == MOM_IDENTITY) continue;
            if (same_as[i] >= 0) {                           // a named matrix is copied once
                cptr[i] = cptr[same_as[i]];
                cstride[i] = cstride[same_as[i]];
                continue;
            }
            if (!plan->slot_used[i]) continue;               // an operand no factor refers to is not uploaded
            cbytes[i] = (size_t)mom::stored_elements(d, mom::slot_storage(*plan, i)) * sizeof(float) * batch;
            cptr[i] = reinterpret_cast<const float *>(cur);
            cstride[i] = mom::stored_elements(d, mom::slot_storage(*plan, i));
            cur += mom::align_up(cbytes[i], mom::WS_ALIGN);
        }
        // upload in the order of first use by the plan's products, so that the first products can start early
        std::vector<int> first_use(n_chain, (int)plan->steps.size());
        for (size_t s = 0; s < plan->steps.size(); ++s)
            for (int32_t v : {plan->steps[s].pub.lhs, plan->steps[s].pub.rhs})
                if (v < (int32_t)plan->factor_ptr.size() && plan->factor_ptr[v] >= 0)
                    first_use[plan->factor_ptr[v]] = std::min(first_use[plan->factor_ptr[v]], (int)s);
        for (int i = 0; i < n_chain; ++i)                    // a matrix given under several entries is needed when the first is
            if (same_as[i] >= 0) first_use[same_as[i]] = std::min(first_use[same_as[i]], first_use[i]);
        std::vector<int> order(n_chain);
        for (int i = 0; i < n_chain; ++i) order[i] = i;
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return first_use[a] < first_use[b]; });
        // a general operand that a tensor-core product inside the plan reads as its left factor in two row ranges travels in
        // two pieces, with an event between them: that product starts on the first rows while the others are on their way
        std::vector<int> head_rows(n_chain, 0);
        if (any_tc && batch == 1)
            for (size_t s = 0; s < plan->steps.size(); ++s) {
                const int32_t v = plan->steps[s].pub.lhs;
                if (!dev->tc.steps[s].split_a_by_part || v >= (int32_t)plan->factor_ptr.size()) continue;
                const int slot = plan->factor_ptr[v];
                if (slot >= 0 && same_as[slot] < 0 && cbytes[slot] && first_use[slot] == (int)s && !mom::triangular_upload(plan->ptr_desc[slot], batch) && mom::slot_storage(*plan, slot) == MOM_STORAGE_DENSE)
                    head_rows[slot] = dev->tc.steps[s].part_row;
            }
        for (int i : order) {
            if (same_as[i] >= 0) continue;
            if (cbytes[i] && head_rows[i] > 0) {
                const size_t head = (size_t)head_rows[i] * plan->ptr_desc[i].cols * sizeof(float);
                char *dst = reinterpret_cast<char *>(const_cast<float *>(cptr[i]));
                const char *src = reinterpret_cast<const char *>(chain_host[i]);
                if (cudaMemcpyAsync(dst, src, head, cudaMemcpyHostToDevice, dev->copy_stream) != cudaSuccess) return MOM_ERR_CUDA;
                if (cudaEventRecord(dev->slot_head[i], dev->copy_stream) != cudaSuccess) return MOM_ERR_CUDA;
                if (cudaMemcpyAsync(dst + head, src + head, cbytes[i] - head, cudaMemcpyHostToDevice, dev->copy_stream) != cudaSuccess) return MOM_ERR_CUDA;
            } else if (cbytes[i] && mom::triangular_upload(plan->ptr_desc[i], batch, mom::slot_storage(*plan, i))) {
                // a large triangular operand: the host buffer holds zeros outside the triangle (storage contract), so
                // only the 256-row blocks' columns up to (from) the diagonal block cross the bus; the rest is zero-filled here
                const mom_matrix_desc_t &d = plan->ptr_desc[i];
                float *dst = const_cast<float *>(cptr[i]);
                const int64_t n = d.rows;
                if (cudaMemsetAsync(dst, 0, cbytes[i], dev->copy_stream) != cudaSuccess) return MOM_ERR_CUDA;
                for (int64_t r0 = 0; r0 < n; r0 += mom::UPLOAD_BLOCK) {
                    const int64_t r1 = std::min(n, r0 + mom::UPLOAD_BLOCK);
                    const bool lower = mom::kernel_property(d.property) == MOM_LOWER_TRI;
                    const int64_t c0 = lower ? 0 : r0, c1 = lower ? r1 : n;
                    if (cudaMemcpy2DAsync(dst + r0 * n + c0, (size_t)n * sizeof(float), chain_host[i] + r0 * n + c0, (size_t)n * sizeof(float),
                                          (size_t)(c1 - c0) * sizeof(float), (size_t)(r1 - r0), cudaMemcpyHostToDevice, dev->copy_stream) != cudaSuccess)
                        return MOM_ERR_CUDA;
                }
            } else if (cbytes[i] && cudaMemcpyAsync(const_cast<float *>(cptr[i]), chain_host[i], cbytes[i], cudaMemcpyHostToDevice, dev->copy_stream) != cudaSuccess)
                return MOM_ERR_CUDA;
            if (cudaEventRecord(dev->slot_ready[i], dev->copy_stream) != cudaSuccess) return MOM_ERR_CUDA;
            for (int j = i + 1; j < n_chain; ++j)
                if (same_as[j] == i && cudaEventRecord(dev->slot_ready[j], dev->copy_stream) != cudaSuccess) return MOM_ERR_CUDA;
        }
        for (int i = 0; i < n_add; ++i) {
            const mom_matrix_desc_t &d = plan->add[i];
            if (d.property == MOM_IDENTITY) continue;
            const size_t bytes = (size_t)mom::stored_elements(d, mom::term_storage(*plan, i)) * sizeof(float) * batch;
            if (cudaMemcpyAsync(cur, add_host[i], bytes, cudaMemcpyHostToDevice, dev->copy_stream) != cudaSuccess) return MOM_ERR_CUDA;
            if (cudaEventRecord(dev->add_ready[i], dev->copy_stream) != cudaSuccess) return MOM_ERR_CUDA;
            aptr[i] = reinterpret_cast<const float *>(cur);
            astride[i] = mom::stored_elements(d, mom::term_storage(*plan, i));
            cur += mom::align_up(bytes, mom::WS_ALIGN);
        }
        int first_rows = 0;
        const mom::StageEvents staged{dev->slot_ready.data(), dev->add_ready.data(), dev->first_rows_done,
                                      plan->result_storage == MOM_STORAGE_DENSE ? &first_rows : nullptr,
                                      dev->slot_head.data(), head_rows.data()};
        float *x = reinterpret_cast<float *>(cur);
        const int64_t xelems = mom::stored_elements(plan->result_desc, plan->result_storage);
        const size_t xbytes = (size_t)xelems * sizeof(float) * batch;
        cur += mom::align_up(xbytes, mom::WS_ALIGN);
        size_t ws_bytes = 0;
        mom_plan_workspace_bytes(plan, batch, &ws_bytes);
        mom_status_t st = MOM_OK;
        if (batch == 1) {
            st = mom::execute_impl(plan, cptr.data(), nullptr, aptr.data(), nullptr, x, 0, 1, cur, ws_bytes, stream, &staged);
        } else {
            st = mom::execute_impl(plan, cptr.data(), cstride.data(), aptr.data(), astride.data(), x, xelems, batch, cur, ws_bytes, stream, &staged);
        }
        if (st != MOM_OK) return st;
        if (first_rows > 0) {
            // the first rows of X are final before the last launch ends: they travel on a stream of their own meanwhile
            const size_t head = (size_t)first_rows * plan->result_desc.cols * sizeof(float);
            if (cudaStreamWaitEvent(dev->back_stream, dev->first_rows_done, 0) != cudaSuccess) return MOM_ERR_CUDA;
            if (cudaMemcpyAsync(out_host, x, head, cudaMemcpyDeviceToHost, dev->back_stream) != cudaSuccess) return MOM_ERR_CUDA;
            if (cudaEventRecord(dev->back_done, dev->back_stream) != cudaSuccess) return MOM_ERR_CUDA;
            if (cudaMemcpyAsync(reinterpret_cast<char *>(out_host) + head, reinterpret_cast<char *>(x) + head, xbytes - head,
                                cudaMemcpyDeviceToHost, stream) != cudaSuccess) return MOM_ERR_CUDA;
            if (cudaStreamWaitEvent(stream, dev->back_done, 0) != cudaSuccess) return MOM_ERR_CUDA;
        } else if (cudaMemcpyAsync(out_host, x, xbytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess) {
            return MOM_ERR_CUDA;
        }
        return MOM_OK;
    };
    const mom_status_t status = enqueue();
    if (status != MOM_OK) {
        cudaStreamSynchronize(dev->copy_stream);
        cudaStreamSynchronize(dev->back_stream);
        cudaStreamSynchronize(stream);
        return status;
    }
    if (cudaStreamSynchronize(stream) != cudaSuccess) return MOM_ERR_CUDA;
    return MOM_OK;
}

mom_status_t mom_plan_host_upload_bytes(const mom_plan_t *plan, int64_t batch, size_t *bytes) {
    if (!plan || !bytes || batch < 1) return MOM_ERR_INVALID_ARG;
    size_t total = 0;
    const int n = (int)plan->ptr_desc.size();
    for (int i = 0; i < n; ++i) {
        const mom_matrix_desc_t &d = plan->ptr_desc[i];
        if (d.property == MOM_IDENTITY || !plan->slot_used[i]) continue;
        bool seen = false;                               // a named matrix is copied once
        if (!plan->names.empty())
            for (int j = 0; j < i && !seen; ++j) seen = plan->names[j] == plan->names[i] && plan->slot_used[j];
        if (!seen) total += mom::upload_bytes(d, batch, mom::slot_storage(*plan, i));
    }
    for (size_t i = 0; i < plan->add.size(); ++i) {
        const auto &d = plan->add[i];
        if (d.property != MOM_IDENTITY) total += (size_t)mom::stored_elements(d, mom::term_storage(*plan, (int)i)) * sizeof(float) * batch;
    }
    *bytes = total;
    return MOM_OK;
}

mom_status_t mom_plan_enable_step_timing(mom_plan_t *plan, int32_t enable) {
    if (!plan) return MOM_ERR_INVALID_ARG;
    plan->step_timing = enable != 0;
    if (plan->dev) plan->dev->timed_executes = 0;
    return MOM_OK;
}

mom_status_t mom_plan_step_times(const mom_plan_t *plan, int32_t i, float *product_ms, float *prepass_ms) {
    if (!plan || i < 0 || i >= (int32_t)plan->steps.size()) return MOM_ERR_INVALID_ARG;
    const size_t ns = plan->steps.size();
    if (!plan->dev || plan->dev->events.size() != ns * 3 * mom::TIMING_SLOTS || plan->dev->timed_executes < 1) return MOM_ERR_INVALID_ARG;
    const long long have = plan->dev->timed_executes < mom::TIMING_SLOTS ? plan->dev->timed_executes : mom::TIMING_SLOTS;
    float pre = 0.0f, prod = 0.0f;
    for (long long slot = 0; slot < have; ++slot) {        // mean over the recorded executes (the most recent ring-full)
        cudaEvent_t *ev = &plan->dev->events[((size_t)slot * ns + i) * 3];
        float a = 0.0f, b = 0.0f;
        if (cudaEventElapsedTime(&a, ev[0], ev[1]) != cudaSuccess) return MOM_ERR_CUDA;
        if (cudaEventElapsedTime(&b, ev[1], ev[2]) != cudaSuccess) return MOM_ERR_CUDA;
        pre += a;
        prod += b;
    }
    pre /= (float)have;
    prod /= (float)have;
    if (product_ms) *product_ms = prod;
    if (prepass_ms) *prepass_ms = pre;
    return MOM_OK;
}

mom_status_t mom_probe_wait_timeout(const mom_plan_t *plan, double limit_ms, int32_t detail, mom_stream_t stream) {
    if (!plan || !(limit_ms > 0.0) || limit_ms > 1000.0) return MOM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(plan->exec_mutex);
    int device = 0;
    mom_status_t st = mom::check_arch(&device);
    if (st != MOM_OK) return st;
    st = mom::ensure_device_state(plan, device);
    if (st != MOM_OK) return st;
    const unsigned long long limit_ns = (unsigned long long)(limit_ms * 1.0e6);
    return mom::launch_wait_timeout_probe(plan->dev->status, limit_ns, detail, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess
               ? MOM_OK : MOM_ERR_CUDA;
}

mom_status_t mom_plan_device_status(const mom_plan_t *plan, int32_t *code, int32_t *detail) {
    if (!plan || !code) return MOM_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(plan->exec_mutex);
    int32_t host[4] = {0, 0, 0, 0};
    if (plan->dev && plan->dev->status) {
        if (cudaMemcpy(host, plan->dev->status, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess) return MOM_ERR_CUDA;
        if (host[0] != 0 && cudaMemset(plan->dev->status, 0, sizeof(host)) != cudaSuccess) return MOM_ERR_CUDA;
    }
    *code = host[0];
    if (detail) *detail = host[1];
    return MOM_OK;
}

}  // extern "C"
