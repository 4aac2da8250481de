// Batched small equations whose plan is a right-nested chain with a narrow right end,
//     X_i = M_S * ( ... (M_2 * (M_1 * B_i)) ... ) + T_1 + ... + T_t          (thousands of instances i),
// every M at most 64 x 64 (multiples of 16) and B, the intermediates and X at most 16 columns wide.
//
// The work is bound by HBM traffic (a few flops per byte), so the kernel is built around the loads:
//   - Two warps own one instance and nothing is shared beyond that pair: no block-wide barrier anywhere.  A pair
//     meets once per product, on a 64-thread named barrier, when the intermediate changes hands.
//   - The left factors never pass through shared memory.  A thread fetches them from global memory straight into
//     the registers it will feed to the warp-level MMA (m16n8k8, tf32): the contraction index inside each group
//     of 16 columns is renumbered so that thread t of a quad owns columns 4t .. 4t+3 of its rows g and g+8 --
//     one 16-byte load per row, every 32-byte sector fully used -- and the right operand's fragments follow the
//     same renumbering.  The loads of the next product's (or the next instance's) left factor are issued before
//     the current block is multiplied, so each warp keeps up to sixteen 16-byte loads in flight all the time.
//   - The right end B of the NEXT instance is copied asynchronously (cp.async) into a 4.5 KB shared-memory buffer of
//     the pair while the current instance is multiplied; an intermediate is written to such a buffer in accumulator
//     layout; both are read back as right fragments (rows padded by two floats: conflict-free).
//   - Blocks of 16 x 16 that lie outside a triangular factor's structure are neither loaded nor multiplied.
//   - 3xTF32 on the fragments: a = hi + lo, accumulate lo*hi + hi*lo + hi*hi in f32 (hi rounded to tf32 on the bit
//     pattern; lo = a - hi handed over unrounded: the MMA ignores the bits below tf32, worth at most 2^-21 of a,
//     the size of the lo*lo term this scheme omits anyway).
// The per-instance problem is far too small for a tcgen05 / tensor-memory pipeline; the legacy warp-level MMA is
// used on purpose.
#include <algorithm>
#include <mutex>
#include <type_traits>

#include "batched_chain.h"
#include "device_info.h"
#include "packed.cuh"

namespace mom {

namespace {

constexpr int BC_THREADS = 128;                 // four warps: two instances in flight per CTA
constexpr int BC_PAIRS = BC_THREADS / 64;
constexpr int BC_CTAS_PER_SM = 4;
constexpr int T_PAD = 2;                        // extra floats per row of an intermediate in shared memory
constexpr int T_FLOATS = BC_MAX_DIM * (BC_MAX_N + T_PAD);

__device__ __forceinline__ float4 load_once_f4(const float *p) {     // streamed data: keep it out of L1
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void copy_async_8(float *dst_shared, const float *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_shared)), "l"(src) : "memory");
}
__device__ __forceinline__ void copy_async_wait_all() {
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ float2 load_once_f2(const float *p) {
    float2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ void pair_barrier(int pair) {
    asm volatile("bar.sync %0, 64;" ::"r"(pair + 1) : "memory");
}
__device__ __forceinline__ void split_tf32(float a, uint32_t &hi, uint32_t &lo) {
    hi = (__float_as_uint(a) + 0x1000u) & 0xFFFFE000u;
    lo = __float_as_uint(a - __uint_as_float(hi));
}
__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// NT: 8-column tiles of the right operand (n = 8 NT).
template <int NT>
__global__ void __launch_bounds__(BC_THREADS, BC_CTAS_PER_SM)
batched_chain_kernel(const BatchedChainPlan bp) {
    __shared__ __align__(16) float tbuf[BC_PAIRS][2][T_FLOATS];      // intermediates: product s reads [s & 1], writes [(s + 1) & 1]
    __shared__ __align__(16) float bbuf[BC_PAIRS][2][T_FLOATS];      // the right end B of this instance and of the next
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int pair = warp >> 1, w = warp & 1;
    constexpr int LD = 8 * NT + T_PAD;
    const int S = bp.n_steps;
    const long long pairs_total = (long long)gridDim.x * BC_PAIRS;
    long long inst = (long long)blockIdx.x * BC_PAIRS + pair;

    float4 buf[2][4][2];             // [slot][16-column chunk][row g / row g + 8] of the left factor

    // 16-byte loads of one row block of a left factor (only the chunks that its structure needs)
    auto issue_lhs = [&](auto slot, int s, long long at) {
        constexpr int q = decltype(slot)::value;
        const BatchedChainStep &st = bp.steps[s];
        const int rb = st.rb[w][q];
        if (rb < 0) return;
        const unsigned mask = st.chunks[w][q];
        if (st.packed) {
            // a packed triangle: each row's stored columns start at its own offset; what the container does not hold
            // (beyond the diagonal's group of four) is zero and is not loaded
            const PackedRow p0 = packed_row(st.packed == 1, st.m, 16 * rb + g), p1 = packed_row(st.packed == 1, st.m, 16 * rb + g + 8);
            const float *row0 = st.lhs + at * st.lhs_stride + p0.offset - p0.first, *row1 = st.lhs + at * st.lhs_stride + p1.offset - p1.first;
#pragma unroll
            for (int c = 0; c < 4; ++c)
                if ((mask >> c) & 1u) {
                    const int col = 16 * c + 4 * t;
                    if (c != rb) {                           // a block off the diagonal is stored in full
                        buf[q][c][0] = load_once_f4(row0 + col);
                        buf[q][c][1] = load_once_f4(row1 + col);
                    } else {
                        buf[q][c][0] = col >= p0.first && col < p0.end ? load_once_f4(row0 + col) : make_float4(0.f, 0.f, 0.f, 0.f);
                        buf[q][c][1] = col >= p1.first && col < p1.end ? load_once_f4(row1 + col) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            return;
        }
        const float *row0 = st.lhs + at * st.lhs_stride + (long long)(16 * rb + g) * st.k + 4 * t;
        const float *row1 = row0 + 8 * st.k;
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if ((mask >> c) & 1u) {
                buf[q][c][0] = load_once_f4(row0 + 16 * c);
                buf[q][c][1] = load_once_f4(row1 + 16 * c);
            }
    };
    // this warp's half of the right end of instance `at`, 8 bytes per copy (the padded rows are 8-byte aligned)
    auto issue_rhs = [&](long long at, int parity) {
        const float *b = bp.rhs + at * bp.rhs_stride;
        float *dst = bbuf[pair][parity];
        const int pieces = bp.steps[0].k * 4 * NT;
        for (int p = 32 * w + lane; p < pieces; p += 64) {
            const int row = p / (4 * NT), col = 2 * (p % (4 * NT));
            copy_async_8(dst + row * LD + col, b + row * (8 * NT) + col);
        }
    };

    // one row block of product s: multiply, then hand the block on (intermediate) or finish it (X)
    auto process = [&](auto slot, int s, long long at, int parity) {
        constexpr int q = decltype(slot)::value;
        const BatchedChainStep &st = bp.steps[s];
        const int rb = st.rb[w][q];
        if (rb < 0) return;
        const unsigned mask = st.chunks[w][q];
        const bool last = s + 1 == S;
        const int r0 = 16 * rb + g, r1 = r0 + 8;
        // the first Add term's entries are fetched before the arithmetic: their latency hides behind it
        float2 pre[NT][2];
        const float *term0 = last && bp.add.count > 0 ? bp.add.ptr[0] : nullptr;
        if (term0) {
            term0 += at * bp.add.stride[0];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                pre[nt][0] = load_once_f2(term0 + r0 * (8 * NT) + 8 * nt + 2 * t);
                pre[nt][1] = load_once_f2(term0 + r1 * (8 * NT) + 8 * nt + 2 * t);
            }
        }
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[nt][i] = 0.0f;
        const float *rhs = s == 0 ? bbuf[pair][parity] : tbuf[pair][s & 1];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (!((mask >> c) & 1u)) continue;
            // right fragments in the renumbered order: k-step j, entry e is row 16 c + 4 t + 2 j + e
            float b[2][2][NT];
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
                for (int e = 0; e < 2; ++e)
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) b[j][e][nt] = rhs[(16 * c + 4 * t + 2 * j + e) * LD + g + 8 * nt];
            const float4 v0 = buf[q][c][0], v1 = buf[q][c][1];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                uint32_t a_hi[4], a_lo[4];
                split_tf32(j ? v0.z : v0.x, a_hi[0], a_lo[0]);       // (row g,     k 4t + 2j)
                split_tf32(j ? v1.z : v1.x, a_hi[1], a_lo[1]);       // (row g + 8, k 4t + 2j)
                split_tf32(j ? v0.w : v0.y, a_hi[2], a_lo[2]);       // (row g,     k 4t + 2j + 1)
                split_tf32(j ? v1.w : v1.y, a_hi[3], a_lo[3]);       // (row g + 8, k 4t + 2j + 1)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    uint32_t b_hi[2], b_lo[2];
                    split_tf32(b[j][0][nt], b_hi[0], b_lo[0]);
                    split_tf32(b[j][1][nt], b_hi[1], b_lo[1]);
                    mma_tf32(acc[nt], a_lo, b_hi);                   // small terms first
                    mma_tf32(acc[nt], a_hi, b_lo);
                    mma_tf32(acc[nt], a_hi, b_hi);
                }
            }
        }
        if (!last) {
            float *out_t = tbuf[pair][(s + 1) & 1];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                *reinterpret_cast<float2 *>(out_t + r0 * LD + 8 * nt + 2 * t) = make_float2(acc[nt][0], acc[nt][1]);
                *reinterpret_cast<float2 *>(out_t + r1 * LD + 8 * nt + 2 * t) = make_float2(acc[nt][2], acc[nt][3]);
            }
            return;
        }
        // X = chain value + Add terms (left to right), masked to the result's structure
        if (term0) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                acc[nt][0] += pre[nt][0].x; acc[nt][1] += pre[nt][0].y;
                acc[nt][2] += pre[nt][1].x; acc[nt][3] += pre[nt][1].y;
            }
        }
#pragma unroll 1
        for (int term = term0 ? 1 : 0; term < bp.add.count; ++term) {
            const float *p = bp.add.ptr[term];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int c0 = 8 * nt + 2 * t;
                if (!p) {                                            // Identity term
                    acc[nt][0] += r0 == c0 ? 1.0f : 0.0f; acc[nt][1] += r0 == c0 + 1 ? 1.0f : 0.0f;
                    acc[nt][2] += r1 == c0 ? 1.0f : 0.0f; acc[nt][3] += r1 == c0 + 1 ? 1.0f : 0.0f;
                } else {
                    const float *pi = p + at * bp.add.stride[term];
                    const float2 x = load_once_f2(pi + r0 * (8 * NT) + c0), y = load_once_f2(pi + r1 * (8 * NT) + c0);
                    acc[nt][0] += x.x; acc[nt][1] += x.y; acc[nt][2] += y.x; acc[nt][3] += y.y;
                }
            }
        }
        float *x = bp.out + at * bp.out_stride;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int c0 = 8 * nt + 2 * t;
            if (bp.pout != MOM_GENERAL && bp.pout != MOM_SYMMETRIC) {
                acc[nt][0] = in_structure(bp.pout, r0, c0) ? acc[nt][0] : 0.0f;
                acc[nt][1] = in_structure(bp.pout, r0, c0 + 1) ? acc[nt][1] : 0.0f;
                acc[nt][2] = in_structure(bp.pout, r1, c0) ? acc[nt][2] : 0.0f;
                acc[nt][3] = in_structure(bp.pout, r1, c0 + 1) ? acc[nt][3] : 0.0f;
            }
            *reinterpret_cast<float2 *>(x + r0 * (8 * NT) + c0) = make_float2(acc[nt][0], acc[nt][1]);
            *reinterpret_cast<float2 *>(x + r1 * (8 * NT) + c0) = make_float2(acc[nt][2], acc[nt][3]);
        }
    };

    using Slot0 = std::integral_constant<int, 0>;
    using Slot1 = std::integral_constant<int, 1>;
    int parity = 0;
    if (inst < bp.batch) {
        issue_rhs(inst, 0);
        issue_lhs(Slot0{}, 0, inst);
        issue_lhs(Slot1{}, 0, inst);
        copy_async_wait_all();
    }
    pair_barrier(pair);                                  // both halves of B are in place
    for (; inst < bp.batch; inst += pairs_total, parity ^= 1) {
        const long long next_inst = inst + pairs_total;
        if (next_inst < bp.batch) issue_rhs(next_inst, parity ^ 1);
#pragma unroll 1
        for (int s = 0; s < S; ++s) {
            // what this warp loads next: the following product of this instance, or the first one of its next instance
            const bool wraps = s + 1 == S;
            const int ns = wraps ? 0 : s + 1;
            const long long ni = wraps ? next_inst : inst;
            const bool more = ni < bp.batch;
            process(Slot0{}, s, inst, parity);
            if (more) issue_lhs(Slot0{}, ns, ni);
            process(Slot1{}, s, inst, parity);
            if (more) issue_lhs(Slot1{}, ns, ni);
            // the intermediate changes hands; after the last product the next instance's B must have landed
            if (wraps) copy_async_wait_all();
            pair_barrier(pair);
        }
    }
}

}  // namespace

void batched_chain_assign(const unsigned char *needed, int row_blocks, BatchedChainStep *step) {
    // heaviest row block first, each to the warp with less work so far; at most two row blocks per warp
    int order[4] = {0, 1, 2, 3};
    auto weight = [&](int rb) { return __builtin_popcount(needed[rb]); };
    std::stable_sort(order, order + row_blocks, [&](int a, int b) { return weight(a) > weight(b); });
    int load[2] = {0, 0}, count[2] = {0, 0};
    for (int w = 0; w < 2; ++w)
        for (int q = 0; q < 2; ++q) { step->rb[w][q] = -1; step->chunks[w][q] = 0; }
    for (int i = 0; i < row_blocks; ++i) {
        const int rb = order[i];
        int w = load[1] < load[0] ? 1 : 0;
        if (count[w] == 2) w ^= 1;
        step->rb[w][count[w]] = (signed char)rb;
        step->chunks[w][count[w]] = needed[rb];
        load[w] += weight(rb);
        ++count[w];
    }
}

cudaError_t launch_batched_chain(const BatchedChainPlan &bp, cudaStream_t stream) {
    const int sms = current_sm_count();
    if (sms < 1) return cudaErrorInvalidDevice;
    // persistent pairs of warps, instances dealt round-robin; no more CTAs than there are pairs of instances
    long long grid = (long long)sms * BC_CTAS_PER_SM;
    const long long wanted = (bp.batch + BC_PAIRS - 1) / BC_PAIRS;
    if (grid > wanted) grid = wanted;
    if (bp.n == 8) batched_chain_kernel<1><<<(unsigned)grid, BC_THREADS, 0, stream>>>(bp);
    else batched_chain_kernel<2><<<(unsigned)grid, BC_THREADS, 0, stream>>>(bp);
    return cudaGetLastError();
}

}  // namespace mom
