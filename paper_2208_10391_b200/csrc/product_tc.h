// Tensor-core (tcgen05, 3xTF32) product path: host-side interface used by the launcher.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include "kernels.h"
#include "mom_internal.h"

namespace mom {

struct TcStepState {
    int4 *tiles = nullptr;      // device: work-sorted tile table {row0, col0, k_begin, k_end}
    int num_tiles = 0;
    bool pair = false;          // tiles are 256 rows high and run on CTA pairs (cta_group::2)
    bool mirror = false;        // Gram product: tiles on and below the diagonal only, the others written as mirror images
    // The product that writes X can also run as two launches, rows [0, part_row) first: the host-staging entry
    // point copies those rows back while the second launch runs.  part_row == 0: no such tables.
    int part_row = 0;
    int4 *part_tiles[2] = {nullptr, nullptr};
    int part_num[2] = {0, 0};
    int part_units[2] = {1, 1};
    // A product that is not the one writing X, whose left operand is a general matrix read as stored: the same two row
    // ranges let the host-staging entry point upload that operand in two pieces and start on the first one while the
    // second is still on its way; then each launch splits its own rows of the operand.  False: splits happen in part 1.
    bool split_a_by_part = false;
    int cluster_split = 0;      // > 1: split-K inside thread-block clusters of this size (table in tile order, one entry per CTA)
    int units = 1;              // CTAs (or CTA pairs) the table was laid out for: unit u owns entries u, u + units, ...
};

struct TcPlanState {
    bool ready = false;
    std::vector<TcStepState> steps;     // one entry per plan step (unused for FFMA steps)
    void *block = nullptr;              // single device allocation backing all tables
};

// Builds the tile tables of every tensor-core step (first call only; one cudaMalloc).
mom_status_t tc_prepare(const mom_plan &p, TcPlanState &s);

// Enqueues the operand splits and the product kernel of step `step`.  `before_product`, when not
// null, is recorded on the stream between the splits and the product kernel.
// `part`: 0 the whole product; 1 the operand splits and the rows [0, part_row); 2 the remaining rows (no splits,
// unless split_a_by_part: then part 1 splits the left operand's rows [0, part_row) and part 2 the others).
mom_status_t tc_launch_step(const mom_plan &p, TcPlanState &s, int step, const ProductArgs &a, char *workspace,
                            int32_t *status, cudaStream_t stream, int *launches, cudaEvent_t before_product, int part = 0);

void tc_release(TcPlanState &s);

// Tensor map of a 2-D f32 row-major matrix (rows x cols) with a box of box_rows x box_cols elements.
bool tc_make_map(CUtensorMap *map, const void *ptr, int rows, int cols, int box_rows, int box_cols, CUtensorMapSwizzle swizzle);

// The small / mid-size product kernel (product_tc_inline.cu): one launch, operands read as stored and split in shared
// memory.  Returns cudaErrorNotSupported when the product is not of a shape it takes (the caller then uses another kernel).
cudaError_t launch_product_tc_inline(const ProductArgs &a, int32_t *status, cudaStream_t stream);
bool product_tc_inline_takes(int64_t m, int64_t n, int64_t k, int lhs_transposed, int rhs_transposed, int pa, int pb);

// One thread waits with the product kernels' bounded wait on a barrier nothing arrives on; after `limit_ns` it
// records {MOM_ERR_DEVICE_TIMEOUT, detail} in `status` (device, 4 ints) and the kernel ends.
cudaError_t launch_wait_timeout_probe(int32_t *status, unsigned long long limit_ns, int detail, cudaStream_t stream);

}  // namespace mom
