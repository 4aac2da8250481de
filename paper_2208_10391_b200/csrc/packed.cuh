// Packed storage of triangular matrices (one of the "more appropriate containers" the paper's Section 2 leaves to
// future work): only the triangle is kept, row by row, every stored row a whole number of 16-byte groups so that
// rows stay addressable by 16-byte accesses.
//   lower triangle: row i holds columns [0, 4 * (i / 4 + 1))
//   upper triangle: row i holds columns [4 * (i / 4), n rounded up to a multiple of 4)
// Rows follow each other without gaps.  The stored entries outside the triangle (fewer than four per row next to
// the diagonal) and beyond the last column are padding and hold zeros.
#pragma once

#include <cuda_runtime.h>

namespace mom {

struct PackedRow {
    long long offset;     // position of the row's first stored entry
    int first, end;       // stored columns [first, end)
};

// Closed forms of the row starts: with q = i / 4 full groups of four rows before row i's group,
//   lower: four rows of 4 (p + 1) entries for every p < q, then (i - 4 q) rows of 4 (q + 1);
//   upper: every row r < i has n4 - 4 (r / 4) entries.
// i == n gives the size of the container.
__host__ __device__ inline PackedRow packed_row(bool lower, int n, int i) {
    const long long q = i >> 2, rest = i - 4 * q;
    PackedRow r;
    if (lower) {
        r.first = 0;
        r.end = 4 * (int)(q + 1);
        r.offset = 8 * q * (q + 1) + rest * 4 * (q + 1);
    } else {
        const long long n4 = (n + 3) & ~3;
        r.first = 4 * (int)q;
        r.end = (int)n4;
        r.offset = (long long)i * n4 - 8 * q * (q - 1) - 4 * q * rest;
    }
    return r;
}

__host__ __device__ inline long long packed_elements(bool lower, int n) { return packed_row(lower, n, n).offset; }

}  // namespace mom
