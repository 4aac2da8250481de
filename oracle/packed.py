"""Packed storage of triangular matrices: the index map, by its plain definition.  TEST INFRASTRUCTURE ONLY.

The paper stores every matrix as a dense buffer and names "more appropriate containers" as future work
(Section 2, "Matrix Attribute"; the conclusion speaks of non-rectangular iteration spaces).  The container
defined here keeps only the triangle, row by row, with every stored row a whole number of 16-byte groups so
that rows stay addressable by 16-byte accesses:

    lower triangle, n x n: row i holds columns [0, 4 * (i // 4 + 1))   -- the diagonal's group of four included
    upper triangle, n x n: row i holds columns [4 * (i // 4), N4)      -- N4 = n rounded up to a multiple of 4

Rows follow each other without gaps, so row i starts at the sum of the lengths of the rows before it.  The few
stored entries that lie outside the triangle (at most three per row, next to the diagonal) and those beyond
column n - 1 are padding and hold zeros.  Strictly and unit triangular matrices use the container of the
ordinary triangle of the same orientation (their diagonal is stored like any entry).

Everything here is written as the definition reads (loops over rows, one entry at a time); the library's closed
forms are compared with it in the tests.  Only tests, the smoke check and the benchmark's CPU-baseline leg may
use this module.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np

GENERAL, LOWER_TRI, UPPER_TRI, IDENTITY, DIAGONAL, SYMMETRIC = 0, 1, 2, 3, 4, 5
STRICT_LOWER, STRICT_UPPER, UNIT_LOWER, UNIT_UPPER = 6, 7, 8, 9
DENSE, PACKED = 0, 1

_LOWER = (LOWER_TRI, STRICT_LOWER, UNIT_LOWER)
_UPPER = (UPPER_TRI, STRICT_UPPER, UNIT_UPPER)


def packable(prop: int) -> bool:
    """Only triangular matrices have a packed container."""
    return prop in _LOWER or prop in _UPPER


def row_range(n: int, prop: int, i: int) -> Tuple[int, int]:
    """Columns [first, end) that the container holds of row i."""
    if not 0 <= i < n:
        raise IndexError(i)
    if prop in _LOWER:
        return 0, 4 * (i // 4 + 1)
    if prop in _UPPER:
        return 4 * (i // 4), 4 * ((n + 3) // 4)
    raise ValueError("only triangular matrices can be packed")


def row_offset(n: int, prop: int, i: int) -> int:
    """Position of row i's first stored entry: the lengths of all earlier rows added up."""
    total = 0
    for r in range(i):
        first, end = row_range(n, prop, r)
        total += end - first
    return total


def elements(n: int, prop: int) -> int:
    """Number of f32 entries of the container."""
    total = 0
    for r in range(n):
        first, end = row_range(n, prop, r)
        total += end - first
    return total


def index(n: int, prop: int, i: int, j: int) -> int:
    """Position of entry (i, j) in the container, or -1 when the container does not hold it."""
    first, end = row_range(n, prop, i)
    if not first <= j < end:
        return -1
    return row_offset(n, prop, i) + (j - first)


def pack(a: np.ndarray, prop: int) -> np.ndarray:
    """The container of the dense triangular matrix `a` (float32): row by row, the stored column range copied;
    positions beyond column n - 1 stay zero."""
    a = np.asarray(a)
    n = a.shape[0]
    if a.shape != (n, n):
        raise ValueError("triangular matrices are square")
    out = np.zeros(elements(n, prop), dtype=np.float32)
    at = 0
    for i in range(n):
        first, end = row_range(n, prop, i)
        inside = min(end, n) - first
        out[at:at + inside] = a[i, first:first + inside]
        at += end - first
    return out


def unpack(p: np.ndarray, n: int, prop: int) -> np.ndarray:
    """The dense n x n matrix a container stands for (entries the container does not hold are zero)."""
    p = np.asarray(p)
    if p.shape != (elements(n, prop),):
        raise ValueError(f"a packed {n} x {n} triangle has {elements(n, prop)} entries, not {p.shape}")
    a = np.zeros((n, n), dtype=p.dtype)
    at = 0
    for i in range(n):
        first, end = row_range(n, prop, i)
        inside = min(end, n) - first
        a[i, first:first + inside] = p[at:at + inside]
        at += end - first
    return a
