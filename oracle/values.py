"""Value oracle: the equation's result in double precision.  TEST INFRASTRUCTURE ONLY.

The reference value of  X = M1*M2*...*Mn + T1 + ... + Tk  is its plain definition: every operand
is materialised as a dense fp64 matrix (Identity as an actual identity matrix, so that A*I = A is
*computed*, not assumed -- paper Section 2, "Types"), the chain is multiplied strictly left to
right with the triple loop of `matmul_f64.c`, and the Add terms (paper Table 1, "Add") are added
one after the other.  No property is exploited anywhere in this file.

Only tests, the smoke check and the benchmark's CPU-baseline leg may use this module; the CUDA
library neither imports nor links it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

GENERAL, LOWER_TRI, UPPER_TRI, IDENTITY, DIAGONAL, SYMMETRIC = 0, 1, 2, 3, 4, 5
STRICT_LOWER, STRICT_UPPER, UNIT_LOWER, UNIT_UPPER = 6, 7, 8, 9

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "matmul_f64.c")
_LIB = os.path.join(_HERE, "liboracle_matmul.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C triple loop with gcc (no BLAS, no vendor library)."""
    stale = force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if stale:
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.mom_oracle_matmul_f64.restype = ctypes.c_int
        lib.mom_oracle_matmul_f64.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                              ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int]
        _lib = lib
    return _lib


def host_threads() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


_last_threads_used = 1


def threads_used() -> int:
    """Threads the most recent matmul actually ran on."""
    return _last_threads_used


def matmul(a: np.ndarray, b: np.ndarray, threads: Optional[int] = None) -> np.ndarray:
    """C = A*B, fp64, the definition C[i][j] = sum_l A[i][l]*B[l][j]."""
    global _last_threads_used
    a = np.ascontiguousarray(a, dtype=np.float64)
    b = np.ascontiguousarray(b, dtype=np.float64)
    if a.ndim != 2 or b.ndim != 2 or a.shape[1] != b.shape[0]:
        raise ValueError(f"shape mismatch {a.shape} x {b.shape}")
    c = np.empty((a.shape[0], b.shape[1]), dtype=np.float64)
    t = host_threads() if threads is None else int(threads)
    _last_threads_used = _load().mom_oracle_matmul_f64(
        a.ctypes.data, b.ctypes.data, c.ctypes.data, a.shape[0], a.shape[1], b.shape[1], t)
    return c


def dense(arr: Optional[np.ndarray], desc: Tuple[int, int, int]) -> np.ndarray:
    """The operand as a dense fp64 matrix; Identity becomes an explicit identity matrix."""
    rows, cols, prop = desc
    if prop == IDENTITY:
        if rows != cols:
            raise ValueError("Identity is square")
        return np.eye(rows, dtype=np.float64)
    a = np.asarray(arr, dtype=np.float64)
    if a.shape != (rows, cols):
        raise ValueError(f"operand shape {a.shape} differs from its descriptor {(rows, cols)}")
    return a


def transposed_operands(arrays, descs, flags):
    """Operands as the equation uses them: entry i transposed (array and descriptor) where flags[i] is set.

    The transpose of a stored lowerTri matrix is upperTri and vice versa (the paper's printed inference
    rule), likewise the strict and the unit triangles; Identity, Diagonal, Symmetric and general keep their
    property.  Dense storage is simply transposed with NumPy.
    """
    swap = {LOWER_TRI: UPPER_TRI, UPPER_TRI: LOWER_TRI, STRICT_LOWER: STRICT_UPPER, STRICT_UPPER: STRICT_LOWER,
            UNIT_LOWER: UNIT_UPPER, UNIT_UPPER: UNIT_LOWER}
    out_a, out_d = [], []
    flags = list(flags) + [False] * (len(descs) - len(flags))
    for a, (r, c, p), t in zip(arrays, descs, flags):
        if t:
            out_a.append(None if a is None else np.ascontiguousarray(np.asarray(a).T))
            out_d.append((c, r, swap.get(p, p)))
        else:
            out_a.append(a)
            out_d.append((r, c, p))
    return out_a, out_d


def evaluate(chain: Sequence[Optional[np.ndarray]], chain_descs: Sequence[Tuple[int, int, int]],
             add: Sequence[Optional[np.ndarray]] = (), add_descs: Sequence[Tuple[int, int, int]] = (),
             rows: Optional[np.ndarray] = None, threads: Optional[int] = None
             ) -> Tuple[np.ndarray, np.ndarray]:
    """(X_ref, D): the equation's value and the error denominator, both fp64.

    X_ref = ((M1*M2)*M3)...*Mn + T1 + ... + Tk, left to right.
    D     = |M1|*|M2|*...*|Mn| + |T1| + ... + |Tk|   (entrywise absolute values).
    With `rows` (an index array) only those rows of X_ref and D are computed: row i of a product
    is (row i of the left factor) times the right factor, so the selection is applied to M1 and to
    the Add terms and nothing else changes.
    """
    mats = [dense(a, d) for a, d in zip(chain, chain_descs)]
    x = mats[0] if rows is None else mats[0][rows, :]
    d = np.abs(x)
    for m in mats[1:]:
        x = matmul(x, m, threads)
        d = matmul(d, np.abs(m), threads)
    if len(mats) == 1:
        x = x.copy()
        d = d.copy()
    for t, td in zip(add, add_descs):
        tm = dense(t, td)
        if rows is not None:
            tm = tm[rows, :]
        x = x + tm
        d = d + np.abs(tm)
    return x, d


def evaluate_sum(chains: Sequence[Sequence[Optional[np.ndarray]]],
                 chain_descs: Sequence[Sequence[Tuple[int, int, int]]],
                 rows: Optional[np.ndarray] = None, threads: Optional[int] = None
                 ) -> Tuple[np.ndarray, np.ndarray]:
    """(X_ref, D) of a sum of Mul chains, X = prod(chain_1) + ... + prod(chain_c)  (paper Section 2,
    "Operations": Mul and Add are both variadic and an Equation holds a bag of them).

    Every chain is evaluated by `evaluate` on its own, left to right, and the values are added in the
    order written; D adds up the chains' denominators.  Operands are given as the equation uses them
    (apply `transposed_operands` first where a factor enters transposed).
    """
    x = d = None
    for mats, descs in zip(chains, chain_descs):
        xc, dc = evaluate(mats, descs, rows=rows, threads=threads)
        x = xc if x is None else x + xc
        d = dc if d is None else d + dc
    return x, d


def evaluate_expr(expr, arrays: Sequence[Optional[np.ndarray]], descs: Sequence[Tuple[int, int, int]],
                  threads: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """(X_ref, D) of a nested expression, by its plain definition (paper Section 2, "Operations": Mul, Add
    and Transpose inside one Equation).  `expr` is an operand index, ("t", e), ("mul", [e...]) or
    ("add", [e...]); operands are the stored matrices.  A product is multiplied left to right with the
    fp64 triple loop, a sum is added left to right, a transpose is NumPy's.  D follows the same recursion
    on absolute values: D(operand) = |A|, D(product) = product of the D's, D(sum) = sum of the D's.
    """
    def walk(e):
        if isinstance(e, int):
            a = dense(arrays[e], descs[e])
            return a, np.abs(a)
        kind = e[0]
        if kind == "t":
            x, d = walk(e[1])
            return np.ascontiguousarray(x.T), np.ascontiguousarray(d.T)
        parts = [walk(c) for c in e[1]]
        x, d = parts[0]
        for xc, dc in parts[1:]:
            if kind == "mul":
                x, d = matmul(x, xc, threads), matmul(d, dc, threads)
            elif kind == "add":
                x, d = x + xc, d + dc
            else:
                raise ValueError(f"unknown operation {kind!r}")
        return x, d

    x, d = walk(expr)
    return np.array(x, dtype=np.float64, copy=True), np.array(d, dtype=np.float64, copy=True)


def evaluate_steps(chain: Sequence[Optional[np.ndarray]], chain_descs: Sequence[Tuple[int, int, int]],
                   steps, add: Sequence[Optional[np.ndarray]] = (),
                   add_descs: Sequence[Tuple[int, int, int]] = (), threads: Optional[int] = None) -> np.ndarray:
    """The equation's value following a plan's binary products (ids as in `oracle.plan.Step`).

    Used to check associativity (any parenthesization gives the left-to-right value up to fp64
    rounding) and as the timed CPU baseline; products stay dense and property-blind.
    """
    vals = {i: (None if chain_descs[i][2] == IDENTITY else np.asarray(chain[i], dtype=np.float64))
            for i in range(len(chain))}
    last = None
    for s in steps:
        rhs = np.ascontiguousarray(vals[s.lhs].T) if getattr(s, "gram", False) else vals[s.rhs]   # Y * Y^T
        vals[s.out] = matmul(vals[s.lhs], rhs, threads)
        last = s.out
    if last is None:
        kept = [i for i in range(len(chain)) if chain_descs[i][2] != IDENTITY]
        x = dense(None, chain_descs[0]) if not kept else vals[kept[0]].copy()
    else:
        x = vals[last]
    for t, td in zip(add, add_descs):
        x = x + dense(t, td)
    return x


def normwise_error(x: np.ndarray, x_ref: np.ndarray, d: np.ndarray) -> float:
    """||X - X_ref||_F / ||D||_F in fp64 (0/0 counts as 0)."""
    num = float(np.linalg.norm(np.asarray(x, dtype=np.float64) - x_ref))
    den = float(np.linalg.norm(d))
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return num / den


def off_structure_mask(rows: int, cols: int, prop: int, row_index: Optional[np.ndarray] = None) -> np.ndarray:
    """Boolean mask of entries that lie OUTSIDE the structure of `prop` (must hold exact zeros)."""
    i = (np.arange(rows) if row_index is None else np.asarray(row_index))[:, None]
    j = np.arange(cols)[None, :]
    if prop in (GENERAL, SYMMETRIC):
        return np.zeros((i.shape[0], cols), dtype=bool)
    if prop in (LOWER_TRI, UNIT_LOWER):
        return i < j
    if prop in (UPPER_TRI, UNIT_UPPER):
        return i > j
    if prop == STRICT_LOWER:
        return i <= j
    if prop == STRICT_UPPER:
        return i >= j
    if prop in (IDENTITY, DIAGONAL):
        return i != j
    raise ValueError("unknown property")


def unit_diagonal_exactly_one(x: np.ndarray, prop: int, row_index: Optional[np.ndarray] = None) -> bool:
    """True iff the property fixes no diagonal of ones, or every diagonal entry of x (rows `row_index`) is exactly 1."""
    if prop not in (UNIT_LOWER, UNIT_UPPER):
        return True
    x = np.asarray(x)
    rows = np.arange(x.shape[-2]) if row_index is None else np.asarray(row_index)
    inside = rows < x.shape[-1]
    return bool(np.all(x[..., np.nonzero(inside)[0], rows[inside]] == 1.0))


def off_structure_exactly_zero(x: np.ndarray, prop: int, row_index: Optional[np.ndarray] = None) -> bool:
    """True iff every entry outside the structure is +0.0 or -0.0 numerically equal to zero."""
    x = np.asarray(x)
    mask = off_structure_mask(x.shape[-2] if row_index is None else len(row_index), x.shape[-1], prop, row_index)
    return bool(np.all(x[..., mask] == 0))
