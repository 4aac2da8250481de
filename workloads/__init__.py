"""Seeded synthetic Linnea equations: shapes, properties and random entries.

This module is shared by the CPU oracle's tests, the GPU parity tests and the
benchmark.  It only *describes* equations and draws their entries; it holds no
planning and no product arithmetic, so neither implementation can inherit the
other's mistakes through it.

An equation is ``X = M1 * M2 * ... * Mn + T1 + ... + Tk`` (paper Section 2,
"Operations": variadic Mul and Add inside an Equation).  Every matrix carries
one compile-time property (paper Section 2, "Matrix Attribute" and "Types").

Storage convention for generated data (paper Section 2: the property dictates
how the dense buffer is filled): dense row-major float32; entries outside a
triangular or diagonal operand's structure are ``+0.0``; Identity operands are
never materialised (``None``).

Random stream: NumPy's Philox counter-based generator keyed by
``(seed, operand index)``; operand indices count the chain first, then the
Add terms.  The same key always yields the same matrix.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional, Sequence

import numpy as np

GENERAL, LOWER_TRI, UPPER_TRI, IDENTITY, DIAGONAL, SYMMETRIC = 0, 1, 2, 3, 4, 5
STRICT_LOWER, STRICT_UPPER, UNIT_LOWER, UNIT_UPPER = 6, 7, 8, 9
PROPERTY_NAMES = {GENERAL: "general", LOWER_TRI: "lowerTri", UPPER_TRI: "upperTri", IDENTITY: "Identity",
                  DIAGONAL: "diagonal", SYMMETRIC: "symmetric", STRICT_LOWER: "strictLowerTri",
                  STRICT_UPPER: "strictUpperTri", UNIT_LOWER: "unitLowerTri", UNIT_UPPER: "unitUpperTri"}
_TRIANGLE_KINDS = (STRICT_LOWER, STRICT_UPPER, UNIT_LOWER, UNIT_UPPER)


@dataclass(frozen=True)
class Operand:
    """One matrix of an equation: static shape, property and entry distribution.

    dist: "uniform"  -> U(-1, 1)
          "normal"   -> N(0, sigma^2)
          "ones"     -> every structural entry 1 (the paper's Listing 2 fill)
    Triangular operands always use: strict part from `dist`, diagonal 1 + U(0, 1)
    (except dist == "ones"), other half exactly zero.  Diagonal operands: diagonal
    1 + U(0, 1) (or ones), everything else exactly zero.  Symmetric operands: the lower triangle
    from `dist`, mirrored into the upper one (exactly symmetric in float32).
    """
    rows: int
    cols: int
    prop: int = GENERAL
    dist: str = "uniform"
    sigma: float = 1.0


@dataclass(frozen=True)
class Equation:
    name: str
    seed: int
    chain: Sequence[Operand]
    add: Sequence[Operand] = field(default_factory=tuple)
    batch: int = 1  # > 1: `batch` independent instances sharing one plan
    chain_t: Sequence[bool] = ()   # operand i of the chain enters the equation transposed (stored as given)
    add_t: Sequence[bool] = ()

    def descs(self):
        return [(o.rows, o.cols, o.prop) for o in self.chain]

    def add_descs(self):
        return [(o.rows, o.cols, o.prop) for o in self.add]


def _draw(rng: np.random.Generator, shape, dist: str, sigma: float) -> np.ndarray:
    if dist == "uniform":
        return (rng.random(shape, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)).astype(np.float32)
    if dist == "normal":
        return (rng.standard_normal(shape, dtype=np.float32) * np.float32(sigma)).astype(np.float32)
    if dist == "ones":
        return np.ones(shape, dtype=np.float32)
    raise ValueError(f"unknown distribution {dist!r}")


def generate_operand(op: Operand, seed: int, index: int, batch: int = 1) -> Optional[np.ndarray]:
    """Dense float32 array for one operand; shape (rows, cols), or (batch, rows, cols) if batch > 1.

    Returns None for Identity (it is a type, not data).
    """
    if op.prop == IDENTITY:
        return None
    rng = np.random.Generator(np.random.Philox(key=[int(seed), int(index)]))
    shape = (batch, op.rows, op.cols) if batch > 1 else (op.rows, op.cols)
    m = _draw(rng, shape, op.dist, op.sigma)
    if op.prop in (LOWER_TRI, UPPER_TRI, DIAGONAL):
        if op.rows != op.cols:
            raise ValueError("triangular and diagonal operands are square")
        n = op.rows
        if op.dist != "ones":
            diag = np.float32(1.0) + rng.random(shape[:-1], dtype=np.float32)
            idx = np.arange(n)
            m[..., idx, idx] = diag
        keep = (np.tril(np.ones((n, n), dtype=bool)) if op.prop == LOWER_TRI else
                np.triu(np.ones((n, n), dtype=bool)) if op.prop == UPPER_TRI else np.eye(n, dtype=bool))
        m = np.where(keep, m, np.float32(0.0)).astype(np.float32)
    if op.prop in _TRIANGLE_KINDS:
        # strictly triangular: zeros on the diagonal; unit triangular: ones there, stored as 1.0
        if op.rows != op.cols:
            raise ValueError("triangular operands are square")
        n = op.rows
        lower = op.prop in (STRICT_LOWER, UNIT_LOWER)
        keep = np.tril(np.ones((n, n), dtype=bool), -1) if lower else np.triu(np.ones((n, n), dtype=bool), 1)
        m = np.where(keep, m, np.float32(0.0)).astype(np.float32)
        if op.prop in (UNIT_LOWER, UNIT_UPPER):
            idx = np.arange(n)
            m[..., idx, idx] = np.float32(1.0)
    if op.prop == SYMMETRIC:
        if op.rows != op.cols:
            raise ValueError("symmetric operands are square")
        low = np.tril(m)
        m = low + np.swapaxes(np.tril(m, -1), -1, -2)
    return np.ascontiguousarray(m, dtype=np.float32)


def generate(eq: Equation):
    """(chain arrays, add-term arrays); Identity entries are None."""
    chain = [generate_operand(o, eq.seed, i, eq.batch) for i, o in enumerate(eq.chain)]
    add = [generate_operand(o, eq.seed, len(eq.chain) + i, eq.batch) for i, o in enumerate(eq.add)]
    return chain, add


def pack_triangle(a: np.ndarray, lower: bool) -> np.ndarray:
    """A dense triangular matrix (or a stack of them, instance first) as a packed container: rows one after the other,
    row i holding columns [0, 4 * (i // 4 + 1)) of a lower triangle, or [4 * (i // 4), n rounded up to a multiple of 4)
    of an upper one; positions past the last column are zero.  Layout only: an input is re-arranged, nothing is computed."""
    a = np.asarray(a, dtype=np.float32)
    n = a.shape[-1]
    n4 = 4 * ((n + 3) // 4)
    padded = np.zeros(a.shape[:-1] + (n4,), dtype=np.float32)
    padded[..., :n] = a
    rows = np.arange(n)[:, None]
    cols = np.arange(n4)[None, :]
    group = 4 * (rows // 4)
    keep = (cols < group + 4) if lower else (cols >= group)
    return np.ascontiguousarray(padded[..., keep])          # boolean selection walks the matrix row by row


# --------------------------------------------------------------------------
# The benchmark's configurations (shapes, properties, distributions, seeds).
# --------------------------------------------------------------------------

def config_tiny(seed: int = 0) -> Equation:
    """X = L*A*B: L 64x64 lowerTri, A 64x32, B 32x48, U(-1,1)."""
    return Equation("tiny_LAB", seed, (
        Operand(64, 64, LOWER_TRI), Operand(64, 32), Operand(32, 48)))


def config_tiny_identity_left(seed: int = 0) -> Equation:
    """X = I*L (the product must vanish from the plan)."""
    return Equation("tiny_IL", seed, (Operand(64, 64, IDENTITY), Operand(64, 64, LOWER_TRI)))


def config_tiny_identity_right(seed: int = 0) -> Equation:
    """X = L*I."""
    return Equation("tiny_LI", seed, (Operand(64, 64, LOWER_TRI), Operand(64, 64, IDENTITY)))


def config_five_general(seed: int = 1) -> Equation:
    """Five general matrices whose parenthesization dominates the cost; N(0,1)."""
    dims = [1024, 256, 2048, 64, 1024, 512]
    return Equation("five_general", seed, tuple(
        Operand(dims[i], dims[i + 1], GENERAL, "normal") for i in range(5)))


def config_property_heavy(n: int = 4096, seed: int = 2) -> Equation:
    """X = L*U*I*B + C, all n x n; the Identity between U and B is to be eliminated."""
    return Equation(f"LUIB_plus_C_{n}", seed, (
        Operand(n, n, LOWER_TRI), Operand(n, n, UPPER_TRI), Operand(n, n, IDENTITY),
        Operand(n, n, GENERAL, "normal")), (Operand(n, n, GENERAL, "normal"),))


def config_large_square(n: int = 8192, seed: int = 3) -> Equation:
    """X = L*A*U*B, all n x n; A, B ~ N(0, 1/n) so that magnitudes stay O(1)."""
    s = float(n) ** -0.5
    return Equation(f"LAUB_{n}", seed, (
        Operand(n, n, LOWER_TRI), Operand(n, n, GENERAL, "normal", s),
        Operand(n, n, UPPER_TRI), Operand(n, n, GENERAL, "normal", s)))


def config_batched(batch: int = 4096, seed: int = 4) -> Equation:
    """`batch` instances of X_i = L_i*A_i*B_i + C_i (64x64, 64x64, 64x16, 64x16), U(-1,1)."""
    return Equation(f"batched_LAB_plus_C_x{batch}", seed, (
        Operand(64, 64, LOWER_TRI), Operand(64, 64), Operand(64, 16)), (Operand(64, 16),), batch=batch)


def config_paper_chain(seed: int = 5) -> Equation:
    """The chain of the paper's Section 4: 800x1100, 1100x900, 900x1200, 1200x100; N(0,1)."""
    dims = [800, 1100, 900, 1200, 100]
    return Equation("paper_section4_chain", seed, tuple(
        Operand(dims[i], dims[i + 1], GENERAL, "normal") for i in range(4)))


def config_transposed(n: int = 4096, seed: int = 6) -> Equation:
    """X = L^T * A * U^T * B + C^T, all n x n: the Transpose op on chain operands and on an Add term.

    L is stored lower triangular (used as upper), U stored upper (used as lower)."""
    s = float(n) ** -0.5
    return Equation(f"LtAUtB_plus_Ct_{n}", seed, (
        Operand(n, n, LOWER_TRI), Operand(n, n, GENERAL, "normal", s),
        Operand(n, n, UPPER_TRI), Operand(n, n, GENERAL, "normal", s)), (Operand(n, n, GENERAL, "normal"),),
        chain_t=(True, False, True, False), add_t=(True,))


def config_diagonal(n: int = 4096, seed: int = 10) -> Equation:
    """X = L * D * A * U + C: a Diagonal factor between a triangle and a general matrix (it joins the
    triangle: n(n+1)/2 multiplications instead of n^2), then two triangular x general products."""
    s = 1.0 / np.sqrt(n)
    return Equation(f"LDAU_plus_C_{n}", seed, (
        Operand(n, n, LOWER_TRI), Operand(n, n, DIAGONAL), Operand(n, n, GENERAL, "normal", s), Operand(n, n, UPPER_TRI)),
        (Operand(n, n, GENERAL, "normal"),))


def config_square_product(n: int = 1024, seed: int = 12) -> Equation:
    """One general product A*B, both n x n, N(0, 1/n): the mid-size range between the small-product kernel and the large
    tensor-core products (timed at 1024, 1536 and 2048)."""
    g = Operand(n, n, GENERAL, "normal", 1.0 / np.sqrt(n))
    return Equation(f"GG_{n}", seed, (g, g))


def config_packed_triangular(n: int = 4096, seed: int = 13) -> Equation:
    """X = L*L + L with both factors, the term and X meant for packed storage (the storage is chosen by the caller)."""
    return Equation(f"LL_plus_L_{n}", seed, (Operand(n, n, LOWER_TRI), Operand(n, n, LOWER_TRI)), (Operand(n, n, LOWER_TRI),))


def config_listing2() -> Equation:
    """Listing 2 of the paper: two 5x5 lowerTri matrices filled with the constant 1."""
    return Equation("listing2_LL_5", 0, (
        Operand(5, 5, LOWER_TRI, "ones"), Operand(5, 5, LOWER_TRI, "ones")))


def random_equation(seed: int, max_len: int = 6, max_dim: int = 96, allow_add: bool = True,
                    dim_multiple: int = 1, diagonal: bool = False, kinds: bool = False) -> Equation:
    """A random well-formed equation (for property tests): random length, dims, properties.

    Triangular / Identity operands are only placed where the neighbouring dimensions are equal,
    which the generator arranges by repeating a dimension.  With `diagonal` about a quarter of the
    operands and Add terms are Diagonal (the streams without it are unchanged).  With `kinds` a third of them
    are strictly or unit triangular (a stream of its own, Diagonal included).
    """
    diagonal = diagonal or kinds
    rng = np.random.Generator(np.random.Philox(key=[int(seed), 0x7D1A6 if kinds else 0xD1A6 if diagonal else 0xC0FFEE]))
    n = int(rng.integers(1, max_len + 1))
    chain: List[Operand] = []
    cur = int(rng.integers(1, max_dim // dim_multiple + 1)) * dim_multiple
    for _ in range(n):
        kind = int(rng.integers(0, 12 if kinds else 8 if diagonal else 6))
        if kind >= 8:
            chain.append(Operand(cur, cur, _TRIANGLE_KINDS[kind - 8]))
        elif kind >= 6:
            chain.append(Operand(cur, cur, DIAGONAL))
        elif kind == 0:
            chain.append(Operand(cur, cur, LOWER_TRI))
        elif kind == 1:
            chain.append(Operand(cur, cur, UPPER_TRI))
        elif kind == 2:
            chain.append(Operand(cur, cur, IDENTITY))
        else:
            nxt = int(rng.integers(1, max_dim // dim_multiple + 1)) * dim_multiple
            chain.append(Operand(cur, nxt, GENERAL, "normal" if kind == 3 else "uniform"))
            cur = nxt
    rows, cols = chain[0].rows, chain[-1].cols
    add: List[Operand] = []
    if allow_add:
        for _ in range(int(rng.integers(0, 3))):
            kind = int(rng.integers(0, 11 if kinds else 7 if diagonal else 5))
            if rows == cols and kind >= 7:
                add.append(Operand(rows, cols, _TRIANGLE_KINDS[kind - 7]))
            elif rows == cols and kind >= 5:
                add.append(Operand(rows, cols, DIAGONAL))
            elif rows == cols and kind == 0:
                add.append(Operand(rows, cols, LOWER_TRI))
            elif rows == cols and kind == 1:
                add.append(Operand(rows, cols, UPPER_TRI))
            elif rows == cols and kind == 2:
                add.append(Operand(rows, cols, IDENTITY))
            else:
                add.append(Operand(rows, cols, GENERAL))
    return Equation(f"random_{seed}", seed, tuple(chain), tuple(add))


def with_batch(eq: Equation, batch: int) -> Equation:
    return replace(eq, batch=batch, name=f"{eq.name}_x{batch}")


# --------------------------------------------------------------------------
# Sums of several Mul chains (paper Section 2, "Operations": Mul and Add are
# variadic and one Equation holds a bag of them).
# --------------------------------------------------------------------------

@dataclass(frozen=True)
class SumEquation:
    """X = prod(chains[0]) + prod(chains[1]) + ...; a chain of one factor is a plain Add term.

    names[c][f] identifies the stored matrix behind factor f of chain c: equal names mean the same
    matrix (drawn once, keyed by its name); transposed[c][f] says the factor enters transposed.
    """
    name: str
    seed: int
    chains: Sequence[Sequence[Operand]]
    transposed: Sequence[Sequence[bool]]
    names: Sequence[Sequence[int]]

    def descs(self):
        return [[(o.rows, o.cols, o.prop) for o in chain] for chain in self.chains]


def generate_sum(eq: SumEquation):
    """Per chain, per factor: the stored float32 array (None for Identity); one array object per name."""
    by_name = {}
    out = []
    for chain, names in zip(eq.chains, eq.names):
        row = []
        for o, nm in zip(chain, names):
            if nm not in by_name:
                by_name[nm] = generate_operand(o, eq.seed, nm)
            row.append(by_name[nm])
        out.append(row)
    return out


def random_sum_equation(seed: int, max_chains: int = 4, max_len: int = 5, max_dim: int = 48,
                        dim_multiple: int = 1, share: float = 0.5, diagonal: bool = False,
                        kinds: bool = False) -> SumEquation:
    """Random well-formed sum of chains.  With probability `share`/2 a chain starts with a run of factors
    copied (same names and flags) from an earlier chain, so that shared products occur.  With `diagonal`
    some square factors are Diagonal (the streams without it are unchanged); with `kinds` some are strictly or
    unit triangular as well (a stream of its own)."""
    diagonal = diagonal or kinds
    rng = np.random.Generator(np.random.Philox(key=[int(seed), 0x75D1A6 if kinds else 0x5D1A6 if diagonal else 0x5EED5]))
    rows = int(rng.integers(1, max_dim // dim_multiple + 1)) * dim_multiple
    cols = int(rng.integers(1, max_dim // dim_multiple + 1)) * dim_multiple
    if rng.random() < 0.4:
        cols = rows
    chains, flags, names = [], [], []
    next_name = 0

    def new_factor(r, c):
        nonlocal next_name
        """One stored factor whose type AS USED is r x c, with a random property and transposition."""
        kind = int(rng.integers(0, 13 if kinds else 9 if diagonal else 7))
        t = bool(rng.integers(0, 3) == 0)
        if r == c and kind >= 9:
            o = Operand(r, r, _TRIANGLE_KINDS[kind - 9])
        elif r == c and kind >= 7:
            o = Operand(r, r, DIAGONAL)
        elif r == c and kind == 0:
            o = Operand(r, r, LOWER_TRI)
        elif r == c and kind == 1:
            o = Operand(r, r, UPPER_TRI)
        elif r == c and kind == 2:
            o = Operand(r, r, IDENTITY)
        else:
            o = Operand(c, r, GENERAL) if t else Operand(r, c, GENERAL)
        nm = next_name
        next_name += 1
        return o, t, nm

    def used_shape(o, t):
        return (o.cols, o.rows) if t else (o.rows, o.cols)

    for c in range(int(rng.integers(1, max_chains + 1))):
        length = int(rng.integers(1, max_len + 1))
        ops, ts, nms = [], [], []
        if chains and rng.random() < share:
            src = int(rng.integers(0, len(chains)))
            take = int(rng.integers(1, len(chains[src]) + 1))
            if rng.random() < 0.5:                         # copy a prefix: its first factor has `rows` rows
                ops, ts, nms = list(chains[src][:take]), list(flags[src][:take]), list(names[src][:take])
        cur = used_shape(ops[-1], ts[-1])[1] if ops else rows
        while len(ops) < length - 1 or not ops:
            last = len(ops) >= length - 1
            nxt = cols if last else int(rng.integers(1, max_dim // dim_multiple + 1)) * dim_multiple
            if not last and rng.random() < 0.4:
                nxt = cur
            o, t, nm = new_factor(cur, nxt)
            ops.append(o); ts.append(t); nms.append(nm)
            cur = nxt
        if cur != cols:                                    # a copied prefix that does not end on `cols`
            o, t, nm = new_factor(cur, cols)
            ops.append(o); ts.append(t); nms.append(nm)
        chains.append(tuple(ops)); flags.append(tuple(ts)); names.append(tuple(nms))
    return SumEquation(f"random_sum_{seed}", seed, tuple(chains), tuple(flags), tuple(names))


def random_gram_sum(seed: int, max_dim: int = 40, dim_multiple: int = 1) -> SumEquation:
    """Random sum of chains in which Gram products occur: every chain is (prefix) * Y-factors * mirrored
    Y-factors * (suffix), where the mirrored half names the same matrices with the transposition flags
    flipped (or, for Symmetric and Diagonal factors, sometimes kept); later chains often reuse the first
    chain's Y, so that Gram products and their halves are shared between chains."""
    rng = np.random.Generator(np.random.Philox(key=[int(seed), 0x6AA3]))
    dim = lambda: int(rng.integers(1, max_dim // dim_multiple + 1)) * dim_multiple
    next_name = [0]

    def factor(r, c):
        """(stored operand, transposed flag, name) of a new matrix used as r x c"""
        kind = int(rng.integers(0, 8))
        t = bool(rng.integers(0, 2))
        if r == c and kind < 4:
            o = Operand(r, r, (LOWER_TRI, UPPER_TRI, SYMMETRIC, DIAGONAL)[kind])
        else:
            o = Operand(c, r, GENERAL, "normal") if t else Operand(r, c, GENERAL, "normal")
        next_name[0] += 1
        return o, t, next_name[0]

    n = dim()                                              # every chain's value is n x n
    halves = []
    chains, flags, names = [], [], []
    for c in range(int(rng.integers(1, 4))):
        if halves and rng.random() < 0.6:
            half = halves[int(rng.integers(0, len(halves)))]
        else:
            half, cur = [], n
            for q in range(int(rng.integers(1, 4))):
                nxt = cur if rng.random() < 0.4 else dim()
                half.append(factor(cur, nxt))
                cur = nxt
            halves.append(half)
        mirrored = [(o, (t if o.prop in (SYMMETRIC, DIAGONAL) and rng.random() < 0.5 else not t), nm) for o, t, nm in reversed(half)]
        body = list(half) + mirrored
        if rng.random() < 0.3:                             # a square factor in front or behind breaks the symmetry of the chain
            extra = factor(n, n)
            body = [extra] + body if rng.random() < 0.5 else body + [extra]
        chains.append(tuple(o for o, _, _ in body)); flags.append(tuple(t for _, t, _ in body)); names.append(tuple(nm for _, _, nm in body))
    return SumEquation(f"random_gram_{seed}", seed, tuple(chains), tuple(flags), tuple(names))


def config_gram(n: int = 4096, k: int = 2048, seed: int = 11) -> SumEquation:
    """X = A * B * B^T * A^T + S: A n x k, B k x k general, S Symmetric.  The chain reads Y * Y^T with Y = A * B:
    one general product, then only the lower triangle of Y * Y^T (mirrored), plus a Symmetric summand."""
    a = Operand(n, k, GENERAL, "normal", 1.0 / np.sqrt(k))
    b = Operand(k, k, GENERAL, "normal", 1.0 / np.sqrt(k))
    return SumEquation(f"ABBtAt_plus_S_{n}", seed, ((a, b, b, a), (Operand(n, n, SYMMETRIC, "normal"),)),
                       ((False, False, True, True), (False,)), ((0, 1, 1, 0), (2,)))


def config_sum_shared(n: int = 4096, seed: int = 7) -> SumEquation:
    """X = C*A*B + D*A*B, all general n x n: every tree ties, the right-nested one is taken, and A*B is
    below the root in both chains, so it is multiplied once (3 products instead of 4)."""
    g = Operand(n, n, GENERAL, "normal", 1.0 / np.sqrt(n))
    return SumEquation(f"CAB_plus_DAB_{n}", seed, ((g, g, g), (g, g, g)), ((False,) * 3, (False,) * 3),
                       ((2, 0, 1), (3, 0, 1)))


def config_sum_triangular(n: int = 4096, seed: int = 8) -> SumEquation:
    """X = L*A + B*U + C: L lowerTri, U upperTri, A, B, C general n x n."""
    g = Operand(n, n, GENERAL, "normal", 1.0 / np.sqrt(n))
    return SumEquation(f"LA_plus_BU_plus_C_{n}", seed,
                       ((Operand(n, n, LOWER_TRI), g), (g, Operand(n, n, UPPER_TRI)), (g,)),
                       ((False, False), (False, False), (False,)), ((0, 1), (2, 3), (4,)))


# --------------------------------------------------------------------------
# Nested expressions: an operand index, ("t", e), ("mul", [e, ...]) or
# ("add", [e, ...]) over a table of operands (paper Section 2, "Operations").
# --------------------------------------------------------------------------

@dataclass(frozen=True)
class Expression:
    name: str
    seed: int
    operands: Sequence[Operand]
    expr: object

    def descs(self):
        return [(o.rows, o.cols, o.prop) for o in self.operands]


def generate_expression(ex: Expression):
    """Stored float32 arrays of the operand table (None for Identity)."""
    return [generate_operand(o, ex.seed, i) for i, o in enumerate(ex.operands)]


def random_expression(seed: int, max_depth: int = 3, max_dim: int = 40, dim_multiple: int = 1,
                      diagonal: bool = False, kinds: bool = False) -> Expression:
    """Random well-formed nested expression; operands are reused where an existing one has the needed type.
    With `diagonal` some square operands are Diagonal (the streams without it are unchanged); with `kinds` some
    are strictly or unit triangular as well (a stream of its own)."""
    diagonal = diagonal or kinds
    rng = np.random.Generator(np.random.Philox(key=[int(seed), 0x7ED1A6 if kinds else 0xED1A6 if diagonal else 0xE4B8]))
    operands: List[Operand] = []

    def dim():
        return int(rng.integers(1, max_dim // dim_multiple + 1)) * dim_multiple

    def leaf(r, c):
        t = bool(rng.integers(0, 4) == 0)
        sr, sc = (c, r) if t else (r, c)
        same = [i for i, o in enumerate(operands) if (o.rows, o.cols) == (sr, sc)]
        if same and rng.random() < 0.5:
            i = int(rng.choice(same))
        else:
            kind = int(rng.integers(0, 13 if kinds else 9 if diagonal else 7))
            prop = {0: LOWER_TRI, 1: UPPER_TRI, 2: IDENTITY, 7: DIAGONAL, 8: DIAGONAL, 9: STRICT_LOWER, 10: STRICT_UPPER,
                    11: UNIT_LOWER, 12: UNIT_UPPER}.get(kind, GENERAL) if sr == sc else GENERAL
            operands.append(Operand(sr, sc, prop, "normal" if kind == 3 else "uniform"))
            i = len(operands) - 1
        return ("t", i) if t else i

    def gen(r, c, depth):
        kind = int(rng.integers(0, 10)) if depth > 0 else 0
        if kind <= 2:
            return leaf(r, c)
        if kind <= 5:
            n = int(rng.integers(2, 4))
            inner = [r] + [r if rng.random() < 0.3 else dim() for _ in range(n - 1)] + [c]
            return ("mul", [gen(inner[i], inner[i + 1], depth - 1) for i in range(n)])
        if kind <= 8:
            return ("add", [gen(r, c, depth - 1) for _ in range(int(rng.integers(2, 4)))])
        return ("t", gen(c, r, depth - 1))

    r = dim()
    c = r if rng.random() < 0.4 else dim()
    top = int(rng.integers(0, 3))
    if top == 0:
        expr = ("mul", [gen(r, r, max_depth - 1), ("add", [gen(r, c, max_depth - 2), gen(r, c, max_depth - 2)])])
    else:
        expr = gen(r, c, max_depth)
    return Expression(f"random_expr_{seed}", seed, tuple(operands), expr)


def config_expression(n: int = 4096, seed: int = 9) -> Expression:
    """X = (A + L) * (B + C^T) * U + D:  two nested sums, one chain of three factors, one Add term."""
    g = Operand(n, n, GENERAL, "normal", 1.0 / np.sqrt(n))
    ops = (g, Operand(n, n, LOWER_TRI), g, g, Operand(n, n, UPPER_TRI), g)
    expr = ("add", [("mul", [("add", [0, 1]), ("add", [2, ("t", 3)]), 4]), 5])
    return Expression(f"ApL_times_BpCt_times_U_plus_D_{n}", seed, ops, expr)
