"""Plan oracle: exhaustive parenthesization of a Linnea Mul chain.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plainly-correct statement of what the planner must return.  It shares no
code with the CUDA library and must never be imported by the product path; only tests, the smoke
check and the benchmark's CPU-baseline leg use it.

What it follows (paper Section 2):
  * "Types": a Matrix is (property, static [rows, cols], element type); Identity is a square matrix
    with ones on the diagonal, there so that A*I = A and I*I = I can be expressed.
  * "Transformations": identity simplification (A*I -> A), matrix-chain reordering that "minimizes
    the number of scalar multiplications", generalised to account for matrix properties, and
    property propagation that turns the equation's Term into a concrete Matrix type.

The chain-reordering transformation is a dynamic program that reaches the minimum-cost binary tree;
the plain definition of that result is "the cheapest of ALL binary trees", so the oracle enumerates
every tree (Catalan many) and keeps the cheapest.

Readings taken where the paper is silent (each also listed in the design notes):
  * cost of one product = number of scalar multiplications a_il * b_lj in which BOTH factors are
    structurally non-zero (non-strict triangles: the diagonal is an ordinary entry);
  * Identity operands are removed before the enumeration and never appear in the result string;
  * ties: the tree whose pre-order list of split positions is lexicographically smallest;
  * property of a product = join in  Identity < Diagonal < {lowerTri, upperTri} < general;
  * Diagonal (one of the "more properties" the paper's conclusion announces; the paper prints no rule
    for it): a square matrix stored densely whose entries off the diagonal are zero.  Unlike Identity
    its diagonal is data, so it is never simplified away; D*A costs one multiplication per structural
    entry of A; the transpose of a Diagonal matrix is Diagonal;
  * Symmetric (another of those properties, again without a printed rule): a square matrix stored densely
    in full with a_ij = a_ji.  Its structure is full, so it costs what a general matrix costs; S^T = S; a
    product with a Symmetric factor is general (S*I = S); a sum of Symmetric, Diagonal and Identity
    summands is Symmetric;
  * Gram products: when the factors are named (equal names = the same matrix) and a sub-chain reads
    Y * Y^T factor by factor (second half = first half reversed, every factor transposed; Symmetric and
    Diagonal factors are their own transposes), its value is Symmetric whatever the tree, and the tree that
    splits it in the middle computes only Y and then the lower triangle of Y * Y^T: the right half costs
    nothing and the product costs the multiplications of the entries (i, j) with i >= j;
  * strictly triangular and unit triangular (two more of those properties; no printed rule): square, stored
    densely; a strictly triangular matrix also has zeros on its diagonal, a unit triangular one has ones there
    (stored as 1.0).  An entry known to be 1 needs no multiplication, exactly as Identity needs none: a
    multiplication a_il * b_lj counts only when both entries are structural non-zeros and neither is a known 1.
    So a unit triangle costs what the strict one costs.  Within one orientation a product's diagonal is the
    product of the diagonals (zero if either is zero, one if both are one); in a sum the diagonals add
    (zero + zero = zero, zero + one = one, anything else is ordinary data), so I + strictly lower = unit lower;
  * a transposed operand (paper Table 1, "Transpose") takes part with its transposed type: shape
    swapped and lowerTri <-> upperTri (the inference rule the paper prints), likewise for the strict and unit kinds;
  * reported mul_flops = 2 * multiplications; add_flops = structural non-zeros of the Add terms.
    (The factor 2 and the add_flops convention are bookkeeping of this project: parity unpinned by
    the paper, which only speaks of scalar multiplications.)
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

GENERAL, LOWER_TRI, UPPER_TRI, IDENTITY, DIAGONAL, SYMMETRIC = 0, 1, 2, 3, 4, 5
STRICT_LOWER, STRICT_UPPER, UNIT_LOWER, UNIT_UPPER = 6, 7, 8, 9
PROPERTIES = (GENERAL, LOWER_TRI, UPPER_TRI, IDENTITY, DIAGONAL, SYMMETRIC,
              STRICT_LOWER, STRICT_UPPER, UNIT_LOWER, UNIT_UPPER)
LOWER_KINDS = (LOWER_TRI, STRICT_LOWER, UNIT_LOWER)
UPPER_KINDS = (UPPER_TRI, STRICT_UPPER, UNIT_UPPER)


class OracleError(ValueError):
    """Raised with a short reason code: 'invalid_arg', 'property', 'shape_mismatch'."""

    def __init__(self, code: str, msg: str = ""):
        super().__init__(f"{code}: {msg}" if msg else code)
        self.code = code


@dataclass(frozen=True)
class Desc:
    rows: int
    cols: int
    prop: int


@dataclass(frozen=True)
class Step:
    lhs: int          # ids: 0..n-1 original chain operands, n.. intermediates in emission order
    rhs: int
    out: int
    m: int
    n: int
    k: int
    lhs_prop: int
    rhs_prop: int
    out_prop: int
    mults: int
    gram: bool = False   # out = lhs * lhs^T (rhs is the same value, read transposed); only entries i >= j are counted


@dataclass(frozen=True)
class Plan:
    paren: str
    mults: int
    mul_flops: int
    add_flops: int
    steps: Tuple[Step, ...]
    product_desc: Desc     # the Mul chain's value before the Add terms
    result_desc: Desc      # the equation's Term made concrete
    kept: Tuple[int, ...]  # original indices that survive identity simplification


# ----------------------------------------------------------------------------------------------
# structure and cost of one product
# ----------------------------------------------------------------------------------------------

def in_structure(prop: int, i: int, j: int) -> bool:
    """Is entry (i, j) a structural non-zero of a matrix with this property?"""
    if prop in (GENERAL, SYMMETRIC):
        return True
    if prop in (LOWER_TRI, UNIT_LOWER):
        return i >= j
    if prop in (UPPER_TRI, UNIT_UPPER):
        return i <= j
    if prop == STRICT_LOWER:
        return i > j
    if prop == STRICT_UPPER:
        return i < j
    if prop in (IDENTITY, DIAGONAL):
        return i == j
    raise OracleError("property", f"unknown property {prop}")


def known_one(prop: int, i: int, j: int) -> bool:
    """Is entry (i, j) known to be 1 from the type alone?  (The diagonal of Identity and of the unit triangles.)"""
    return i == j and prop in (IDENTITY, UNIT_LOWER, UNIT_UPPER)


def multiplies(prop: int, i: int, j: int) -> bool:
    """Does entry (i, j) take part in multiplications: a structural non-zero that is not a known 1?"""
    return in_structure(prop, i, j) and not known_one(prop, i, j)


def brute_force_nonzeros(d: Desc) -> int:
    """Structural non-zeros by counting (tiny shapes; used to check `structural_nonzeros`)."""
    return sum(1 for i in range(d.rows) for j in range(d.cols) if in_structure(d.prop, i, j))


def structural_nonzeros(d: Desc) -> int:
    if d.prop in (GENERAL, SYMMETRIC):
        return d.rows * d.cols
    if d.prop in (LOWER_TRI, UPPER_TRI, UNIT_LOWER, UNIT_UPPER):
        return d.rows * (d.rows + 1) // 2
    if d.prop in (STRICT_LOWER, STRICT_UPPER):
        return d.rows * (d.rows - 1) // 2
    return d.rows                   # Identity, Diagonal


def multiplying_entries(d: Desc) -> int:
    """Structural non-zeros that are not known ones (what a Diagonal factor has to scale)."""
    if d.prop == IDENTITY:
        return 0
    if d.prop in (UNIT_LOWER, UNIT_UPPER):
        return d.rows * (d.rows - 1) // 2
    return structural_nonzeros(d)


def brute_force_mults(a: Desc, b: Desc) -> int:
    """#{(i, l, j): (i, l) and (l, j) both structural non-zeros, neither a known 1} by counting, for tiny shapes."""
    assert a.cols == b.rows
    count = 0
    for i in range(a.rows):
        for l in range(a.cols):
            if not multiplies(a.prop, i, l):
                continue
            for j in range(b.cols):
                if multiplies(b.prop, l, j):
                    count += 1
    return count


def product_mults(a: Desc, b: Desc) -> int:
    """Useful scalar multiplications of A*B in closed form (both operands non-Identity)."""
    assert a.cols == b.rows
    ta = a.prop in LOWER_KINDS + UPPER_KINDS
    tb = b.prop in LOWER_KINDS + UPPER_KINDS
    if a.prop == IDENTITY or b.prop == IDENTITY:
        return 0
    if a.prop == DIAGONAL:         # row l of B is scaled by d_l: one multiplication per multiplying entry of B
        return multiplying_entries(b)
    if b.prop == DIAGONAL:         # column l of A is scaled by d_l
        return multiplying_entries(a)
    if not ta and not tb:
        return a.rows * a.cols * b.cols
    # a strict or unit triangle multiplies with the entries strictly off its diagonal only
    sa = 0 if a.prop in (LOWER_TRI, UPPER_TRI) else 1
    sb = 0 if b.prop in (LOWER_TRI, UPPER_TRI) else 1
    if ta and not tb:
        n = a.rows
        return b.cols * (n * (n + 1) // 2 - sa * n)
    if tb and not ta:
        n = b.rows
        return a.rows * (n * (n + 1) // 2 - sb * n)
    n = a.rows
    if (a.prop in LOWER_KINDS) == (b.prop in LOWER_KINDS):
        # L*L: triples i >= l + sa, l >= j + sb: choose three of n + 2 - sa - sb places
        t = n + 2 - sa - sb
        return t * (t - 1) * (t - 2) // 6
    # L*U (U*L): column l of A and row l of B both hold t = n - l (l + 1) entries, less the excluded diagonal:
    # sum over t = 1..n of (t - sa)(t - sb)
    return n * (n + 1) * (2 * n + 1) // 6 - (sa + sb) * n * (n + 1) // 2 + sa * sb * n


def brute_force_gram_mults(y: Desc) -> int:
    """#{(i, l, j): i >= j, (i, l) in S(Y) and (j, l) in S(Y)}: the multiplications of the lower triangle of Y*Y^T."""
    return sum(1 for i in range(y.rows) for j in range(i + 1) for l in range(y.cols)
               if multiplies(y.prop, i, l) and multiplies(y.prop, j, l))


def gram_mults(y: Desc) -> int:
    """The same in closed form (Y general, Symmetric or one of the triangular kinds)."""
    if y.prop in (LOWER_TRI, UPPER_TRI):
        n = y.rows
        return n * (n + 1) * (n + 2) // 6
    if y.prop in LOWER_KINDS + UPPER_KINDS:     # strict or unit: the diagonal takes no part
        n = y.rows
        return (n + 1) * n * (n - 1) // 6
    return y.cols * y.rows * (y.rows + 1) // 2


def _region(p: int) -> str:
    """Where the structural non-zeros may lie: 'D'iagonal, 'L'ower, 'U'pper, 'S'ymmetric (full), 'G'eneral (full)."""
    if p in LOWER_KINDS:
        return "L"
    if p in UPPER_KINDS:
        return "U"
    return {GENERAL: "G", SYMMETRIC: "S", IDENTITY: "D", DIAGONAL: "D"}[p]


def _diagonal(p: int) -> str:
    """What the type says about the diagonal: 'zero', 'one' or ordinary 'data'."""
    if p in (STRICT_LOWER, STRICT_UPPER):
        return "zero"
    if p in (IDENTITY, UNIT_LOWER, UNIT_UPPER):
        return "one"
    return "data"


def _triangle(region: str, diagonal: str) -> int:
    kinds = {"data": (LOWER_TRI, UPPER_TRI), "zero": (STRICT_LOWER, STRICT_UPPER), "one": (UNIT_LOWER, UNIT_UPPER)}
    return kinds[diagonal][0 if region == "L" else 1]


def join(p: int, q: int) -> int:
    """Property of a product: least upper bound in Identity < Diagonal < {lowerTri, upperTri} < general;
    a product with a Symmetric factor is general (only S*I = S).  Inside one triangle the diagonal of the
    product is the entrywise product of the diagonals: zero if either is zero, one if both are one."""
    if p == IDENTITY:
        return q
    if q == IDENTITY:
        return p
    if SYMMETRIC in (p, q):
        return GENERAL
    rp, rq = _region(p), _region(q)
    if rp == "D" and rq == "D":
        return DIAGONAL
    region = rq if rp == "D" else rp if rq == "D" else rp if rp == rq else "G"
    if region not in ("L", "U"):
        return GENERAL
    dp, dq = _diagonal(p), _diagonal(q)
    return _triangle(region, "zero" if "zero" in (dp, dq) else "one" if dp == dq == "one" else "data")


def sum_property(product_prop: int, add_props: Sequence[int]) -> int:
    """Property of (chain value) + T1 + ... + Tk.  With no terms it is the product's own property.

    A sum with at least one term is never typed Identity (I + I = 2I): an Identity summand counts
    through its footprint, the diagonal, so it is joined as a Diagonal matrix.  The result is the
    least type that holds every summand's footprint: Diagonal < {lowerTri, upperTri} < general.
    """
    if not add_props:
        return product_prop
    summands = [product_prop] + list(add_props)
    if SYMMETRIC in summands:       # Symmetric + (Symmetric | Diagonal | Identity) is Symmetric; a triangle or a general summand breaks it
        return SYMMETRIC if all(p in (SYMMETRIC, DIAGONAL, IDENTITY) for p in summands) else GENERAL
    regions = {_region(p) for p in summands}
    if "G" in regions or {"L", "U"} <= regions:
        return GENERAL
    if regions == {"D"}:
        return DIAGONAL
    # one triangle (plus diagonal summands): the diagonals add up
    diagonal = "zero"
    for p in summands:
        d = _diagonal(p)
        diagonal = d if diagonal == "zero" else diagonal if d == "zero" else "data"
    return _triangle("L" if "L" in regions else "U", diagonal)


# ----------------------------------------------------------------------------------------------
# validation and identity simplification
# ----------------------------------------------------------------------------------------------

def _validate(chain: Sequence[Desc], add: Sequence[Desc]) -> None:
    if len(chain) < 1:
        raise OracleError("invalid_arg", "empty chain")
    for d in list(chain) + list(add):
        if d.rows < 1 or d.cols < 1:
            raise OracleError("invalid_arg", "non-positive dimension")
        if d.prop not in PROPERTIES:
            raise OracleError("property", "unknown property")
        if d.prop != GENERAL and d.rows != d.cols:
            raise OracleError("property", "triangular / Diagonal / Symmetric / Identity matrices are square")
    for a, b in zip(chain[:-1], chain[1:]):
        if a.cols != b.rows:
            raise OracleError("shape_mismatch", "inner dimensions differ")
    rows, cols = chain[0].rows, chain[-1].cols
    for t in add:
        if (t.rows, t.cols) != (rows, cols):
            raise OracleError("shape_mismatch", "Add term shape differs from the chain's")


# ----------------------------------------------------------------------------------------------
# exhaustive enumeration
# ----------------------------------------------------------------------------------------------

# A tree over reduced positions lo..hi is either the int `lo` (a leaf, lo == hi) or (split, left, right)
# where left covers lo..split and right covers split+1..hi.

def all_trees(lo: int, hi: int):
    if lo == hi:
        yield lo
        return
    for split in range(lo, hi):
        for left in all_trees(lo, split):
            for right in all_trees(split + 1, hi):
                yield (split, left, right)


def _span(tree) -> Tuple[int, int]:
    if isinstance(tree, int):
        return tree, tree
    _, left, right = tree
    return _span(left)[0], _span(right)[1]


def _reads_as_gram(lo: int, hi: int, descs: Sequence[Desc], ident) -> bool:
    """Do the factors lo..hi read Y * Y^T?  `ident[i]` = (name, transposed) of factor i, or None when nothing
    is known about it.  Factor hi - q must be the transpose of factor lo + q: the same matrix with the other
    flag, or the same matrix with any flag when it is its own transpose (Symmetric, Diagonal)."""
    if ident is None or (hi - lo + 1) % 2:
        return False
    for q in range((hi - lo + 1) // 2):
        a, b = ident[lo + q], ident[hi - q]
        if a is None or b is None or a[0] != b[0]:
            return False
        if a[1] == b[1] and descs[lo + q].prop not in (SYMMETRIC, DIAGONAL):
            return False
    return True


def _tree_desc_cost(tree, descs: Sequence[Desc], ident=None) -> Tuple[Desc, int]:
    if isinstance(tree, int):
        return descs[tree], 0
    split, left, right = tree
    lo, hi = _span(tree)
    dl, cl = _tree_desc_cost(left, descs, ident)
    dr, cr = _tree_desc_cost(right, descs, ident)
    prop = join(dl.prop, dr.prop)
    gram = prop == GENERAL and _reads_as_gram(lo, hi, descs, ident)
    node = Desc(dl.rows, dr.cols, SYMMETRIC if gram else prop)
    if gram and 2 * split == lo + hi - 1:           # split in the middle: the right half is never computed
        return node, cl + gram_mults(dl)
    return node, cl + cr + product_mults(dl, dr)


def _preorder_splits(tree) -> List[int]:
    if isinstance(tree, int):
        return []
    split, left, right = tree
    return [split] + _preorder_splits(left) + _preorder_splits(right)


def _paren(tree, kept: Sequence[int], transposed: Sequence[bool] = ()) -> str:
    if isinstance(tree, int):
        i = kept[tree]
        return str(i) + ("^T" if transposed and transposed[i] else "")
    _, left, right = tree
    return "(" + _paren(left, kept, transposed) + "*" + _paren(right, kept, transposed) + ")"


def transpose_desc(d: Desc) -> Desc:
    """Type of A^T given the type of A: shape swapped; paper Section 2, "Transformations", prints the
    inference rule lowerTriangular(A) -> upperTriangular(A^T) (and symmetrically); general, Diagonal,
    Symmetric and Identity keep their property."""
    swap = {LOWER_TRI: UPPER_TRI, UPPER_TRI: LOWER_TRI, STRICT_LOWER: STRICT_UPPER, STRICT_UPPER: STRICT_LOWER,
            UNIT_LOWER: UNIT_UPPER, UNIT_UPPER: UNIT_LOWER}
    return Desc(d.cols, d.rows, swap.get(d.prop, d.prop))


def plan(chain: Sequence[Tuple[int, int, int]], add: Sequence[Tuple[int, int, int]] = (),
         chain_transposed: Sequence[bool] = (), add_transposed: Sequence[bool] = (),
         names: Optional[Sequence[int]] = None) -> Plan:
    """Plan `X = prod(chain) + sum(add)`; operands are (rows, cols, property) triples of the STORED matrices.

    `chain_transposed[i]` / `add_transposed[i]` say that the equation uses the transpose of that operand
    (paper Table 1, "Transpose"); the plan then works with the transposed type and prints the operand as `i^T`.
    `names[i]` identifies the matrix behind chain operand i (equal names = the same matrix); only with names can
    a sub-chain be recognised as a Gram product Y * Y^T.
    """
    stored_c = [Desc(*c) for c in chain]
    stored_a = [Desc(*a) for a in add]
    for d in stored_c + stored_a:               # the stored matrices must be well-typed themselves
        if d.prop not in PROPERTIES:
            raise OracleError("property", "unknown property")
    tc = list(chain_transposed) + [False] * (len(stored_c) - len(chain_transposed))
    ta = list(add_transposed) + [False] * (len(stored_a) - len(add_transposed))
    cdescs = [transpose_desc(d) if t else d for d, t in zip(stored_c, tc)]
    adescs = [transpose_desc(d) if t else d for d, t in zip(stored_a, ta)]
    _validate(cdescs, adescs)
    n = len(cdescs)
    rows, cols = cdescs[0].rows, cdescs[-1].cols

    kept = tuple(i for i, d in enumerate(cdescs) if d.prop != IDENTITY)
    add_flops = sum(structural_nonzeros(t) for t in adescs)

    if not kept:     # I*I*...*I = I
        product = Desc(rows, cols, IDENTITY)
        return Plan("I", 0, 0, add_flops, (), product,
                    Desc(rows, cols, sum_property(IDENTITY, [t.prop for t in adescs])), kept)

    reduced = [cdescs[i] for i in kept]
    ident = None if names is None else [(names[i], bool(tc[i])) for i in kept]
    best = None
    for tree in all_trees(0, len(reduced) - 1):
        _, cost = _tree_desc_cost(tree, reduced, ident)
        key = (cost, _preorder_splits(tree))
        if best is None or key < best[0]:
            best = (key, tree)
    (cost, _), tree = best

    steps: List[Step] = []
    next_id = [n]

    def emit(t) -> Tuple[int, Desc]:
        if isinstance(t, int):
            return kept[t], reduced[t]
        split, left, right = t
        lo, hi = _span(t)
        lid, ld = emit(left)
        oid_prop = _tree_desc_cost(t, reduced, ident)[0].prop
        if oid_prop == SYMMETRIC and 2 * split == lo + hi - 1 and _reads_as_gram(lo, hi, reduced, ident):
            # Y * Y^T: the right half is the same value read transposed; nothing is emitted for it
            rt = transpose_desc(ld)
            oid = next_id[0]
            next_id[0] += 1
            steps.append(Step(lid, lid, oid, ld.rows, ld.rows, ld.cols, ld.prop, rt.prop, SYMMETRIC, gram_mults(ld), True))
            return oid, Desc(ld.rows, ld.rows, SYMMETRIC)
        rid, rd = emit(right)
        out = Desc(ld.rows, rd.cols, oid_prop)
        oid = next_id[0]
        next_id[0] += 1
        steps.append(Step(lid, rid, oid, ld.rows, rd.cols, ld.cols, ld.prop, rd.prop, out.prop,
                          product_mults(ld, rd)))
        return oid, out

    _, product = emit(tree)
    assert sum(s.mults for s in steps) == cost
    result = Desc(rows, cols, sum_property(product.prop, [t.prop for t in adescs]))
    return Plan(_paren(tree, kept, tc), cost, 2 * cost, add_flops, tuple(steps), product, result, kept)


def catalan(r: int) -> int:
    """Number of binary trees over r leaves (r >= 1)."""
    c = 1
    for i in range(r - 1):
        c = c * 2 * (2 * i + 1) // (i + 2)
    return c


# ----------------------------------------------------------------------------------------------
# sums of several Mul chains
# ----------------------------------------------------------------------------------------------
# Paper Section 2, "Operations": an Equation holds a bag of Mul and Add operations, both variadic, so
# its value can be a sum of several products,  X = prod(chain_1) + ... + prod(chain_c);  a chain of
# one factor is a plain Add term.  Readings taken here (the paper gives no rule):
#   * Add is linear in each summand, so every chain is parenthesized on its own, exactly as `plan` does;
#   * factors are numbered 0..F-1 across all chains in the order written, intermediates F.. in the order
#     the chains' products are emitted (chain by chain, each in post-order);
#   * reuse between chains: a product below the root of its chain's tree is computed once when the same
#     run of factors (same matrix names, same transposition flags) was already multiplied by an earlier
#     chain, also below that chain's root; its multiplications are then counted once.  A chain's root
#     product is never shared: it is what the chain adds to X;
#   * the result property folds `sum_property` over the chains' product types;
#   * add_flops = structural non-zeros of every summand after the first.

@dataclass(frozen=True)
class SumPlan:
    paren: str
    mults: int
    mul_flops: int
    add_flops: int
    steps: Tuple[Step, ...]        # global ids, reused products appear once
    chain_values: Tuple[int, ...]  # per chain: id of its value (a factor id, a step's out), -1 for Identity
    chain_descs: Tuple[Desc, ...]  # per chain: type of its product
    result_desc: Desc
    reused: int                    # products not emitted because an earlier chain computed them


def plan_sum(chains: Sequence[Sequence[Tuple[int, int, int]]],
             transposed: Sequence[Sequence[bool]] = (),
             names: Sequence[Sequence[int]] = ()) -> SumPlan:
    """Plan X = sum over chains of prod(chain).  `names[c][f]` identifies the matrix behind factor f of
    chain c (equal names = the same stored matrix); without names every factor is its own matrix."""
    if len(chains) < 1:
        raise OracleError("invalid_arg", "no chain")
    flags = [list(transposed[c]) if c < len(transposed) else [] for c in range(len(chains))]
    flags = [f + [False] * (len(ch) - len(f)) for f, ch in zip(flags, chains)]
    total = sum(len(ch) for ch in chains)
    if names:
        if [len(n) for n in names] != [len(ch) for ch in chains]:
            raise OracleError("invalid_arg", "names do not match the chains")
        by_name = {}
        for ch, fl, nm in zip(chains, flags, names):
            for d, n in zip(ch, nm):
                if by_name.setdefault(n, tuple(d)) != tuple(d):
                    raise OracleError("invalid_arg", "one name, two types")
    else:
        counter = iter(range(total))
        names = [[next(counter) for _ in ch] for ch in chains]

    plans = [plan(ch, (), fl, (), nm) for ch, fl, nm in zip(chains, flags, names)]
    rows, cols = plans[0].product_desc.rows, plans[0].product_desc.cols
    for p in plans[1:]:
        if (p.product_desc.rows, p.product_desc.cols) != (rows, cols):
            raise OracleError("shape_mismatch", "summands differ in shape")

    steps: List[Step] = []
    seen = {}                      # (names and flags of a factor run) -> global id of its product
    reused = 0
    next_id = total
    base = 0
    values: List[int] = []
    parens: List[str] = []
    for c, (p, ch) in enumerate(zip(plans, chains)):
        n_local = len(ch)
        # local id -> the run of (name, transposed) factors it multiplies; the right half of a Gram product
        # Y * Y^T is Y's run reversed with every flag flipped
        run = {i: ((names[c][i], flags[c][i]),) for i in range(n_local)}
        to_global = {i: base + i for i in range(n_local)}
        for s in p.steps:
            if s.gram:
                run[s.out] = run[s.lhs] + tuple((nm, not fl) for nm, fl in reversed(run[s.lhs]))
            else:
                run[s.out] = run[s.lhs] + run[s.rhs]
            kept_run = run[s.out]
            is_root = s is p.steps[-1]
            if not is_root and kept_run in seen:
                to_global[s.out] = seen[kept_run]
                reused += 1
                continue
            gid = next_id
            next_id += 1
            to_global[s.out] = gid
            if not is_root:
                seen[kept_run] = gid
            steps.append(Step(to_global[s.lhs], to_global[s.rhs], gid, s.m, s.n, s.k,
                              s.lhs_prop, s.rhs_prop, s.out_prop, s.mults, s.gram))
        if p.steps:
            values.append(to_global[p.steps[-1].out])
        elif p.kept:
            values.append(base + p.kept[0])
        else:
            values.append(-1)
        # the chain's string with its factor numbers moved to the global numbering
        out, num = [], ""
        for chr_ in p.paren + "\0":
            if chr_.isdigit():
                num += chr_
                continue
            if num:
                out.append(str(int(num) + base))
                num = ""
            if chr_ != "\0":
                out.append(chr_)
        parens.append("".join(out))
        base += n_local

    mults = sum(s.mults for s in steps)
    descs = tuple(p.product_desc for p in plans)
    result_prop = sum_property(descs[0].prop, [d.prop for d in descs[1:]])
    add_flops = sum(structural_nonzeros(d) for d in descs[1:])
    return SumPlan("+".join(parens), mults, 2 * mults, add_flops, tuple(steps), tuple(values), descs,
                   Desc(rows, cols, result_prop), reused)


# ----------------------------------------------------------------------------------------------
# nested expressions
# ----------------------------------------------------------------------------------------------
# Paper Section 2, "Operations": the body of an Equation is a bag of Mul, Add and Transpose operations
# that is walked from the yield, so Mul and Add may nest:  A*(B + C),  (A + B)^T * C,  ...
# An expression is written here as a nested Python value:
#     int i                     operand i of the operand table
#     ("t", e)                  transpose of e
#     ("mul", [e1, e2, ...])    product, left to right
#     ("add", [e1, e2, ...])    sum
# Readings (the paper gives no rule for any of this):
#   * transposes are pushed down to the operands: (e1*e2)^T = e2^T*e1^T, (e1+e2)^T = e1^T+e2^T, (e^T)^T = e;
#   * a product inside a product and a sum inside a sum are flattened (associativity);
#   * a sum inside a product is MATERIALIZED: it is evaluated on its own (as a sum of chains, see `plan_sum`)
#     into a temporary whose type is the sum's result type, and the temporary is one factor of the outer
#     chain.  Nothing is distributed: A*(B+C) costs one product and one addition;
#   * two nested sums with the same normal form are the same temporary, evaluated once;
#   * sharing of products (`plan_sum`) works within one sum; operands are named by their index, a temporary
#     by its normal form;
#   * nested sums are planned before the sum that uses them, in order of first appearance;
#   * in the string an operand prints as its index (with ^T), a temporary as [its sum's string].

@dataclass(frozen=True)
class ExprPlan:
    paren: str
    mults: int
    mul_flops: int
    add_flops: int
    result_desc: Desc
    products: Tuple[Tuple[int, int, int, int, int, int, int], ...]   # (m, n, k, lhs_prop, rhs_prop, out_prop, mults) in order
    reused: int
    temporaries: int       # distinct nested sums that were materialized


def normalize_expr(expr, transposed: bool = False):
    """Normal form: a sum = tuple of chains; a chain = tuple of factors; a factor = ("leaf", operand, t) or
    ("sum", <normal form of the nested sum>)."""
    if isinstance(expr, int):
        return ((("leaf", expr, transposed),),)
    kind = expr[0]
    if kind == "t":
        return normalize_expr(expr[1], not transposed)
    children = list(expr[1])
    if not children:
        raise OracleError("invalid_arg", "operation without operands")
    if kind == "add":
        out = []
        for c in children:
            out.extend(normalize_expr(c, transposed))
        return tuple(out)
    if kind == "mul":
        if transposed:
            children.reverse()
        chain = []
        for c in children:
            s = normalize_expr(c, transposed)
            if len(s) == 1:
                chain.extend(s[0])
            else:
                chain.append(("sum", s))
        return (tuple(chain),)
    raise OracleError("invalid_arg", f"unknown operation {kind!r}")


def plan_expr(expr, operands: Sequence[Tuple[int, int, int]]) -> ExprPlan:
    stored = [Desc(*d) for d in operands]
    temporaries = {}                  # normal form -> (name, result Desc, string)
    products: List[Tuple[int, ...]] = []
    totals = {"mults": 0, "add": 0, "reused": 0}

    def plan_one(sum_nf) -> Tuple[Desc, str]:
        chains, flags, names, labels = [], [], [], []
        for chain in sum_nf:
            cd, cf, cn, cl = [], [], [], []
            for f in chain:
                if f[0] == "leaf":
                    _, i, t = f
                    if not 0 <= i < len(stored):
                        raise OracleError("invalid_arg", "operand index out of range")
                    cd.append(tuple(operands[i])); cf.append(t); cn.append(i); cl.append(str(i))
                else:
                    nf = f[1]
                    if nf not in temporaries:
                        desc, text = plan_one(nf)
                        temporaries[nf] = (len(stored) + len(temporaries), desc, text)
                    name, desc, text = temporaries[nf]
                    cd.append((desc.rows, desc.cols, desc.prop)); cf.append(False); cn.append(name)
                    cl.append("[" + text + "]")
            chains.append(cd); flags.append(cf); names.append(cn); labels.extend(cl)
        sp = plan_sum(chains, flags, names)
        totals["mults"] += sp.mults
        totals["add"] += sp.add_flops
        totals["reused"] += sp.reused
        products.extend((s.m, s.n, s.k, s.lhs_prop, s.rhs_prop, s.out_prop, s.mults) for s in sp.steps)
        # positions -> labels
        out, num = [], ""
        for ch in sp.paren + "\0":
            if ch.isdigit():
                num += ch
                continue
            if num:
                out.append(labels[int(num)])
                num = ""
            if ch != "\0":
                out.append(ch)
        return sp.result_desc, "".join(out)

    desc, text = plan_one(normalize_expr(expr))
    return ExprPlan(text, totals["mults"], 2 * totals["mults"], totals["add"], desc, tuple(products),
                    totals["reused"], len(temporaries))
