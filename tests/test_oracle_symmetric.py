"""Pins of the oracle for the Symmetric property and for Gram products Y * Y^T (the paper's conclusion
announces more properties and algebraic transformations and prints no rule for them; every pin here comes
from counting, from exact symmetry of the fp64 triple loop, or from hand-computed costs)."""
import itertools

import numpy as np
import pytest

import workloads as wl
from oracle import plan as op
from oracle import values as ov
from oracle.plan import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I, DIAGONAL as D, SYMMETRIC as S, Desc


def test_gram_closed_forms_equal_brute_force_counts():
    for n in range(1, 8):
        for prop in (G, S, L, U):
            assert op.gram_mults(Desc(n, n, prop)) == op.brute_force_gram_mults(Desc(n, n, prop)), (n, prop)
        assert op.gram_mults(Desc(n, n + 3, G)) == op.brute_force_gram_mults(Desc(n, n + 3, G))
        assert op.gram_mults(Desc(n + 2, n, G)) == op.brute_force_gram_mults(Desc(n + 2, n, G))
    # the lower triangle of Y*Y^T needs one multiplication per (i >= j, l): k * m(m+1)/2
    assert op.gram_mults(Desc(10, 4, G)) == 4 * 55


def test_symmetric_type_rules():
    assert op.structural_nonzeros(Desc(6, 6, S)) == 36 and op.in_structure(S, 1, 4)
    assert op.product_mults(Desc(6, 6, S), Desc(6, 3, G)) == 6 * 6 * 3       # full structure: as a general matrix
    assert op.join(S, I) == S and op.join(I, S) == S
    for p in (G, L, U, D, S):
        assert op.join(S, p) == G and op.join(p, S) == G                      # S*S and D*S are not symmetric in general
    for a, b, c in itertools.product([G, L, U, I, D, S], repeat=3):
        assert op.join(op.join(a, b), c) == op.join(a, op.join(b, c))
    assert op.transpose_desc(Desc(5, 5, S)) == Desc(5, 5, S)
    assert op.sum_property(S, [S]) == S and op.sum_property(S, [D, I]) == S and op.sum_property(I, [S]) == S
    assert op.sum_property(S, [L]) == G and op.sum_property(U, [S]) == G and op.sum_property(S, [G]) == G
    with pytest.raises(op.OracleError):
        op.plan([(3, 4, S)])


def test_symmetric_sums_stay_symmetric_numerically():
    eq = wl.Equation("s", 51, (wl.Operand(9, 9, S),), (wl.Operand(9, 9, S, "normal"), wl.Operand(9, 9, D), wl.Operand(9, 9, I)))
    chain, add = wl.generate(eq)
    assert np.array_equal(chain[0], chain[0].T) and np.array_equal(add[0], add[0].T)
    x, _ = ov.evaluate(chain, eq.descs(), add, eq.add_descs())
    assert np.array_equal(x, x.T) and op.plan(eq.descs(), eq.add_descs()).result_desc.prop == S


def test_hand_costs_of_gram_products():
    a = (10, 4, G)
    # A * A^T, named: the lower triangle only; unnamed or not transposed: an ordinary product
    p = op.plan([a, (4, 10, G)], names=[0, 0])
    assert p.mults == 400 and p.result_desc.prop == G and not p.steps[0].gram          # A * A (4x10 is another matrix shape): no
    p = op.plan([a, a], chain_transposed=[False, True], names=[0, 0])
    assert (p.paren, p.mults) == ("(0*1^T)", 220) and p.result_desc == Desc(10, 10, S)
    assert p.steps[0].gram and (p.steps[0].lhs, p.steps[0].rhs, p.steps[0].m, p.steps[0].n, p.steps[0].k) == (0, 0, 10, 10, 4)
    assert op.plan([a, a], chain_transposed=[False, True]).mults == 400
    assert op.plan([a, a], chain_transposed=[False, True], names=[0, 1]).mults == 400
    # A^T * A is a Gram product of Y = A^T (4 x 10): 10 * 4*5/2
    p = op.plan([a, a], chain_transposed=[True, False], names=[0, 0])
    assert p.mults == 100 and p.result_desc == Desc(4, 4, S) and p.steps[0].gram
    # A * B * B^T * A^T, A 10x6, B 6x3: split in the middle: (A*B) 180, then the lower triangle of Y*Y^T with Y 10x3: 165
    b = (6, 3, G)
    p = op.plan([(10, 6, G), b, b, (10, 6, G)], chain_transposed=[False, False, True, True], names=[0, 1, 1, 0])
    assert (p.paren, p.mults) == ("((0*1)*(2^T*3^T))", 180 + 165) and p.result_desc.prop == S
    assert [(s.lhs, s.rhs, s.gram) for s in p.steps] == [(0, 1, False), (4, 4, True)]
    # the inner B * B^T alone is symmetric too, but using it costs more: 63 + 6*6*10 + 10*6*10
    assert 63 + 360 + 600 > p.mults
    # L * L^T (n = 6): entries i >= j, l <= j: n(n+1)(n+2)/6 = 56, against the sum of squares 91 of an ordinary L * U
    p = op.plan([(6, 6, L), (6, 6, L)], chain_transposed=[False, True], names=[3, 3])
    assert p.mults == 56 and p.result_desc.prop == S and p.steps[0].rhs_prop == U
    # a Symmetric factor is its own transpose: S * S reads as Y * Y^T
    p = op.plan([(6, 6, S), (6, 6, S)], names=[0, 0])
    assert p.mults == 6 * 21 and p.result_desc.prop == S
    # D * D^T stays Diagonal (cheaper than any Gram rule)
    p = op.plan([(6, 6, D), (6, 6, D)], chain_transposed=[False, True], names=[0, 0])
    assert p.mults == 6 and p.result_desc.prop == D


def test_gram_value_is_exactly_symmetric_and_steps_reproduce_it():
    eq = wl.Equation("g", 52, (wl.Operand(13, 7, G, "normal"), wl.Operand(7, 5, G), wl.Operand(7, 5, G), wl.Operand(13, 7, G, "normal")),
                     (), 1, (False, False, True, True))
    chain, _ = wl.generate(eq)
    chain[2], chain[3] = chain[1], chain[0]                       # the same matrices
    p = op.plan(eq.descs(), (), eq.chain_t, (), names=[0, 1, 1, 0])
    used, used_d = ov.transposed_operands(chain, eq.descs(), eq.chain_t)
    x, d = ov.evaluate(used, used_d)
    y = ov.evaluate_steps(chain, eq.descs(), p.steps)
    assert p.steps[-1].gram and np.array_equal(y, y.T)            # a_il*a_jl commutes exactly in the triple loop
    assert ov.normwise_error(y, x, d) <= 1e-12


def test_chosen_tree_is_a_minimum_under_independent_brute_force_costs():
    # every tree costed again with brute-force counts and a separately written test for "reads as Y * Y^T"
    rng = np.random.default_rng(31)
    grams = 0
    for _ in range(60):
        half = int(rng.integers(1, 4))
        left, cur = [], int(rng.integers(1, 6))
        for q in range(half):
            kind = int(rng.integers(0, 5))
            if kind == 0:
                left.append(((cur, cur, L), q, bool(rng.integers(0, 2))))
            elif kind == 1:
                left.append(((cur, cur, S), q, bool(rng.integers(0, 2))))
            else:
                nxt = int(rng.integers(1, 6))
                t = bool(rng.integers(0, 2))
                left.append((((nxt, cur, G) if t else (cur, nxt, G)), q, t))
                cur = nxt
        right = [(d, nm, (not t) if d[2] != S or rng.integers(0, 2) else t) for d, nm, t in reversed(left)]
        d0, _, t0 = left[0]
        y_rows = d0[1] if t0 else d0[0]                             # Y * Y^T is y_rows x y_rows
        extra = [((y_rows, int(rng.integers(1, 6)), G), 99, False)] if rng.integers(0, 2) else []   # sometimes one more factor
        factors = left + right + extra
        stored = [f[0] for f in factors]
        names = [f[1] for f in factors]
        flags = [f[2] for f in factors]
        used = [op.transpose_desc(Desc(*d)) if t else Desc(*d) for d, t in zip(stored, flags)]
        n = len(used)

        def mirror(lo, hi):
            if (hi - lo + 1) % 2:
                return False
            return all(names[lo + q] == names[hi - q] and (flags[lo + q] != flags[hi - q] or used[lo + q].prop in (S, D))
                       for q in range((hi - lo + 1) // 2))

        def brute(tree):
            if isinstance(tree, int):
                return used[tree], 0, (tree, tree)
            split, lt, rt = tree
            dl, cl, (lo, _) = brute(lt)
            dr, cr, (_, hi) = brute(rt)
            prop = op.join(dl.prop, dr.prop)
            gram = prop == G and mirror(lo, hi)
            node = Desc(dl.rows, dr.cols, S if gram else prop)
            if gram and split == (lo + hi - 1) // 2:
                return node, cl + op.brute_force_gram_mults(dl), (lo, hi)
            return node, cl + cr + op.brute_force_mults(dl, dr), (lo, hi)

        p = op.plan(stored, (), flags, (), names=names)
        assert p.mults == min(brute(t)[1] for t in op.all_trees(0, n - 1))
        grams += any(s.gram for s in p.steps)
    assert grams >= 20
