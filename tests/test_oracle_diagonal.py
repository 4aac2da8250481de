"""Pins of the oracle for the Diagonal property (one of the "more properties" the paper's conclusion
announces; the paper prints no rule for it, so every pin here comes from the mathematics: counting,
Boolean structure products, and NumPy broadcasting as the textbook form of a diagonal scaling)."""
import itertools

import numpy as np
import pytest

import workloads as wl
from oracle import plan as op
from oracle import values as ov
from oracle.plan import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I, DIAGONAL as D, Desc


def test_hand_costs_of_products_with_a_diagonal_factor():
    # D*A scales the rows of A: one multiplication per structural entry of A (and likewise A*D)
    assert op.product_mults(Desc(7, 7, D), Desc(7, 3, G)) == 21
    assert op.product_mults(Desc(5, 7, G), Desc(7, 7, D)) == 35
    assert op.product_mults(Desc(6, 6, D), Desc(6, 6, L)) == 21
    assert op.product_mults(Desc(6, 6, U), Desc(6, 6, D)) == 21
    assert op.product_mults(Desc(6, 6, D), Desc(6, 6, D)) == 6


def test_the_diagonal_factor_joins_the_cheaper_side():
    # A (30x20) * D (20) * B (20x50): (A*D) costs 600, (D*B) costs 1000; the big product costs 30000 either way
    p = op.plan([(30, 20, G), (20, 20, D), (20, 50, G)])
    assert (p.paren, p.mults) == ("((0*1)*2)", 600 + 30_000)
    p = op.plan([(50, 20, G), (20, 20, D), (20, 30, G)])
    assert (p.paren, p.mults) == ("(0*(1*2))", 600 + 30_000)
    # a tie (square): smallest pre-order split list, i.e. 0*(1*2)
    p = op.plan([(8, 8, G), (8, 8, D), (8, 8, G)])
    assert (p.paren, p.mults) == ("(0*(1*2))", 64 + 512)
    # L * D * U at n = 6: D goes to either triangle for 21, then L*U costs the sum of squares 91
    p = op.plan([(6, 6, L), (6, 6, D), (6, 6, U)])
    assert p.mults == 21 + 91 and p.result_desc == Desc(6, 6, G)
    # D * D * A: (D*D) first costs 6 + 6*4, A first costs 24 + 24
    p = op.plan([(6, 6, D), (6, 6, D), (6, 4, G)])
    assert (p.paren, p.mults) == ("((0*1)*2)", 6 + 24)
    assert [s.out_prop for s in p.steps] == [D, G]


def test_a_diagonal_operand_is_never_simplified_away():
    p = op.plan([(9, 9, D), (9, 9, I), (9, 4, G)])
    assert (p.paren, p.kept, p.mults) == ("(0*2)", (0, 2), 36)
    p = op.plan([(9, 9, D)])
    assert (p.paren, len(p.steps)) == ("0", 0) and p.result_desc == Desc(9, 9, D)
    p = op.plan([(9, 9, D)], chain_transposed=[True])
    assert p.paren == "0^T" and p.result_desc == Desc(9, 9, D)


def test_chosen_tree_is_a_minimum_under_brute_force_costs_with_diagonals():
    rng = np.random.default_rng(23)
    seen_diag = 0
    for _ in range(40):
        n = int(rng.integers(2, 6))
        cur = int(rng.integers(1, 6))
        chain = []
        for _ in range(n):
            kind = int(rng.integers(0, 6))
            if kind < 3:
                chain.append((cur, cur, (L, U, D)[kind]))
                seen_diag += kind == 2
            else:
                nxt = int(rng.integers(1, 6))
                chain.append((cur, nxt, G))
                cur = nxt
        descs = [Desc(*c) for c in chain]

        def brute(tree):
            if isinstance(tree, int):
                return descs[tree], 0
            _, lt, rt = tree
            dl, cl = brute(lt)
            dr, cr = brute(rt)
            return Desc(dl.rows, dr.cols, op.join(dl.prop, dr.prop)), cl + cr + op.brute_force_mults(dl, dr)

        assert op.plan(chain).mults == min(brute(t)[1] for t in op.all_trees(0, n - 1))
    assert seen_diag > 10


def test_sum_type_is_the_least_type_that_holds_every_footprint():
    n = 4
    order = {D: 0, L: 1, U: 1, G: 2}

    def footprint(p):
        return np.array([[op.in_structure(p, i, j) for j in range(n)] for i in range(n)])

    for props in itertools.chain(itertools.product([G, L, U, I, D], repeat=2), itertools.product([G, L, U, I, D], repeat=3)):
        got = op.sum_property(props[0], props[1:])
        union = np.zeros((n, n), dtype=bool)
        for p in props:
            union |= footprint(p)
        assert got != I
        assert not (union & ~footprint(got)).any(), props                 # it holds the sum
        for smaller in (D, L, U, G):                                        # and nothing smaller does
            if order[smaller] < order[got]:
                assert (union & ~footprint(smaller)).any(), (props, smaller)


def test_diagonal_products_are_scalings():
    # the dense fp64 triple loop against NumPy broadcasting (the textbook form of D*A and A*D)
    eq = wl.Equation("DA", 41, (wl.Operand(37, 37, D), wl.Operand(37, 22, G)))
    (d, a), _ = wl.generate(eq)
    assert np.count_nonzero(d) == 37 and np.array_equal(d, np.diag(np.diag(d)))
    x, den = ov.evaluate([d, a], eq.descs())
    want = np.diag(d).astype(np.float64)[:, None] * a.astype(np.float64)
    assert np.array_equal(x, want) and np.array_equal(den, np.abs(want))

    eq = wl.Equation("AD", 42, (wl.Operand(19, 37, G), wl.Operand(37, 37, D)))
    (a, d), _ = wl.generate(eq)
    x, _ = ov.evaluate([a, d], eq.descs())
    assert np.array_equal(x, a.astype(np.float64) * np.diag(d).astype(np.float64)[None, :])

    # D1 * L * D2 keeps the triangle; D1 * D2 stays diagonal: exact zeros elsewhere
    eq = wl.Equation("DLD", 43, (wl.Operand(16, 16, D), wl.Operand(16, 16, L), wl.Operand(16, 16, D)))
    (d1, l, d2), _ = wl.generate(eq)
    x, _ = ov.evaluate([d1, l, d2], eq.descs())
    p = op.plan(eq.descs())
    assert p.result_desc.prop == L and ov.off_structure_exactly_zero(x, L)
    x, _ = ov.evaluate([d1, d2], [eq.descs()[0], eq.descs()[2]])
    assert ov.off_structure_exactly_zero(x, D) and np.array_equal(np.diag(x), np.diag(d1).astype(np.float64) * np.diag(d2))


def test_a_diagonal_of_ones_computes_what_identity_states():
    # same value as the chain with Identity in its place; only the plan differs (Identity vanishes, Diagonal is data)
    eq = wl.Equation("A1B", 44, (wl.Operand(12, 9, G), wl.Operand(9, 9, D, "ones"), wl.Operand(9, 5, G)))
    (a, d, b), _ = wl.generate(eq)
    x, _ = ov.evaluate([a, d, b], eq.descs())
    xi, _ = ov.evaluate([a, None, b], [(12, 9, G), (9, 9, I), (9, 5, G)])
    assert np.array_equal(x, xi)
    assert op.plan(eq.descs()).mults == 45 + 12 * 9 * 5 and op.plan([(12, 9, G), (9, 9, I), (9, 5, G)]).mults == 12 * 9 * 5


@pytest.mark.parametrize("seed", range(12))
def test_plan_steps_reproduce_left_to_right_values_with_diagonals(seed):
    eq = wl.random_equation(1000 + seed, max_len=5, max_dim=24, diagonal=True)
    chain, add = wl.generate(eq)
    p = op.plan(eq.descs(), eq.add_descs())
    x, d = ov.evaluate(chain, eq.descs(), add, eq.add_descs())
    y = ov.evaluate_steps(chain, eq.descs(), p.steps, add, eq.add_descs())
    assert ov.normwise_error(y, x, d) <= 1e-12
    assert ov.off_structure_exactly_zero(x, p.result_desc.prop)
