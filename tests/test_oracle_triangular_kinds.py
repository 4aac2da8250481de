"""Pins of the oracle for the strictly triangular and unit triangular properties (two of the "more
properties" the paper's conclusion announces; it prints no rule for them).  Every pin comes from the
mathematics: counting on tiny shapes, hand arithmetic, and the numeric values of products and sums of
matrices drawn with each type (positive entries, so nothing cancels)."""
import itertools

import numpy as np
import pytest

from oracle import plan as op
from oracle import values as ov
from oracle.plan import (GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I, DIAGONAL as D, SYMMETRIC as S,
                         STRICT_LOWER as SL, STRICT_UPPER as SU, UNIT_LOWER as UL, UNIT_UPPER as UU, Desc)

ALL = (G, L, U, I, D, S, SL, SU, UL, UU)
NAMES = {G: "G", L: "L", U: "U", I: "I", D: "D", S: "S", SL: "sL", SU: "sU", UL: "uL", UU: "uU"}


def draw(rng, n, prop):
    """A matrix of the given type with entries in (0.5, 1.5) wherever the type leaves them free."""
    a = rng.uniform(0.5, 1.5, size=(n, n))
    if prop in (L, UL):
        a = np.tril(a)
    elif prop in (U, UU):
        a = np.triu(a)
    elif prop == SL:
        a = np.tril(a, -1)
    elif prop == SU:
        a = np.triu(a, 1)
    elif prop == D:
        a = np.diag(np.diag(a))
    elif prop == I:
        a = np.eye(n)
    elif prop == S:
        a = a + a.T
    if prop in (UL, UU):
        np.fill_diagonal(a, 1.0)
    return a


def fits(x, prop):
    """Does the numeric matrix x satisfy everything the type states?"""
    n = x.shape[0]
    if x[ov.off_structure_mask(n, n, prop)].any():
        return False
    if prop in (I, UL, UU) and not np.all(np.diag(x) == 1.0):
        return False
    if prop == S and not np.array_equal(x, x.T):
        return False
    return True


def implies(rng, p, q):
    """Every matrix of type p is a matrix of type q (decided on one matrix of type p with generic entries)."""
    return fits(draw(rng, 5, p), q)


def test_structure_counts_equal_brute_force():
    for prop in ALL:
        for n in range(1, 7):
            d = Desc(n, n, prop)
            assert op.structural_nonzeros(d) == op.brute_force_nonzeros(d), (NAMES[prop], n)
            free = sum(1 for i in range(n) for j in range(n) if op.multiplies(prop, i, j))
            assert op.multiplying_entries(d) == free, (NAMES[prop], n)


def test_structure_predicates_by_hand():
    assert [op.in_structure(SL, i, j) for i, j in ((0, 0), (1, 0), (0, 1))] == [False, True, False]
    assert [op.in_structure(SU, i, j) for i, j in ((0, 0), (1, 0), (0, 1))] == [False, False, True]
    assert [op.in_structure(UL, i, j) for i, j in ((0, 0), (1, 0), (0, 1))] == [True, True, False]
    assert [op.known_one(UU, i, j) for i, j in ((0, 0), (0, 1), (2, 2))] == [True, False, True]
    assert not op.known_one(L, 1, 1) and not op.known_one(SL, 1, 1) and op.known_one(I, 3, 3)


def test_product_costs_equal_brute_force_for_every_pair_of_types():
    for pa, pb in itertools.product(ALL, repeat=2):
        for n in range(1, 7):
            a, b = Desc(n, n, pa), Desc(n, n, pb)
            assert op.product_mults(a, b) == op.brute_force_mults(a, b), (NAMES[pa], NAMES[pb], n)
    for p in (SL, SU, UL, UU):                     # rectangular general partner
        for n, c in itertools.product(range(1, 6), range(1, 5)):
            assert op.product_mults(Desc(n, n, p), Desc(n, c, G)) == op.brute_force_mults(Desc(n, n, p), Desc(n, c, G))
            assert op.product_mults(Desc(c, n, G), Desc(n, n, p)) == op.brute_force_mults(Desc(c, n, G), Desc(n, n, p))


def test_hand_costs():
    d = lambda n, p, c=None: Desc(n, n if c is None else c, p)
    # rows of a strictly lower 4 x 4 matrix hold 0, 1, 2, 3 entries: 6 per column of the general factor
    assert op.product_mults(d(4, SL), d(4, G, 3)) == 18
    assert op.product_mults(d(4, UL), d(4, G, 3)) == 18            # the ones on the diagonal multiply nothing
    assert op.product_mults(d(4, L), d(4, G, 3)) == 30
    # unit lower * unit lower, n = 4: triples i > l > j, C(4, 3)
    assert op.product_mults(d(4, UL), d(4, UL)) == 4
    # strictly lower * lower, n = 4: triples i > l >= j, C(5, 3)
    assert op.product_mults(d(4, SL), d(4, L)) == 10
    # strictly lower * strictly upper, n = 3: column l of A and row l of B hold 2, 1, 0 entries: 4 + 1 + 0
    assert op.product_mults(d(3, SL), d(3, SU)) == 5
    # unit lower * upper, n = 3: (3 - 1) 3 + (2 - 1) 2 + (1 - 1) 1
    assert op.product_mults(d(3, UL), d(3, U)) == 8
    # a Diagonal factor scales the entries that are not known ones
    assert op.product_mults(d(4, D), d(4, UU)) == 6 and op.product_mults(d(4, SL), d(4, D)) == 6
    assert op.product_mults(d(4, D), d(4, U)) == 10
    # Add terms: a unit triangle adds its ones too, a strict one has no diagonal to add
    assert op.plan([(4, 4, G)], [(4, 4, UL), (4, 4, SU)]).add_flops == 10 + 6


def test_gram_costs_equal_brute_force():
    for p in (SL, SU, UL, UU):
        for n in range(1, 7):
            assert op.gram_mults(Desc(n, n, p)) == op.brute_force_gram_mults(Desc(n, n, p)), (NAMES[p], n)
    assert op.gram_mults(Desc(4, 4, SL)) == 10        # i >= j > l: C(5, 3)


def test_product_type_is_the_least_type_of_the_numeric_product():
    rng = np.random.default_rng(3)
    n = 5
    for pa, pb in itertools.product(ALL, repeat=2):
        x = draw(rng, n, pa) @ draw(rng, n, pb)
        got = op.join(pa, pb)
        assert fits(x, got), (NAMES[pa], NAMES[pb], NAMES[got])
        for other in ALL:
            if other != got and fits(x, other) and implies(rng, other, got):
                # a strictly tighter type also fits this value: allowed only where the lattice has no name for
                # the general rule (S*S is symmetric only when the factors commute: here never, entries are generic)
                assert implies(rng, got, other), (NAMES[pa], NAMES[pb], NAMES[got], NAMES[other])


def test_sum_type_is_the_least_type_of_the_numeric_sum():
    rng = np.random.default_rng(4)
    n = 5
    for props in itertools.chain(itertools.product(ALL, repeat=2), itertools.product((L, I, D, SL, SU, UL, UU), repeat=3)):
        x = sum(draw(rng, n, p) for p in props)
        got = op.sum_property(props[0], props[1:])
        assert got != I and fits(x, got), ([NAMES[p] for p in props], NAMES[got])
        for other in ALL:
            if other != got and other != I and fits(x, other) and implies(rng, other, got):
                assert implies(rng, got, other), ([NAMES[p] for p in props], NAMES[got], NAMES[other])


def test_rules_by_hand():
    assert op.join(SL, L) == SL and op.join(L, SL) == SL and op.join(SL, UL) == SL
    assert op.join(UL, UL) == UL and op.join(UL, L) == L and op.join(UU, UU) == UU
    assert op.join(UL, UU) == G and op.join(SL, SU) == G and op.join(SL, U) == G
    assert op.join(D, UL) == L and op.join(D, SL) == SL and op.join(SU, D) == SU
    assert op.join(I, UL) == UL and op.join(SU, I) == SU and op.join(S, SL) == G
    assert op.sum_property(I, [SL]) == UL and op.sum_property(SU, [I]) == UU
    assert op.sum_property(UL, [UL]) == L and op.sum_property(UL, [SL]) == UL and op.sum_property(SL, [SL]) == SL
    assert op.sum_property(SL, [D]) == L and op.sum_property(SL, [SU]) == G and op.sum_property(S, [SL]) == G
    assert op.sum_property(I, [SL, I]) == L and op.sum_property(SL, [SL, I]) == UL
    assert op.transpose_desc(Desc(4, 4, SL)).prop == SU and op.transpose_desc(Desc(4, 4, UU)).prop == UL


def test_a_nilpotent_chain_is_cheapest_through_its_strict_factors():
    # N strictly lower, A general 6 x 40: (N*N)*A costs C(6,3) + 15*40 = 620, N*(N*A) costs 2*15*40 = 1200
    p = op.plan([(6, 6, SL), (6, 6, SL), (6, 40, G)])
    assert p.paren == "((0*1)*2)" and p.mults == 20 + 15 * 40
    assert p.steps[0].out_prop == SL
    # with plain lower triangles the same tree costs C(8,3) + 21*40 = 896
    assert op.plan([(6, 6, L), (6, 6, L), (6, 40, G)]).mults == 56 + 21 * 40


@pytest.mark.parametrize("seed", range(6))
def test_chosen_tree_is_a_minimum_under_brute_force_costs(seed):
    rng = np.random.default_rng(100 + seed)
    for _ in range(12):
        n = int(rng.integers(2, 6))
        cur = int(rng.integers(1, 6))
        chain = []
        for _ in range(n):
            kind = int(rng.integers(0, 10))
            if kind < 7:
                chain.append((cur, cur, (L, U, D, SL, SU, UL, UU)[kind]))
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


def test_values_keep_the_stated_diagonal():
    rng = np.random.default_rng(9)
    n = 7
    a, b, c = draw(rng, n, UL), draw(rng, n, UL), draw(rng, n, SL)
    x, _ = ov.evaluate([a, b], [(n, n, UL), (n, n, UL)])
    assert ov.off_structure_exactly_zero(x, UL) and ov.unit_diagonal_exactly_one(x, UL)
    y, _ = ov.evaluate([a, c], [(n, n, UL), (n, n, SL)])
    assert ov.off_structure_exactly_zero(y, SL)
    assert not ov.unit_diagonal_exactly_one(2 * x, UL) and ov.unit_diagonal_exactly_one(2 * x, L)
    assert ov.unit_diagonal_exactly_one(x[[0, 3, 6]], UL, row_index=np.array([0, 3, 6]))


@pytest.mark.parametrize("seed", range(16))
def test_plan_steps_reproduce_left_to_right_values(seed):
    import workloads as wl
    eq = wl.random_equation(2000 + seed, max_len=5, max_dim=24, kinds=True)
    chain, add = wl.generate(eq)
    p = op.plan(eq.descs(), eq.add_descs())
    x, d = ov.evaluate(chain, eq.descs(), add, eq.add_descs())
    y = ov.evaluate_steps(chain, eq.descs(), p.steps, add, eq.add_descs())
    assert ov.normwise_error(y, x, d) <= 1e-12
    assert ov.off_structure_exactly_zero(x, p.result_desc.prop)
    assert ov.unit_diagonal_exactly_one(x, p.result_desc.prop)
    for o, a in zip(eq.chain + eq.add, list(chain) + list(add)):       # the generator keeps the storage contract
        if a is not None:
            assert ov.off_structure_exactly_zero(a, o.prop) and ov.unit_diagonal_exactly_one(a, o.prop)
