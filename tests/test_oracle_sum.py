"""Pins for the sum-of-chains oracle (`plan_sum`, `evaluate_sum`): each check compares it with something
that is not itself -- distributivity through a library routine, hand arithmetic, brute-force structure
counts on numeric values, and the single-chain functions pinned elsewhere."""
import numpy as np
import pytest

from oracle import plan as op
from oracle import values as ov
from oracle.plan import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I, DIAGONAL as D


def rnd(rng, rows, cols, prop=G):
    a = rng.uniform(0.5, 1.5, size=(rows, cols))        # strictly positive: no cancellation in any sum
    if prop == L:
        a = np.tril(a)
    if prop == U:
        a = np.triu(a)
    if prop == D:
        a = np.diag(np.diag(a))
    return a


def test_sum_of_two_products_is_distributivity_through_the_library_routine():
    # A*C + B*C = (A + B) @ C : a dropped chain, a doubled chain or a wrong sign cannot pass
    rng = np.random.default_rng(1)
    a, b, c = rnd(rng, 7, 5), rnd(rng, 7, 5), rnd(rng, 5, 9)
    x, d = ov.evaluate_sum([[a, c], [b, c]], [[(7, 5, G), (5, 9, G)]] * 2)
    np.testing.assert_allclose(x, (a + b) @ c, rtol=1e-13)
    np.testing.assert_allclose(d, (np.abs(a) + np.abs(b)) @ np.abs(c), rtol=1e-13)


def test_sum_with_single_factor_chains_equals_the_single_chain_oracle_with_add_terms():
    rng = np.random.default_rng(2)
    a, b, t1 = rnd(rng, 6, 4), rnd(rng, 4, 6), rnd(rng, 6, 6, L)
    x1, d1 = ov.evaluate([a, b], [(6, 4, G), (4, 6, G)], [t1, None], [(6, 6, L), (6, 6, I)])
    x2, d2 = ov.evaluate_sum([[a, b], [t1], [None]], [[(6, 4, G), (4, 6, G)], [(6, 6, L)], [(6, 6, I)]])
    assert np.array_equal(x1, x2) and np.array_equal(d1, d2)


def test_row_subset_of_a_sum():
    rng = np.random.default_rng(3)
    a, b, c, e = rnd(rng, 9, 4), rnd(rng, 4, 5), rnd(rng, 9, 9, U), rnd(rng, 9, 5)
    chains, descs = [[a, b], [c, e]], [[(9, 4, G), (4, 5, G)], [(9, 9, U), (9, 5, G)]]
    x, d = ov.evaluate_sum(chains, descs)
    rows = np.array([0, 4, 8])
    xs, ds = ov.evaluate_sum(chains, descs, rows=rows)
    assert np.array_equal(xs, x[rows]) and np.array_equal(ds, d[rows])


def test_cost_of_a_sum_by_hand():
    # two general n x n x n products: 2 n^3 multiplications; add_flops = n^2 (one matrix addition)
    n = 11
    sp = op.plan_sum([[(n, n, G), (n, n, G)], [(n, n, G), (n, n, G)]])
    assert sp.mults == 2 * n ** 3 and sp.mul_flops == 4 * n ** 3 and sp.add_flops == n * n
    assert sp.paren == "(0*1)+(2*3)" and sp.reused == 0
    # the paper's Section-4 chain twice costs twice its printed optimum, each chain parenthesized on its own
    chain = [(800, 1100, G), (1100, 900, G), (900, 1200, G), (1200, 100, G)]
    sp = op.plan_sum([chain, chain])
    assert sp.mults == 2 * 295_000_000
    assert sp.paren == "(0*(1*(2*3)))+(4*(5*(6*7)))"


def test_single_chain_sum_equals_the_chain_plan():
    chain = [(9, 9, L), (9, 4, G), (4, 4, U), (4, 6, G)]
    p, sp = op.plan(chain), op.plan_sum([chain])
    assert (sp.paren, sp.mults, sp.add_flops, sp.result_desc) == (p.paren, p.mults, 0, p.result_desc)
    assert sp.steps == p.steps


def test_chains_of_one_factor_behave_like_add_terms():
    chain = [(9, 9, L), (9, 9, L)]
    for terms in ([(9, 9, L)], [(9, 9, U)], [(9, 9, I)], [(9, 9, I), (9, 9, G)]):
        p = op.plan(chain, terms)
        sp = op.plan_sum([chain] + [[t] for t in terms])
        assert sp.result_desc == p.result_desc and sp.add_flops == p.add_flops and sp.mults == p.mults


@pytest.mark.parametrize("props", [((L, L), (L, L)), ((L, L), (U, U)), ((L, G), (L, L)), ((U, U), (U, I)),
                                   ((I, I), (I, I)), ((L, I), (I, I)), ((I, I), (U, U)),
                                   ((D, D), (I, I)), ((D, L), (D, I)), ((D, U), (L, D)), ((G, D), (D, D))])
def test_result_property_is_the_tightest_that_holds_the_numeric_pattern(props):
    # With positive entries nothing cancels, so the non-zero pattern of the numeric value is the true
    # structure; the inferred property must contain it and no tighter property may.
    n = 6
    rng = np.random.default_rng(5)
    chains = [[(n, n, p) for p in chain] for chain in props]
    mats = [[None if p == I else rnd(rng, n, n, p) for p in chain] for chain in props]
    x, _ = ov.evaluate_sum(mats, chains)
    sp = op.plan_sum(chains)
    pattern = x != 0
    holds = {p: not pattern[ov.off_structure_mask(n, n, p)].any() for p in (G, L, U, D)}
    got = sp.result_desc.prop
    assert got != I and holds[got]              # a sum of at least two summands is never typed Identity (I + I = 2 I)
    if got == G:
        assert not holds[L] and not holds[U]
    elif got in (L, U):
        assert not holds[D]
    else:
        assert got == D


def test_reuse_of_a_shared_product_counts_it_once():
    # A(8x50) B(50x8) C(8x100): (A*B)*C is the cheaper tree (3200 + 6400 against 80000), so A*B sits below
    # the root in both chains and is multiplied once: 3200 + 6400 + 6400.
    a, b, c1, c2 = (8, 50, G), (50, 8, G), (8, 100, G), (8, 100, G)
    sp = op.plan_sum([[a, b, c1], [a, b, c2]], names=[[0, 1, 2], [0, 1, 3]])
    assert sp.reused == 1 and sp.mults == 3200 + 6400 + 6400
    assert sp.paren == "((0*1)*2)+((3*4)*5)"
    assert [(s.lhs, s.rhs, s.out) for s in sp.steps] == [(0, 1, 6), (6, 2, 7), (6, 5, 8)]
    # without names nothing is known to be the same matrix
    assert op.plan_sum([[a, b, c1], [a, b, c2]]).mults == 2 * (3200 + 6400)
    # a transposed use is another product
    sp = op.plan_sum([[a, b, c1], [(50, 8, G), b, c2]], transposed=[[False] * 3, [True, False, False]],
                     names=[[0, 1, 2], [4, 1, 3]])
    assert sp.reused == 0
    # a chain's root is never shared, even when another chain repeats it
    sp = op.plan_sum([[a, b], [a, b]], names=[[0, 1], [0, 1]])
    assert sp.reused == 0 and sp.mults == 2 * 3200


def test_reuse_keeps_the_value():
    rng = np.random.default_rng(7)
    a, b, c1, c2 = rnd(rng, 8, 50), rnd(rng, 50, 8), rnd(rng, 8, 100), rnd(rng, 8, 100)
    descs = [[(8, 50, G), (50, 8, G), (8, 100, G)]] * 2
    x, _ = ov.evaluate_sum([[a, b, c1], [a, b, c2]], descs)
    np.testing.assert_allclose(x, (a @ b) @ (c1 + c2), rtol=1e-13)


def test_sum_errors():
    with pytest.raises(op.OracleError) as e:
        op.plan_sum([])
    assert e.value.code == "invalid_arg"
    with pytest.raises(op.OracleError) as e:
        op.plan_sum([[(4, 5, G)], [(5, 4, G)]])
    assert e.value.code == "shape_mismatch"
    with pytest.raises(op.OracleError) as e:
        op.plan_sum([[(4, 5, G), (4, 5, G)]])
    assert e.value.code == "shape_mismatch"
    with pytest.raises(op.OracleError) as e:
        op.plan_sum([[(4, 4, G)], [(4, 4, L)]], names=[[0], [0]])
    assert e.value.code == "invalid_arg"
