"""Pins for the value oracle: closed forms, identities, a library routine, brute force on tiny inputs."""
import numpy as np
import pytest

from oracle import plan as op
from oracle import values as ov
from oracle.plan import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I
import workloads as wl


def test_matmul_against_the_library_routine_on_rectangular_inputs():
    # non-square, non-symmetric: a transposed operand or swapped dimension cannot pass
    rng = np.random.default_rng(0)
    for (m, k, n) in [(1, 1, 1), (7, 3, 5), (33, 65, 17), (128, 40, 257)]:
        a = rng.standard_normal((m, k))
        b = rng.standard_normal((k, n))
        ref = a @ b
        got = ov.matmul(a, b)
        assert got.shape == (m, n)
        assert np.max(np.abs(got - ref)) <= 1e-12 * np.max(np.abs(a) @ np.abs(b))


def test_matmul_against_python_loops_on_tiny_integers():
    a = np.array([[1, 2, 3], [4, 5, 6]], dtype=np.float64)
    b = np.array([[1, -1], [0, 2], [5, 7]], dtype=np.float64)
    want = [[sum(a[i, l] * b[l, j] for l in range(3)) for j in range(2)] for i in range(2)]
    assert want == [[16.0, 24.0], [34.0, 48.0]]          # hand-checked
    assert ov.matmul(a, b).tolist() == want


def test_matmul_does_not_depend_on_thread_count():
    rng = np.random.default_rng(1)
    a = rng.standard_normal((37, 51))
    b = rng.standard_normal((51, 29))
    ref = ov.matmul(a, b, threads=1)
    for t in (2, 3, 8, 64):
        assert np.array_equal(ov.matmul(a, b, threads=t), ref)


def test_ones_times_ones_is_inner_dimension():
    assert np.array_equal(ov.matmul(np.ones((4, 9)), np.ones((9, 6))), np.full((4, 6), 9.0))


def test_identity_laws_hold_bit_exactly():
    # paper Section 2 ("Types"): A*I = A and I*I = I
    eq = wl.Equation("t", 3, (wl.Operand(6, 9, G, "normal"),))
    (a,), _ = wl.generate(eq)
    x, _ = ov.evaluate([a, None], [(6, 9, G), (9, 9, I)])
    assert np.array_equal(x, a.astype(np.float64))
    x, _ = ov.evaluate([None, a], [(6, 6, I), (6, 9, G)])
    assert np.array_equal(x, a.astype(np.float64))
    x, _ = ov.evaluate([None, None], [(5, 5, I), (5, 5, I)])
    assert np.array_equal(x, np.eye(5))
    x, _ = ov.evaluate([None], [(5, 5, I)])
    assert np.array_equal(x, np.eye(5))


def test_listing2_closed_form():
    # two 5x5 lower-triangular matrices of ones: C[i][j] = #{l : j <= l <= i} = i - j + 1 for i >= j
    eq = wl.config_listing2()
    chain, _ = wl.generate(eq)
    assert np.array_equal(chain[0], np.tril(np.ones((5, 5), dtype=np.float32)))
    x, d = ov.evaluate(chain, eq.descs())
    want = np.array([[max(i - j + 1, 0) for j in range(5)] for i in range(5)], dtype=np.float64)
    assert np.array_equal(x, want)
    assert np.array_equal(d, want)
    assert x.sum() == 35                 # one unit per useful multiplication
    assert op.plan(eq.descs()).mults == 35


def test_triangular_products_stay_triangular():
    # paper Listing 3: lowerTri * lowerTri is typed lowerTri
    for prop in (L, U):
        eq = wl.Equation("t", 5, (wl.Operand(23, 23, prop), wl.Operand(23, 23, prop)))
        chain, _ = wl.generate(eq)
        x, _ = ov.evaluate(chain, eq.descs())
        assert ov.off_structure_exactly_zero(x, prop)
        assert not ov.off_structure_exactly_zero(x, U if prop == L else L)
        # diagonal of a triangular product is the product of the diagonals
        assert np.allclose(np.diag(x), np.diag(chain[0]).astype(np.float64) * np.diag(chain[1]).astype(np.float64),
                           rtol=1e-15, atol=0)


def test_mixed_triangular_product_corner_entries():
    # (L*U)[0][j] = L[0][0]*U[0][j] and (U*L)[n-1][j] = U[n-1][n-1]*L[n-1][j]
    eq = wl.Equation("t", 6, (wl.Operand(9, 9, L), wl.Operand(9, 9, U)))
    (l, u), _ = wl.generate(eq)
    x, _ = ov.evaluate([l, u], eq.descs())
    assert np.allclose(x[0, :], np.float64(l[0, 0]) * u[0, :].astype(np.float64), rtol=1e-15)
    x, _ = ov.evaluate([u, l], [(9, 9, U), (9, 9, L)])
    assert np.allclose(x[8, :], np.float64(u[8, 8]) * l[8, :].astype(np.float64), rtol=1e-15)


def test_associativity_any_parenthesization_gives_the_same_value():
    for seed in range(12):
        eq = wl.random_equation(seed, max_len=5, max_dim=24)
        chain, add = wl.generate(eq)
        x, d = ov.evaluate(chain, eq.descs(), add, eq.add_descs())
        p = op.plan(eq.descs(), eq.add_descs())
        y = ov.evaluate_steps(chain, eq.descs(), p.steps, add, eq.add_descs())
        assert y.shape == x.shape
        assert ov.normwise_error(y, x, d) <= 1e-12
        assert ov.off_structure_exactly_zero(x, p.result_desc.prop)


def test_add_terms_are_added_once_each_with_plus_sign():
    a = np.arange(6, dtype=np.float32).reshape(2, 3)
    b = np.ones((3, 2), dtype=np.float32)
    t1 = np.array([[10, 20], [30, 40]], dtype=np.float32)
    t2 = np.array([[-1, -2], [-3, -4]], dtype=np.float32)
    x, d = ov.evaluate([a, b], [(2, 3, G), (3, 2, G)], [t1, t2, None], [(2, 2, G), (2, 2, G), (2, 2, I)])
    assert x.tolist() == [[3 + 10 - 1 + 1, 3 + 20 - 2], [12 + 30 - 3, 12 + 40 - 4 + 1]]
    assert d.tolist() == [[3 + 10 + 1 + 1, 3 + 20 + 2], [12 + 30 + 3, 12 + 40 + 4 + 1]]


def test_denominator_bounds_the_value():
    eq = wl.random_equation(42, max_len=4, max_dim=20)
    chain, add = wl.generate(eq)
    x, d = ov.evaluate(chain, eq.descs(), add, eq.add_descs())
    assert np.all(d >= np.abs(x) - 1e-12 * d)
    # with non-negative inputs the two coincide
    pos = [None if c is None else np.abs(c) for c in chain]
    x2, d2 = ov.evaluate(pos, eq.descs())
    assert np.array_equal(x2, d2)


def test_row_subset_equals_rows_of_the_full_result():
    eq = wl.Equation("t", 9, (wl.Operand(40, 40, L), wl.Operand(40, 13, G, "normal"), wl.Operand(13, 21)),
                     (wl.Operand(40, 21),))
    chain, add = wl.generate(eq)
    x, d = ov.evaluate(chain, eq.descs(), add, eq.add_descs())
    rows = np.array([0, 7, 39, 20])
    xs, ds = ov.evaluate(chain, eq.descs(), add, eq.add_descs(), rows=rows)
    assert np.array_equal(xs, x[rows]) and np.array_equal(ds, d[rows])


def test_normwise_error_and_structure_helpers():
    ref = np.array([[3.0, 4.0]])
    assert ov.normwise_error(ref + np.array([[0.0, 0.5]]), ref, np.array([[6.0, 8.0]])) == pytest.approx(0.05)
    assert ov.normwise_error(np.zeros((1, 2)), np.zeros((1, 2)), np.zeros((1, 2))) == 0.0
    m = ov.off_structure_mask(3, 3, L)
    assert m.tolist() == [[False, True, True], [False, False, True], [False, False, False]]
    assert ov.off_structure_mask(3, 3, U, row_index=np.array([2])).tolist() == [[True, True, False]]
    x = np.tril(np.ones((3, 3)))
    assert ov.off_structure_exactly_zero(x, L) and not ov.off_structure_exactly_zero(x, U)


def test_generated_inputs_follow_the_storage_contract():
    eq = wl.config_tiny()
    (l, a, b), _ = wl.generate(eq)
    assert l.dtype == np.float32 and l.shape == (64, 64)
    assert np.all(np.triu(l, 1) == 0) and not np.signbit(np.triu(l, 1)).any()
    assert np.all((np.diag(l) >= 1) & (np.diag(l) < 2))
    assert np.all(np.abs(np.tril(l, -1)) <= 1) and np.all(np.abs(a) <= 1)
    # same key, same matrix; different operand index, different matrix
    (l2, a2, _), _ = wl.generate(eq)
    assert np.array_equal(l, l2) and np.array_equal(a, a2)
    assert not np.array_equal(a[:, :32], b[:32, :32].T)
    eqb = wl.config_batched(batch=3)
    chain, add = wl.generate(eqb)
    assert chain[0].shape == (3, 64, 64) and add[0].shape == (3, 64, 16)
    assert np.all(np.triu(chain[0], 1) == 0)
    big = wl.config_large_square(n=64)
    (_, a64, _, _), _ = wl.generate(big)
    assert abs(float(a64.std()) - 64 ** -0.5) < 0.02


def test_transposed_operands_follow_the_transpose_identities():
    # (A*B)^T = B^T * A^T, checked through the oracle's own transposed-operand path against NumPy
    rng = np.random.default_rng(5)
    a = rng.standard_normal((6, 9)).astype(np.float32)
    b = rng.standard_normal((9, 4)).astype(np.float32)
    arrs, descs = ov.transposed_operands([b, a], [(9, 4, G), (6, 9, G)], [True, True])
    assert descs == [(4, 9, G), (9, 6, G)]
    x, _ = ov.evaluate(arrs, descs)
    assert np.allclose(x, (a.astype(np.float64) @ b.astype(np.float64)).T, rtol=1e-14)
    # the transpose of a stored lower-triangular matrix is upper triangular, entry for entry
    eq = wl.Equation("t", 12, (wl.Operand(7, 7, L),))
    (l,), _ = wl.generate(eq)
    (lt,), (d,) = ov.transposed_operands([l], eq.descs(), [True])
    assert d == (7, 7, U) and np.array_equal(lt, l.T) and ov.off_structure_exactly_zero(lt, U)
    # untouched operands are passed through
    arrs, descs = ov.transposed_operands([a, None], [(6, 9, G), (9, 9, I)], [False, True])
    assert arrs[0] is a and arrs[1] is None and descs[1] == (9, 9, I)
