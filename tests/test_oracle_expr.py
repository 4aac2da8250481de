"""Pins for the nested-expression oracle (`plan_expr`, `evaluate_expr`, `normalize_expr`): library routines on
the un-normalized expression, hand arithmetic, numeric structure, and the chain / sum oracles pinned elsewhere."""
import numpy as np
import pytest

from oracle import plan as op
from oracle import values as ov
from oracle.plan import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I


def rnd(rng, rows, cols, prop=G):
    a = rng.uniform(0.5, 1.5, size=(rows, cols))
    return np.tril(a) if prop == L else np.triu(a) if prop == U else a


def numpy_value(e, arrays):
    """The expression evaluated by NumPy on the expression AS WRITTEN (no normalization)."""
    if isinstance(e, int):
        return arrays[e]
    if e[0] == "t":
        return numpy_value(e[1], arrays).T
    vals = [numpy_value(c, arrays) for c in e[1]]
    out = vals[0]
    for v in vals[1:]:
        out = out @ v if e[0] == "mul" else out + v
    return out


EXPRS = [
    ("mul", [0, ("add", [1, 2]), 3]),
    ("t", ("mul", [0, ("add", [1, 2, ("mul", [1, 3])]), 3])),
    ("add", [("mul", [0, ("add", [1, 2])]), ("mul", [("t", 0), ("add", [2, 1])]), 1]),
    ("mul", [("add", [0, ("t", 0)]), ("add", [1, ("mul", [0, 2])])]),
    ("mul", [("t", ("add", [1, 2])), ("add", [1, 2])]),
    ("t", ("t", ("mul", [0, 1]))),
]
OPS = [(8, 8, L), (8, 6, G), (8, 6, G), (6, 6, U)]


@pytest.mark.parametrize("expr", EXPRS, ids=[str(i) for i in range(len(EXPRS))])
def test_value_against_numpy_on_the_expression_as_written(expr):
    rng = np.random.default_rng(1)
    arrays = [rnd(rng, *d) for d in OPS]
    x, d = ov.evaluate_expr(expr, arrays, OPS)
    np.testing.assert_allclose(x, numpy_value(expr, arrays), rtol=1e-13)
    np.testing.assert_allclose(d, numpy_value(expr, arrays), rtol=1e-13)       # all entries positive: D = X


@pytest.mark.parametrize("expr", EXPRS, ids=[str(i) for i in range(len(EXPRS))])
def test_normal_form_has_the_same_value_and_the_inferred_structure(expr):
    # evaluate the NORMAL FORM with NumPy: transposes at the leaves, nested sums as sub-values
    rng = np.random.default_rng(2)
    arrays = [rnd(rng, *d) for d in OPS]

    def value(sum_nf):
        total = None
        for chain in sum_nf:
            v = None
            for f in chain:
                m = (arrays[f[1]].T if f[2] else arrays[f[1]]) if f[0] == "leaf" else value(f[1])
                v = m if v is None else v @ m
            total = v if total is None else total + v
        return total

    x = value(op.normalize_expr(expr))
    np.testing.assert_allclose(x, numpy_value(expr, arrays), rtol=1e-13)
    p = op.plan_expr(expr, OPS)
    assert (p.result_desc.rows, p.result_desc.cols) == x.shape
    assert not (x != 0)[ov.off_structure_mask(x.shape[0], x.shape[1], p.result_desc.prop)].any()


def test_costs_by_hand():
    n = 10
    ops = [(n, n, G)] * 3
    # A*(B+C): one product, one addition -- not two products
    p = op.plan_expr(("mul", [0, ("add", [1, 2])]), ops)
    assert (p.mults, p.add_flops, p.temporaries, p.paren) == (n ** 3, n * n, 1, "(0*[1+2])")
    # the distributed form costs two products and shares nothing below a root
    q = op.plan_expr(("add", [("mul", [0, 1]), ("mul", [0, 2])]), ops)
    assert (q.mults, q.add_flops, q.temporaries, q.paren) == (2 * n ** 3, n * n, 0, "(0*1)+(0*2)")
    # the same nested sum twice is one temporary
    r = op.plan_expr(("add", [("mul", [0, ("add", [1, 2])]), ("mul", [1, ("add", [1, 2])])]), ops)
    assert r.temporaries == 1 and r.add_flops == 2 * n * n and r.mults == 2 * n ** 3
    # lowerTri*(lowerTri + lowerTri) stays a triangular product
    t = op.plan_expr(("mul", [0, ("add", [1, 2])]), [(n, n, L)] * 3)
    assert t.mults == n * (n + 1) * (n + 2) // 6 and t.result_desc.prop == L
    assert t.products == ((n, n, n, L, L, L, t.mults),)


def test_expression_without_nesting_equals_the_chain_and_sum_oracles():
    chain = [(9, 9, L), (9, 4, G), (4, 4, U), (4, 6, G)]
    p, e = op.plan(chain), op.plan_expr(("mul", [0, 1, 2, 3]), chain)
    assert (e.paren, e.mults, e.add_flops, e.result_desc) == (p.paren, p.mults, 0, p.result_desc)
    # nested products flatten: ((0*1)*(2*3)) written by the user is still planned as one chain
    e2 = op.plan_expr(("mul", [("mul", [0, 1]), ("mul", [2, 3])]), chain)
    assert e2 == e
    ops = [(8, 50, G), (50, 8, G), (8, 100, G), (8, 100, G)]
    s = op.plan_sum([[ops[0], ops[1], ops[2]], [ops[0], ops[1], ops[3]]], names=[[0, 1, 2], [0, 1, 3]])
    e = op.plan_expr(("add", [("mul", [0, 1, 2]), ("mul", [0, 1, 3])]), ops)
    assert (e.mults, e.reused, e.add_flops) == (s.mults, 1, s.add_flops)
    assert e.paren == "((0*1)*2)+((0*1)*3)"


def test_transpose_of_a_product_reverses_it():
    ops = [(5, 7, G), (7, 3, G)]
    e = op.plan_expr(("t", ("mul", [0, 1])), ops)
    assert e.paren == "(1^T*0^T)" and (e.result_desc.rows, e.result_desc.cols) == (3, 5)
    e = op.plan_expr(("t", ("mul", [0, 1])), [(5, 5, L), (5, 5, L)])
    assert e.result_desc.prop == U


def test_expression_errors():
    with pytest.raises(op.OracleError) as e:
        op.plan_expr(("mul", [0, ("add", [1, 2])]), [(4, 5, G), (5, 6, G), (6, 5, G)])
    assert e.value.code == "shape_mismatch"
    with pytest.raises(op.OracleError) as e:
        op.plan_expr(("mul", [0, 7]), [(4, 5, G)])
    assert e.value.code == "invalid_arg"
    with pytest.raises(op.OracleError) as e:
        op.plan_expr(("add", []), [(4, 5, G)])
    assert e.value.code == "invalid_arg"
