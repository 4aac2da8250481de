"""GPU parity for nested expressions: the CUDA path through the C ABI against the fp64 oracle."""
import numpy as np
import pytest

import paper_2208_10391_b200 as mom
import workloads as wl
from workloads import Operand, Expression, GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I
from gpu_util import run_expression, check_expression_against_oracle

pytestmark = pytest.mark.gpu

VARIANTS = [mom.VARIANT_3XTF32, mom.VARIANT_FFMA, mom.VARIANT_3XTF32_FORCE, mom.VARIANT_3XTF32_WARP, mom.VARIANT_3XTF32_INLINE]


def expression(name, operands, expr, seed=21):
    return Expression(name, seed, tuple(Operand(*o) for o in operands), expr)


@pytest.mark.parametrize("variant", VARIANTS)
def test_random_expressions(variant):
    mult = 4 if variant == mom.VARIANT_3XTF32_FORCE else 1
    for seed in range(60):
        ex = wl.random_expression(seed, max_dim=72, dim_multiple=mult)
        x, plan, arrays = run_expression(ex, variant)
        check_expression_against_oracle(ex, x, plan, arrays)


@pytest.mark.parametrize("variant", VARIANTS)
def test_sum_inside_a_product_on_several_tiles(variant):
    # A*(B + C^T + I)*U with ragged sizes: the temporary is written by one elementwise pass and read as a factor
    n, m = 332, 260
    ex = expression("nested", [(m, n, G), (n, n, G), (n, n, G), (n, n, I), (n, n, U)],
                    ("mul", [0, ("add", [1, ("t", 2), 3]), 4]))
    x, plan, arrays = run_expression(ex, variant)
    assert plan.temporaries() == 1
    check_expression_against_oracle(ex, x, plan, arrays)


@pytest.mark.parametrize("variant", VARIANTS)
def test_nested_sum_that_contains_products(variant):
    # (A*B + C) * (D + E*F + G): both temporaries are written by product roots with fused and accumulated summands
    n = 264
    ex = expression("products_inside", [(n, n, G)] * 7,
                    ("mul", [("add", [("mul", [0, 1]), 2]), ("add", [3, ("mul", [4, 5]), 6])]))
    x, plan, arrays = run_expression(ex, variant)
    assert plan.temporaries() == 2 and plan.num_steps() == 3
    check_expression_against_oracle(ex, x, plan, arrays)


@pytest.mark.parametrize("variant", VARIANTS)
def test_triangular_temporaries_keep_their_structure(variant):
    # (L1 + L2) * (L1 + U^T): both sums are lowerTri, the product is a TT product with a lowerTri result
    n = 296
    ex = expression("tri", [(n, n, L), (n, n, L), (n, n, U)],
                    ("mul", [("add", [0, 1]), ("add", [0, ("t", 2)])]))
    x, plan, arrays = run_expression(ex, variant)
    assert plan.result_desc().property == L and plan.step(0).kind == mom.KIND_TT
    check_expression_against_oracle(ex, x, plan, arrays)


@pytest.mark.parametrize("variant", VARIANTS)
def test_same_nested_sum_used_twice_and_deep_nesting(variant):
    n = 200
    s = ("add", [1, 2])
    ex = expression("twice", [(n, n, G), (n, n, G), (n, n, L), (n, n, U)],
                    ("add", [("mul", [0, s]), ("mul", [s, 3]), ("t", ("mul", [3, ("add", [0, ("mul", [s, s])])]))]))
    x, plan, arrays = run_expression(ex, variant)
    check_expression_against_oracle(ex, x, plan, arrays)


@pytest.mark.parametrize("variant", VARIANTS)
def test_temporary_that_only_meets_identity(variant):
    # I*(A + B): the outer chain reduces to the temporary itself; X = temporary + C
    n = 136
    ex = expression("identity_outer", [(n, n, I), (n, n, G), (n, n, U), (n, n, L)],
                    ("add", [("mul", [0, ("add", [1, 2])]), 3]))
    x, plan, arrays = run_expression(ex, variant)
    assert plan.num_steps() == 0
    check_expression_against_oracle(ex, x, plan, arrays)


def test_expression_through_the_host_entry_point():
    ex = wl.random_expression(3, max_dim=64, dim_multiple=4)
    x, plan, arrays = run_expression(ex, mom.VARIANT_3XTF32, via="host")
    check_expression_against_oracle(ex, x, plan, arrays)


def test_expression_configuration_full_size_sampled_rows():
    ex = wl.config_expression(2048)          # the fp64 oracle evaluates nested sums in full: 2048 keeps it to seconds
    x, plan, arrays = run_expression(ex, mom.VARIANT_3XTF32)
    assert all(s.uses_tensor_cores == 1 for s in plan.steps())
    check_expression_against_oracle(ex, x, plan, arrays)
