"""GPU parity for equations with Diagonal operands: the scaling kernel, its place in chains, sums and
nested expressions, and the fused small-equation kernel, against the fp64 oracle through the C ABI."""
import itertools

import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2208_10391_b200 as mom
import workloads as wl
from workloads import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I, DIAGONAL as D, Operand, Equation
from gpu_util import (run_equation, check_against_oracle, run_sum_equation, check_sum_against_oracle, run_expression,
                      check_expression_against_oracle, stratified_rows)

pytestmark = pytest.mark.gpu

VARIANTS = [mom.VARIANT_FFMA, mom.VARIANT_3XTF32_FORCE, mom.VARIANT_3XTF32_WARP, mom.VARIANT_3XTF32_INLINE]
VNAME = {mom.VARIANT_FFMA: "ffma", mom.VARIANT_3XTF32_FORCE: "tc", mom.VARIANT_3XTF32: "auto", mom.VARIANT_3XTF32_WARP: "warp", mom.VARIANT_3XTF32_INLINE: "inline"}


def both(eq, variant, **kw):
    x, plan, (chain, add) = run_equation(eq, variant)
    return check_against_oracle(eq, x, plan, chain, add, **kw), x, plan


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("other", [G, L, U, D])
@pytest.mark.parametrize("n", [1, 5, 64, 200, 332, 1030])
def test_diagonal_times_every_property(other, n, variant):
    for pa, pb in ((D, other), (other, D)):
        eq = Equation(f"scale_{pa}{pb}_{n}", 300 + n, (Operand(n, n, pa, "normal"), Operand(n, n, pb, "normal")))
        _, x, plan = both(eq, variant)
        assert plan.num_steps() == 1 and plan.step(0).kind == mom.KIND_SCALE
        if n >= 200 and other != D:          # one scaling pass is a single launch, also for large operands
            assert plan.last_launch_count() == 1


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_diagonal_times_rectangular(variant):
    both(Equation("dg", 31, (Operand(392, 392, D), Operand(392, 136, G, "normal"))), variant)
    both(Equation("gd", 32, (Operand(136, 392, G, "normal"), Operand(392, 392, D))), variant)
    both(Equation("dg_odd", 33, (Operand(37, 37, D), Operand(37, 3, G))), variant)        # columns not a multiple of 4
    both(Equation("gd_odd", 34, (Operand(3, 37, G), Operand(37, 37, D))), variant)


@pytest.mark.parametrize("variant", VARIANTS + [mom.VARIANT_3XTF32], ids=VNAME.get)
def test_scalings_inside_chains(variant):
    # the scaled value feeds a tensor-core product, and a tensor-core product feeds a scaling
    both(Equation("adb", 35, (Operand(520, 264, G, "normal"), Operand(264, 264, D), Operand(264, 776, G, "normal"))), variant)
    both(Equation("abd", 36, (Operand(520, 264, G, "normal"), Operand(264, 264, G, "normal"), Operand(264, 264, D))), variant)
    both(Equation("dlu", 37, (Operand(392, 392, D), Operand(392, 392, L), Operand(392, 392, U), Operand(392, 392, D))), variant)
    both(wl.config_diagonal(n=520), variant)
    # Add terms and the structure mask in the scaling kernel's epilogue
    n = 72
    for terms in ([Operand(n, n, L)], [Operand(n, n, U)], [Operand(n, n, I)], [Operand(n, n, D), Operand(n, n, I)],
                  [Operand(n, n, G, "normal") for _ in range(10)]):
        both(Equation("dl_plus", 38, (Operand(n, n, D), Operand(n, n, L)), tuple(terms)), variant)
        both(Equation("dd_plus", 39, (Operand(n, n, D), Operand(n, n, D)), tuple(terms)), variant)


@pytest.mark.parametrize("trans", [False, True])
@pytest.mark.parametrize("side", ["left_row", "left_col", "right_row", "right_col"])
def test_scaling_folded_into_the_operand_split(side, trans):
    # a scaling whose only reader is a tensor-core product costs no launch: the reader's split pass scales as it
    # reads.  The scaled matrix is the product's left or right operand, scaled by rows (D*S) or by columns (S*D),
    # stored as used or transposed.
    m, k, n = 264, 392, 520
    g = lambda r, c: Operand(c, r, G, "normal") if trans else Operand(r, c, G, "normal")
    if side == "left_row":      # (D * A) * B with a tall B, so that D joins A
        chain, ct = (Operand(m, m, D), g(m, k), Operand(k, n, G, "normal")), (False, trans, False)
    elif side == "left_col":    # (A * D) * B
        chain, ct = (g(m, k), Operand(k, k, D), Operand(k, n + 400, G, "normal")), (trans, False, False)
    elif side == "right_row":   # A * (D * B)
        chain, ct = (Operand(m + 400, k, G, "normal"), Operand(k, k, D), g(k, n)), (False, False, trans)
    else:                       # A * (B * D)
        chain, ct = (Operand(m + 400, k, G, "normal"), g(k, n), Operand(n, n, D)), (False, trans, False)
    eq = Equation(f"fold_{side}_{int(trans)}", 50, chain, (), 1, ct)
    _, x, plan = both(eq, mom.VARIANT_3XTF32_FORCE)
    kinds = [plan.step(i).kind for i in range(plan.num_steps())]
    assert kinds.count(mom.KIND_SCALE) == 1 and plan.step(kinds.index(mom.KIND_SCALE)).out != plan.step(plan.num_steps() - 1).out
    assert plan.last_launch_count() == 2        # the operand splits (one launch for both) and the product; no scaling launch
    # the other kernels take the scaled matrix from memory: same values
    both(eq, mom.VARIANT_3XTF32_WARP)
    both(eq, mom.VARIANT_FFMA)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_zero_step_plans_with_diagonals(variant):
    n = 33
    for chain, add in [((Operand(n, n, D),), ()), ((Operand(n, n, I),), (Operand(n, n, I),)),
                       ((Operand(n, n, D),), (Operand(n, n, I), Operand(n, n, D))),
                       ((Operand(n, n, I), Operand(n, n, D), Operand(n, n, I)), (Operand(n, n, U),))]:
        _, x, plan = both(Equation("zero_step_d", 40, chain, add), variant)
        assert plan.num_steps() == 0


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_transposed_operands_with_diagonals(variant):
    # D^T = D; the scaled operand may itself be stored transposed
    eq = Equation("dt_at", 41, (Operand(200, 200, D), Operand(136, 200, G, "normal")), (), 1, (True, True))
    both(eq, variant)
    eq = Equation("at_d", 42, (Operand(200, 136, G, "normal"), Operand(200, 200, D)), (Operand(200, 136, G),), 1, (True, False), (True,))
    both(eq, variant)
    eq = Equation("lt_d", 43, (Operand(65, 65, L), Operand(65, 65, D)), (), 1, (True, True))
    both(eq, variant)


@pytest.mark.parametrize("variant", [mom.VARIANT_FFMA, mom.VARIANT_3XTF32], ids=VNAME.get)
def test_batched_equations_with_diagonals(variant):
    # small: the whole plan in one fused launch; larger: one scaling launch and one product launch for the batch
    eq = Equation("b_small", 44, (Operand(64, 64, L), Operand(64, 64, D), Operand(64, 16, G)), (Operand(64, 16, G),), batch=37)
    _, x, plan = both(eq, variant)
    assert plan.last_launch_count() == 1
    eq = Equation("b_large", 45, (Operand(200, 200, D), Operand(200, 200, G, "normal"), Operand(200, 200, U)), (), batch=5)
    both(eq, variant)
    # tensor-core steps walk the instances one at a time; the folded scaling follows each instance's own D and S
    both(eq, mom.VARIANT_3XTF32_FORCE)
    eq = Equation("b_fold", 46, (Operand(264, 392, G, "normal"), Operand(392, 392, D), Operand(392, 520, G, "normal")), (Operand(264, 520, G),), batch=3)
    both(eq, mom.VARIANT_3XTF32_FORCE)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_random_equations_with_diagonals(variant):
    for seed in range(40):
        eq = wl.random_equation(2000 + seed, max_len=5, max_dim=40, dim_multiple=4 if seed % 2 else 1, diagonal=True)
        both(eq, variant)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_random_sums_and_expressions_with_diagonals(variant):
    for seed in range(25):
        eq = wl.random_sum_equation(3000 + seed, max_dim=40, dim_multiple=4 if seed % 2 else 1, diagonal=True)
        x, plan, arrays = run_sum_equation(eq, variant)
        check_sum_against_oracle(eq, x, plan, arrays)
    for seed in range(25):
        ex = wl.random_expression(3000 + seed, dim_multiple=4 if seed % 2 else 1, diagonal=True)
        x, plan, arrays = run_expression(ex, variant)
        check_expression_against_oracle(ex, x, plan, arrays)


def test_config_diagonal_full_size_sampled_rows():
    eq = wl.config_diagonal()
    x, plan, (chain, add) = run_equation(eq, mom.VARIANT_3XTF32)
    assert [plan.step(i).kind for i in range(plan.num_steps())].count(mom.KIND_SCALE) == 1
    check_against_oracle(eq, x, plan, chain, add, rows=stratified_rows(eq.chain[0].rows, 5))
