"""GPU parity for equations with strictly triangular and unit triangular operands (kernels handle them as the
ordinary triangle around them; the diagonal of a strict result must come out as +0.0f and that of a unit result
as exactly 1) against the fp64 oracle through the C ABI: every kernel path, chains, sums and expressions."""
import itertools

import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2208_10391_b200 as mom
import workloads as wl
from workloads import (GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I, DIAGONAL as D, STRICT_LOWER as SL,
                       STRICT_UPPER as SU, UNIT_LOWER as UL, UNIT_UPPER as UU, Operand, Equation)
from gpu_util import (run_equation, check_against_oracle, run_sum_equation, check_sum_against_oracle, run_expression,
                      check_expression_against_oracle)

pytestmark = pytest.mark.gpu

VARIANTS = [mom.VARIANT_FFMA, mom.VARIANT_3XTF32_FORCE, mom.VARIANT_3XTF32_WARP, mom.VARIANT_3XTF32, mom.VARIANT_3XTF32_INLINE]
VNAME = {mom.VARIANT_FFMA: "ffma", mom.VARIANT_3XTF32_FORCE: "tc", mom.VARIANT_3XTF32: "auto", mom.VARIANT_3XTF32_WARP: "warp", mom.VARIANT_3XTF32_INLINE: "inline"}
KINDS = (SL, SU, UL, UU)


def both(eq, variant, **kw):
    x, plan, (chain, add) = run_equation(eq, variant)
    return check_against_oracle(eq, x, plan, chain, add, **kw), x, plan


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("n", [1, 5, 64, 200, 520])
def test_every_pair_of_types(n, variant):
    for pa, pb in itertools.product((G, L, U, D) + KINDS, KINDS):
        for a, b in ((pa, pb), (pb, pa)):
            eq = Equation(f"pair_{a}{b}_{n}", 500 + n, (Operand(n, n, a, "normal"), Operand(n, n, b, "normal")))
            _, x, plan = both(eq, variant)
            want = {(SL, SL): SL, (UL, UL): UL, (SL, UL): SL, (UL, SL): SL, (SU, SU): SU, (UU, UU): UU}.get((a, b))
            if want is not None:
                assert plan.result_desc().property == want


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_negative_scaling_leaves_plus_zero_on_a_strict_diagonal(variant):
    # d_i < 0 times the stored +0 of a strictly triangular factor is -0 unless the kernel adds +0
    n = 72
    eq = Equation("neg_scale", 77, (Operand(n, n, D), Operand(n, n, SL, "normal")))
    chain, add = wl.generate(eq)
    chain[0] = -chain[0]
    x, plan, _ = run_equation(eq, variant, chain=chain, add=add)
    check_against_oracle(eq, x, plan, chain, add)
    assert plan.result_desc().property == SL
    eq = Equation("neg_scale_r", 78, (Operand(n, n, SU, "normal"), Operand(n, n, D)))
    chain, add = wl.generate(eq)
    chain[1] = -chain[1]
    x, plan, _ = run_equation(eq, variant, chain=chain, add=add)
    check_against_oracle(eq, x, plan, chain, add)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_chains_with_add_terms_and_transposes(variant):
    n = 264
    g = Operand(n, n, G, "normal")
    both(Equation("nna", 80, (Operand(n, n, SL), Operand(n, n, SL), Operand(n, 520, G, "normal"))), variant)
    both(Equation("uub", 81, (Operand(n, n, UU), Operand(n, n, UU)), (Operand(n, n, SU), Operand(n, n, I))), variant)
    both(Equation("ulc", 82, (Operand(n, n, UL), Operand(n, n, SL)), (Operand(n, n, SL),)), variant)
    both(Equation("t", 83, (Operand(n, n, UL), g, Operand(n, n, SU)), (g,), chain_t=(True, False, True), add_t=(True,)), variant)
    both(Equation("tt", 84, (Operand(n, n, SL), Operand(n, n, UU)), (), chain_t=(False, True)), variant)
    both(Equation("i_plus", 85, (Operand(n, n, I),), (Operand(n, n, SL),)), variant)               # I + strictly lower = unit lower
    both(Equation("sum_only", 86, (Operand(n, n, SU),), (Operand(n, n, UU), Operand(n, n, D))), variant)
    both(Equation("dsl", 87, (Operand(n, n, D), Operand(n, n, UL), Operand(n, n, D), Operand(n, n, SL)), (Operand(n, n, SL),)), variant)
    both(Equation("batched", 88, (Operand(64, 64, UL), Operand(64, 64, SL), Operand(64, 16)), (Operand(64, 16),), batch=37), variant)
    both(Equation("batched_tri", 89, (Operand(48, 48, UL), Operand(48, 48, UL)), (Operand(48, 48, SL),), batch=21), variant)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_large_strict_operands_through_the_host_entry_point(variant):
    # triangular operands of 1024 rows and more are uploaded block by block; strict and unit ones likewise
    n = 1288
    eq = Equation("host", 90, (Operand(n, n, SL, "normal"), Operand(n, n, G, "normal"), Operand(n, n, UU, "normal")),
                  (Operand(n, n, G, "normal"),))
    x, plan, (chain, add) = run_equation(eq, variant, via="host")
    rows = np.unique(np.r_[0:3, n - 3:n, np.random.default_rng(1).integers(0, n, 40)])
    check_against_oracle(eq, x, plan, chain, add, rows=rows)
    assert plan.host_upload_bytes() < 3.3 * n * n * 4          # two full matrices and two triangles by blocks


@pytest.mark.parametrize("seed", range(40))
def test_random_equations(seed):
    variant = VARIANTS[seed % len(VARIANTS)]
    eq = wl.random_equation(3000 + seed, max_len=5, max_dim=160, kinds=True, dim_multiple=4 if seed % 3 else 1)
    both(eq, variant)


@pytest.mark.parametrize("seed", range(24))
def test_random_sums_and_expressions(seed):
    variant = VARIANTS[seed % len(VARIANTS)]
    eq = wl.random_sum_equation(3100 + seed, max_dim=96, kinds=True, dim_multiple=4 if seed % 2 else 1)
    x, plan, arrays = run_sum_equation(eq, variant)
    check_sum_against_oracle(eq, x, plan, arrays)
    ex = wl.random_expression(3200 + seed, max_dim=96, kinds=True, dim_multiple=4 if seed % 2 else 1)
    x, plan, arrays = run_expression(ex, variant)
    check_expression_against_oracle(ex, x, plan, arrays)
