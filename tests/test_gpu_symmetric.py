"""GPU parity for Symmetric operands and Gram products Y * Y^T (lower triangle computed, upper one mirrored on
the tensor-core kernel), against the fp64 oracle through the C ABI."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2208_10391_b200 as mom
import workloads as wl
from workloads import (GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I, DIAGONAL as D, SYMMETRIC as S, Operand,
                       Equation, SumEquation)
from gpu_util import run_equation, check_against_oracle, run_sum_equation, check_sum_against_oracle, stratified_rows

pytestmark = pytest.mark.gpu

VARIANTS = [mom.VARIANT_3XTF32, mom.VARIANT_FFMA, mom.VARIANT_3XTF32_FORCE, mom.VARIANT_3XTF32_WARP, mom.VARIANT_3XTF32_INLINE]
VNAME = {mom.VARIANT_FFMA: "ffma", mom.VARIANT_3XTF32_FORCE: "tc", mom.VARIANT_3XTF32: "auto", mom.VARIANT_3XTF32_WARP: "warp", mom.VARIANT_3XTF32_INLINE: "inline"}


def both(eq, variant, **kw):
    x, plan, (chain, add) = run_equation(eq, variant)
    return check_against_oracle(eq, x, plan, chain, add, **kw), x, plan


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("other", [G, L, U, D, S])
@pytest.mark.parametrize("n", [5, 64, 200, 332])
def test_symmetric_operand_with_every_property(other, n, variant):
    for pa, pb in ((S, other), (other, S)):
        eq = Equation(f"sym_{pa}{pb}_{n}", 400 + n, (Operand(n, n, pa, "normal"), Operand(n, n, pb, "normal")),
                      (Operand(n, n, S),), 1, (pa == S, False))      # S^T = S: the flag changes nothing
        _, x, plan = both(eq, variant)
        assert plan.result_desc().property == G


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_symmetric_sums_and_zero_step_plans(variant):
    n = 72
    for chain, add, want in [((Operand(n, n, S),), (Operand(n, n, S), Operand(n, n, D), Operand(n, n, I)), S),
                             ((Operand(n, n, S),), (Operand(n, n, L),), G),
                             ((Operand(n, n, I), Operand(n, n, S)), (), S)]:
        _, x, plan = both(Equation("sym_sum", 60, chain, add), variant)
        assert plan.result_desc().property == want
        if want == S:
            assert np.array_equal(x, x.T)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_random_sums_with_gram_products(variant):
    grams = 0
    for seed in range(40):
        eq = wl.random_gram_sum(5000 + seed, dim_multiple=4 if seed % 2 else 1)
        x, plan, arrays = run_sum_equation(eq, variant)
        check_sum_against_oracle(eq, x, plan, arrays)
        grams += any(s.kind == mom.KIND_GRAM for s in plan.steps())
    assert grams >= 20


@pytest.mark.parametrize("terms", [False, True])
@pytest.mark.parametrize("shape", [(2056, 264), (1800, 520), (1288, 520)])
def test_large_gram_product_is_mirrored(shape, terms):
    # X = A * B * B^T * A^T (+ S): Y = A * B once, then the CTA-pair kernel computes the tiles on and below the diagonal
    # of Y * Y^T and writes the others as mirror images; a Symmetric summand is added on the way (its mirror image is itself).
    n, k = shape
    a = Operand(n, k, G, "normal", 1.0 / np.sqrt(k))
    b = Operand(k, k, G, "normal", 1.0 / np.sqrt(k))
    chains = ((a, b, b, a),) + (((Operand(n, n, S, "normal"),),) if terms else ())
    flags = ((False, False, True, True),) + (((False,),) if terms else ())
    names = ((0, 1, 1, 0),) + (((2,),) if terms else ())
    eq = SumEquation(f"gram_{n}_{k}_{int(terms)}", 61, chains, flags, names)
    x, plan, arrays = run_sum_equation(eq, mom.VARIANT_3XTF32_FORCE)
    steps = plan.steps()
    assert [s.kind for s in steps] == [mom.KIND_GG, mom.KIND_GRAM] and all(s.uses_tensor_cores == 1 for s in steps)
    assert plan.result_desc().property == S
    check_sum_against_oracle(eq, x, plan, arrays, rows=stratified_rows(n, 7, extra=[0, 255, 256, 257, n - 1]))
    pair_tiles = ((n + 255) // 256) ** 2               # the CTA-pair kernel (and with it the mirroring) needs 48 tiles of 256 x 256
    if pair_tiles >= 48:
        # mirror images are exact copies: outside the 256 x 256 diagonal blocks the result is exactly symmetric
        i, j = np.indices((n, n))
        off = (i // 256) != (j // 256)
        assert np.array_equal(x[off], x.T[off])
        # the splits of A and B (one launch), the product Y, the Gram product whose right planes are its left planes (no
        # split at all: Y arrives as planes)
        assert plan.last_launch_count() == 3 or terms
    assert np.allclose(x, x.T, rtol=0, atol=1e-5 * np.abs(x).max())
