"""GPU parity for sums of several Mul chains: the CUDA path through the C ABI against the fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2208_10391_b200 as mom
from oracle import plan as op
from oracle import values as ov
import workloads as wl
from workloads import Operand, SumEquation, GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I
from gpu_util import run_sum_equation, check_sum_against_oracle, stratified_rows, TOL

pytestmark = pytest.mark.gpu

VARIANTS = [mom.VARIANT_3XTF32, mom.VARIANT_FFMA, mom.VARIANT_3XTF32_FORCE, mom.VARIANT_3XTF32_WARP, mom.VARIANT_3XTF32_INLINE]


def sum_eq(name, chains, transposed=None, names=None, seed=11):
    chains = tuple(tuple(Operand(*f) if isinstance(f, tuple) else f for f in c) for c in chains)
    if transposed is None:
        transposed = tuple((False,) * len(c) for c in chains)
    if names is None:
        k = iter(range(10 ** 6))
        names = tuple(tuple(next(k) for _ in c) for c in chains)
    return SumEquation(name, seed, chains, transposed, names)


@pytest.mark.parametrize("variant", VARIANTS)
def test_random_sums(variant):
    # FORCE sends every product with dimensions in multiples of 4 to the tensor-core kernel
    mult = 4 if variant == mom.VARIANT_3XTF32_FORCE else 1
    for seed in range(40):
        eq = wl.random_sum_equation(seed, max_dim=96, dim_multiple=mult)
        x, plan, arrays = run_sum_equation(eq, variant)
        check_sum_against_oracle(eq, x, plan, arrays)


@pytest.mark.parametrize("variant", VARIANTS)
def test_random_sums_without_names(variant):
    for seed in range(40, 60):
        eq = wl.random_sum_equation(seed, max_dim=64, dim_multiple=4)
        x, plan, arrays = run_sum_equation(eq, variant, use_names=False)
        check_sum_against_oracle(eq, x, plan, arrays, use_names=False)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("props", [((L, L), (U, U)), ((L, L), (L, L)), ((U, G), (G, L)), ((L, U), (U, L)),
                                   ((L, I), (G, G)), ((I, I), (G, U)), ((G, G), (I, I)), ((U, U), (I, U))])
def test_structured_pairs_of_chains(variant, props):
    # several tiles with a ragged tail; the first root must also write the part of X outside its own structure
    n = 332
    eq = sum_eq("pairs", [[(n, n, p) for p in chain] for chain in props])
    x, plan, arrays = run_sum_equation(eq, variant)
    check_sum_against_oracle(eq, x, plan, arrays)


@pytest.mark.parametrize("variant", VARIANTS)
def test_sum_without_any_product(variant):
    n = 200
    eq = sum_eq("terms_only", [[(n, n, G)], [(n, n, L)], [(n, n, I)], [(n, n, U)]],
                transposed=((True,), (True,), (False,), (False,)))
    x, plan, arrays = run_sum_equation(eq, variant)
    assert plan.num_steps() == 0
    check_sum_against_oracle(eq, x, plan, arrays)
    eq = sum_eq("identities_only", [[(n, n, I)], [(n, n, I), (n, n, I)]])
    x, plan, arrays = run_sum_equation(eq, variant)
    check_sum_against_oracle(eq, x, plan, arrays)
    assert np.array_equal(x, 2 * np.eye(n, dtype=np.float32))


@pytest.mark.parametrize("variant", VARIANTS)
def test_more_single_factor_chains_than_one_launch_takes(variant):
    m, n = 136, 260
    chains = [[(m, n, G)] for _ in range(5)] + [[(m, 64, G), (64, n, G)]] + [[(m, n, G)] for _ in range(6)]
    eq = sum_eq("many_terms", chains)
    x, plan, arrays = run_sum_equation(eq, variant)
    check_sum_against_oracle(eq, x, plan, arrays)


@pytest.mark.parametrize("variant", VARIANTS)
def test_rectangular_chains_on_several_tiles(variant):
    eq = sum_eq("rect", [[(384, 260, G), (260, 516, G)], [(384, 132, G), (132, 132, L), (132, 516, G)],
                         [(384, 384, U), (384, 516, G)]])
    x, plan, arrays = run_sum_equation(eq, variant)
    check_sum_against_oracle(eq, x, plan, arrays)


def test_split_k_roots_accumulate():
    # few output tiles and a long contraction: both roots run split over k and the second adds to X
    eq = sum_eq("splitk", [[(128, 4096, G), (4096, 256, G)], [(128, 2048, G), (2048, 256, G)]])
    x, plan, arrays = run_sum_equation(eq, mom.VARIANT_3XTF32_FORCE)
    assert all(s.uses_tensor_cores == 1 for s in plan.steps())
    check_sum_against_oracle(eq, x, plan, arrays)
    # the same roots on the warp-level kernel: the contraction is split over a thread-block cluster
    x, plan, arrays = run_sum_equation(eq, mom.VARIANT_3XTF32)
    assert all(s.uses_tensor_cores == 2 for s in plan.steps())
    check_sum_against_oracle(eq, x, plan, arrays)


@pytest.mark.parametrize("variant", VARIANTS)
def test_shared_product_is_computed_once_and_read_twice(variant):
    # (A*B) is below the root in both chains; C and D wide so that ((A*B)*.) is the cheaper tree
    a, b, c = (264, 520, G), (520, 264, G), (264, 1028, G)
    eq = sum_eq("shared", [[a, b, c], [a, b, c]], names=((0, 1, 2), (0, 1, 3)))
    x, plan, arrays = run_sum_equation(eq, variant)
    assert plan.reused_products() == 1 and plan.num_steps() == 3
    check_sum_against_oracle(eq, x, plan, arrays)
    # the same equation with nothing declared shared gives the same value with four products
    x2, plan2, arrays2 = run_sum_equation(eq, variant, use_names=False)
    assert plan2.num_steps() == 4
    check_sum_against_oracle(eq, x2, plan2, arrays2, use_names=False)


@pytest.mark.parametrize("variant", VARIANTS)
def test_shared_product_with_transposed_factors(variant):
    a, c = (520, 264, G), (264, 1028, G)
    eq = sum_eq("shared_t", [[a, (520, 264, G), c], [a, (520, 264, G), c], [(1028, 264, G)]],
                transposed=((True, False, False), (True, False, False), (True,)),
                names=((0, 1, 2), (0, 1, 3), (4,)))
    x, plan, arrays = run_sum_equation(eq, variant)
    assert plan.reused_products() == 1
    check_sum_against_oracle(eq, x, plan, arrays)


def test_named_factors_need_equal_pointers():
    a = (64, 64, G)
    plan = mom.mom_equation_plan_sum([[a, a], [a, a]], None, [[0, 1], [0, 2]])
    t = [torch.zeros(64, 64, device="cuda") for _ in range(4)]
    out = torch.zeros(64, 64, device="cuda")
    ws_bytes = plan.workspace_bytes(1)
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    with pytest.raises(mom.MomError) as e:
        plan.execute([x.data_ptr() for x in t], [], out.data_ptr(), ws.data_ptr(), ws_bytes)
    assert e.value.status == mom.ERR_INVALID_ARG
    plan.execute([t[0].data_ptr(), t[1].data_ptr(), t[0].data_ptr(), t[3].data_ptr()], [], out.data_ptr(),
                 ws.data_ptr(), ws_bytes)
    torch.cuda.synchronize()


def test_sum_through_the_host_entry_point():
    eq = wl.config_sum_shared(256)
    arrays = wl.generate_sum(eq)
    plan = mom.mom_equation_plan_sum(eq.descs(), eq.transposed, eq.names)
    stage_bytes = plan.host_staging_bytes(1)
    staging = torch.empty(stage_bytes, dtype=torch.uint8, device="cuda")
    pinned = {}
    ptrs = []
    for chain, names in zip(arrays, eq.names):
        for a, nm in zip(chain, names):
            if nm not in pinned:
                pinned[nm] = torch.from_numpy(a).pin_memory()
            ptrs.append(pinned[nm].data_ptr())
    out = torch.full((256 * 256,), float("nan")).pin_memory()
    plan.execute_host(ptrs, [], out.data_ptr(), 1, staging.data_ptr(), stage_bytes)
    check_sum_against_oracle(eq, out.numpy().reshape(256, 256).copy(), plan, arrays)


@pytest.mark.parametrize("eq", [wl.config_sum_shared(), wl.config_sum_triangular()], ids=lambda e: e.name)
def test_sum_configurations_full_size_sampled_rows(eq):
    x, plan, arrays = run_sum_equation(eq, mom.VARIANT_3XTF32)
    check_sum_against_oracle(eq, x, plan, arrays, rows=stratified_rows(x.shape[0], 5, extra=[0, x.shape[0] - 1]))


@pytest.mark.parametrize("variant", [mom.VARIANT_3XTF32, mom.VARIANT_3XTF32_FORCE])
def test_named_factor_on_both_sides_and_in_both_orientations(variant):
    # A is the left operand twice (one set of planes), the right operand once and enters transposed once
    n = 392
    a, g, l = (n, n, G), (n, n, G), (n, n, L)
    eq = sum_eq("factor_reuse", [[a, g], [a, l], [g, a], [a, g], [l, a]],
                transposed=((False, False), (False, False), (False, False), (True, False), (False, True)),
                names=((0, 1), (0, 2), (3, 0), (0, 4), (2, 0)))
    x, plan, arrays = run_sum_equation(eq, variant)
    check_sum_against_oracle(eq, x, plan, arrays)
