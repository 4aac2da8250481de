"""GPU parity of the column-slab split: the slabs of X that the devices of a group would compute are evaluated one
after the other on this GPU through the C ABI (each as an equation of its own, as on its own device) and put side by
side; the result must match the fp64 oracle's value of the whole equation."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2208_10391_b200 as mom
import workloads as wl
from workloads import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, Operand, Equation
from oracle import values as ov
from gpu_util import run_equation, TOL
from test_column_slab import slab_arrays, whole_value

pytestmark = pytest.mark.gpu

VARIANTS = [mom.VARIANT_FFMA, mom.VARIANT_3XTF32_FORCE, mom.VARIANT_3XTF32]
VNAME = {mom.VARIANT_FFMA: "ffma", mom.VARIANT_3XTF32_FORCE: "tc", mom.VARIANT_3XTF32: "auto"}


def slab_equation(eq, rank, world):
    got = mom.column_slab_equation(eq.descs(), eq.add_descs(), rank, world, eq.chain_t, eq.add_t)
    if got is None:
        return None
    cd, ad, begin, end = got
    ops = tuple(Operand(d.rows, d.cols, d.property) for d in cd)
    terms = tuple(Operand(d.rows, d.cols, d.property) for d in ad)
    return Equation(f"{eq.name}_slab{rank}of{world}", eq.seed, ops, terms, chain_t=eq.chain_t, add_t=eq.add_t), begin, end


def evaluate_by_slabs(eq, world, variant):
    chain, add = wl.generate(eq)
    x_ref, den = whole_value(eq, chain, add)
    x = np.full(x_ref.shape, np.nan, dtype=np.float32)
    for rank in range(world):
        got = slab_equation(eq, rank, world)
        if got is None:
            continue
        seq, b, e = got
        c, a = slab_arrays(eq, chain, add, b, e)
        xs, plan, _ = run_equation(seq, variant, chain=c, add=a)
        x[:, b:e] = xs
    assert not np.isnan(x).any()
    err = ov.normwise_error(x.astype(np.float64), x_ref, den)
    assert err <= TOL, f"normwise error {err:.3e} ({eq.name}, {world} slabs)"
    return err


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("world", [2, 3, 8])
def test_property_chain_by_slabs(world, variant):
    evaluate_by_slabs(wl.config_large_square(n=776), world, variant)             # L*A*U*B: the slab of B stays general
    evaluate_by_slabs(wl.config_property_heavy(n=520), world, variant)           # L*U*I*B + C
    evaluate_by_slabs(wl.config_transposed(n=392), world, variant)               # transposed factors and Add term


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_ragged_and_degenerate_slabs(variant):
    evaluate_by_slabs(wl.config_paper_chain(), 8, variant)                       # 100 columns over 8 devices: 12, 12, 12, 16, ...
    evaluate_by_slabs(wl.config_tiny(), 16, variant)                             # 48 columns, 16 devices: some get nothing
    eq = Equation("tri_last", 41, (Operand(264, 264, G, "normal"), Operand(264, 264, U)), (Operand(264, 264, L),))
    evaluate_by_slabs(eq, 4, variant)                                            # a triangular last factor and term are cut as general
    eq = Equation("last_t", 42, (Operand(136, 264, G, "normal"), Operand(520, 264, G, "normal")), (), chain_t=(False, True))
    evaluate_by_slabs(eq, 3, variant)                                            # the last factor is used transposed: its slab is a row block
    for seed in range(10):
        evaluate_by_slabs(wl.random_equation(800 + seed, max_len=4, max_dim=120, kinds=True), 1 + seed % 4, variant)
