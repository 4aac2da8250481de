"""Plan parity (integer work, bit-exact): the library's planner against the exhaustive oracle. CPU only."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2208_10391_b200 as mom
from oracle import plan as op
import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def assert_same_plan(chain, add=(), variant=mom.VARIANT_3XTF32):
    want = op.plan(chain, add)
    got = mom.mom_equation_plan(chain, add, variant)
    assert got.parenthesization() == want.paren
    assert got.flops() == (want.mul_flops, want.add_flops)
    rd = got.result_desc()
    assert (rd.rows, rd.cols, rd.property) == (want.result_desc.rows, want.result_desc.cols, want.result_desc.prop)
    steps = got.steps()
    assert len(steps) == len(want.steps)
    for g, w in zip(steps, want.steps):
        assert (g.lhs, g.rhs, g.out, g.m, g.n, g.k) == (w.lhs, w.rhs, w.out, w.m, w.n, w.k)
        assert (g.lhs_property, g.rhs_property, g.out_property, g.useful_mults) == (w.lhs_prop, w.rhs_prop, w.out_prop, w.mults)
    return got, want


def test_header_symbols_are_exported():
    text = open(os.path.join(ROOT, "include", "mom.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(mom_[a-z0-9_]+)\s*\(", text))
    assert {"mom_matrix_desc", "mom_equation_plan", "mom_equation_execute"} <= declared
    lib = ctypes.CDLL(mom.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in mom.h but not exported"
    assert declared == set(mom.EXPORTED)


@pytest.mark.parametrize("eq", [
    wl.config_tiny(), wl.config_tiny_identity_left(), wl.config_tiny_identity_right(), wl.config_five_general(),
    wl.config_property_heavy(), wl.config_large_square(), wl.config_batched(), wl.config_paper_chain(),
    wl.config_listing2()], ids=lambda e: e.name)
def test_benchmark_configurations(eq):
    for variant in (mom.VARIANT_3XTF32, mom.VARIANT_FFMA):
        assert_same_plan(eq.descs(), eq.add_descs(), variant)


def test_random_equations_match_the_oracle():
    for seed in range(300):
        eq = wl.random_equation(seed, max_len=9, max_dim=50)
        assert_same_plan(eq.descs(), eq.add_descs())


def test_random_equations_with_diagonal_operands_match_the_oracle():
    diag = 0
    for seed in range(300):
        eq = wl.random_equation(seed, max_len=9, max_dim=50, diagonal=True)
        got, _ = assert_same_plan(eq.descs(), eq.add_descs())
        diag += any(got.step(i).kind == mom.KIND_SCALE for i in range(got.num_steps()))
    assert diag > 100
    # equal dimensions: many ties between the sides a Diagonal factor can join
    rng = np.random.default_rng(4)
    for _ in range(60):
        chain = [(12, 12, int(rng.integers(0, 5))) for _ in range(int(rng.integers(2, 9)))]
        add = [(12, 12, int(rng.integers(0, 5))) for _ in range(int(rng.integers(0, 3)))]
        assert_same_plan(chain, add)


def test_random_equations_with_strict_and_unit_triangles_match_the_oracle():
    for seed in range(300):
        eq = wl.random_equation(seed, max_len=9, max_dim=50, kinds=True)
        assert_same_plan(eq.descs(), eq.add_descs())
    # equal dimensions, every property: ties and every pair of types in the cost and type rules
    rng = np.random.default_rng(6)
    for _ in range(150):
        chain = [(9, 9, int(rng.integers(0, 10))) for _ in range(int(rng.integers(1, 8)))]
        add = [(9, 9, int(rng.integers(0, 10))) for _ in range(int(rng.integers(0, 4)))]
        assert_same_plan(chain, add)
    for pa in range(10):                                             # each pair, on its own and transposed
        for pb in range(10):
            assert_same_plan([(7, 7, pa), (7, 7, pb)])
            assert_same_plan([(7, 7, pa)], [(7, 7, pb)])
            assert_same_sum_plan([[(7, 7, pa), (7, 7, pb)]], [[True, False]], None)
            assert_same_sum_plan([[(7, 7, pa), (7, 7, pb), (7, 7, pb), (7, 7, pa)]], [[False, False, True, True]], [[0, 1, 1, 0]])
    for seed in range(150):
        eq = wl.random_sum_equation(seed, kinds=True)
        assert_same_sum_plan(eq.descs(), eq.transposed, eq.names)
    for seed in range(150):
        ex = wl.random_expression(seed, kinds=True)
        assert_same_expression_plan(ex.expr, ex.descs())


def test_long_chains_with_many_ties():
    # equal dimensions everywhere: every tree of an all-general chain ties; mixed properties tie partially
    rng = np.random.default_rng(3)
    for _ in range(40):
        n = int(rng.integers(2, 10))
        chain = [(16, 16, int(rng.integers(0, 4))) for _ in range(n)]
        assert_same_plan(chain)


def test_identity_only_and_single_operand():
    got, _ = assert_same_plan([(7, 7, mom.IDENTITY)] * 3)
    assert got.parenthesization() == "I" and got.num_steps() == 0
    got, _ = assert_same_plan([(7, 9, mom.GENERAL)])
    assert got.parenthesization() == "0"
    assert_same_plan([(7, 7, mom.IDENTITY)], [(7, 7, mom.IDENTITY), (7, 7, mom.UPPER_TRI)])


@pytest.mark.parametrize("chain,add,status,code", [
    ([(0, 3, 0)], [], mom.ERR_INVALID_ARG, "invalid_arg"),
    ([(3, 4, 1)], [], mom.ERR_PROPERTY, "property"),
    ([(3, 4, 3)], [], mom.ERR_PROPERTY, "property"),
    ([(3, 4, 4)], [], mom.ERR_PROPERTY, "property"),
    ([(3, 4, 5)], [], mom.ERR_PROPERTY, "property"),
    ([(3, 3, 0)], [(3, 3, 10)], mom.ERR_INVALID_ARG, "property"),
    ([(3, 4, 6)], [], mom.ERR_PROPERTY, "property"),
    ([(3, 4, 9)], [], mom.ERR_PROPERTY, "property"),
    ([(3, 4, 0), (5, 3, 0)], [], mom.ERR_SHAPE_MISMATCH, "shape_mismatch"),
    ([(3, 4, 0)], [(3, 5, 0)], mom.ERR_SHAPE_MISMATCH, "shape_mismatch"),
])
def test_errors_agree_with_the_oracle(chain, add, status, code):
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan(chain, add)
    assert e.value.status == status
    with pytest.raises(op.OracleError) as o:
        op.plan(chain, add)
    assert o.value.code == code


def test_more_errors():
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan([], [])
    assert e.value.status == mom.ERR_INVALID_ARG
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan([(3, 3, 0, 5)], [])
    assert e.value.status == mom.ERR_DTYPE
    with pytest.raises(mom.MomError) as e:
        mom.mom_matrix_desc(3, 4, mom.LOWER_TRI)
    assert e.value.status == mom.ERR_PROPERTY
    big = (1 << 31) - 2048                                    # the largest dimensions the library takes: the count overflows
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan([(big, big, 0), (big, big, 0)], [])
    assert e.value.status == mom.ERR_OVERFLOW
    assert mom.status_string(mom.ERR_OVERFLOW)
    with pytest.raises(mom.MomError) as e:                      # a Gram product's multiplication count overflows too
        mom.mom_equation_plan_sum([[(big, big, 0), (big, big, 0)]], [[False, True]], [[0, 0]])
    assert e.value.status == mom.ERR_OVERFLOW
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan([(4, 4, 0)], [], 5)               # unknown variant
    assert e.value.status == mom.ERR_INVALID_ARG


def test_workspace_covers_intermediates_and_planes():
    eq = wl.config_large_square()
    p = mom.mom_equation_plan(eq.descs(), (), mom.VARIANT_FFMA)
    n = 8192
    # chain of three products: two intermediates are alive at most one at a time besides the one being read
    assert p.workspace_bytes() == 2 * n * n * 4
    assert all(s.uses_tensor_cores == 0 for s in p.steps())
    p = mom.mom_equation_plan(eq.descs(), (), mom.VARIANT_3XTF32)
    assert all(s.uses_tensor_cores == 1 for s in p.steps())
    assert p.workspace_bytes() >= 2 * n * n * 4 + 4 * n * n * 4
    # shapes TMA cannot address fall back to FFMA when the tcgen05 kernel is forced; in the default variant they and small
    # products run on the warp-level kernel, the Section-4 chain's products on the one-launch tcgen05 kernel
    p = mom.mom_equation_plan([(5, 5, 1), (5, 5, 1)], (), mom.VARIANT_3XTF32_FORCE)
    assert p.step(0).uses_tensor_cores == 0
    p = mom.mom_equation_plan(wl.config_tiny().descs(), (), mom.VARIANT_3XTF32)
    assert all(s.uses_tensor_cores == 2 for s in p.steps())
    p = mom.mom_equation_plan(wl.config_paper_chain().descs(), (), mom.VARIANT_3XTF32)
    up = lambda b: (b + 255) // 256 * 256          # two f32 intermediates, no operand planes
    assert all(s.uses_tensor_cores == 3 for s in p.steps()) and p.workspace_bytes() == up(900 * 100 * 4) + up(1100 * 100 * 4)
    p = mom.mom_equation_plan([(1001, 1001, 0), (1001, 1001, 0)], (), mom.VARIANT_3XTF32)
    assert p.step(0).uses_tensor_cores == 2
    p = mom.mom_equation_plan(wl.config_property_heavy().descs(), (), mom.VARIANT_3XTF32_WARP)
    assert all(s.uses_tensor_cores == 2 for s in p.steps())
    p = mom.mom_equation_plan(wl.config_tiny().descs(), (), mom.VARIANT_3XTF32_FORCE)
    assert all(s.uses_tensor_cores == 1 for s in p.steps())
    assert mom.mom_equation_plan(wl.config_tiny_identity_left().descs()).workspace_bytes() == 0


def test_host_upload_bytes_count_triangles_by_blocks():
    n = 1288
    blocks = [(r0, min(n, r0 + 256)) for r0 in range(0, n, 256)]
    lower = sum((r1 - r0) * r1 for r0, r1 in blocks) * 4
    upper = sum((r1 - r0) * (n - r0) for r0, r1 in blocks) * 4
    L, U, G, I = mom.LOWER_TRI, mom.UPPER_TRI, mom.GENERAL, mom.IDENTITY
    p = mom.mom_equation_plan([(n, n, L), (n, n, I), (n, n, G), (n, n, U)], [(n, n, G)])
    assert p.host_upload_bytes(1) == lower + upper + 2 * n * n * 4           # Identity is never copied
    assert p.host_upload_bytes(3) == 3 * 5 * n * n * 4 - 3 * n * n * 4       # batches are copied in full
    small = mom.mom_equation_plan([(512, 512, L), (512, 512, G)])
    assert small.host_upload_bytes(1) == 2 * 512 * 512 * 4                   # below 1024 rows: one plain copy
    shared = mom.mom_equation_plan_sum([[(64, 64, G), (64, 64, G)], [(64, 64, G)]], None, [[0, 1], [0]])
    assert shared.host_upload_bytes(1) == 2 * 64 * 64 * 4                    # a named matrix once


def test_step_kinds():
    L, U, G = mom.LOWER_TRI, mom.UPPER_TRI, mom.GENERAL
    cases = {(G, G): mom.KIND_GG, (L, G): mom.KIND_TG, (U, G): mom.KIND_TG, (G, L): mom.KIND_GT, (G, U): mom.KIND_GT,
             (L, L): mom.KIND_TT, (U, U): mom.KIND_TT, (L, U): mom.KIND_TTMIX, (U, L): mom.KIND_TTMIX}
    D = mom.DIAGONAL
    cases.update({(D, G): mom.KIND_SCALE, (G, D): mom.KIND_SCALE, (D, L): mom.KIND_SCALE, (U, D): mom.KIND_SCALE, (D, D): mom.KIND_SCALE})
    for (a, b), kind in cases.items():
        p = mom.mom_equation_plan([(8, 8, a), (8, 8, b)])
        assert p.step(0).kind == kind
        assert not (kind == mom.KIND_SCALE and p.step(0).uses_tensor_cores)
    # a scaling never runs on tensor cores, whatever its size
    p = mom.mom_equation_plan([(4096, 4096, D), (4096, 4096, G)])
    assert p.step(0).kind == mom.KIND_SCALE and not p.step(0).uses_tensor_cores


def test_transposed_operands_match_the_oracle():
    rng = np.random.default_rng(17)
    for seed in range(200):
        eq = wl.random_equation(5000 + seed, max_len=7, max_dim=40)
        ct = [bool(rng.integers(0, 2)) for _ in eq.chain]
        at = [bool(rng.integers(0, 2)) for _ in eq.add]
        # store the flagged operands transposed, so that the equation as used stays well-formed
        swap = {mom.LOWER_TRI: mom.UPPER_TRI, mom.UPPER_TRI: mom.LOWER_TRI}
        stored_c = [(c, r, swap.get(p, p)) if t else (r, c, p) for (r, c, p), t in zip(eq.descs(), ct)]
        stored_a = [(c, r, swap.get(p, p)) if t else (r, c, p) for (r, c, p), t in zip(eq.add_descs(), at)]
        want = op.plan(stored_c, stored_a, ct, at)
        got = mom.mom_equation_plan_transposed(stored_c, ct, stored_a, at)
        assert got.parenthesization() == want.paren
        assert got.flops() == (want.mul_flops, want.add_flops)
        rd = got.result_desc()
        assert (rd.rows, rd.cols, rd.property) == (want.result_desc.rows, want.result_desc.cols, want.result_desc.prop)
        for g, w in zip(got.steps(), want.steps):
            assert (g.lhs, g.rhs, g.out, g.m, g.n, g.k, g.useful_mults) == (w.lhs, w.rhs, w.out, w.m, w.n, w.k, w.mults)
            assert g.lhs_transposed == int(g.lhs < len(ct) and ct[g.lhs]) and g.rhs_transposed == int(g.rhs < len(ct) and ct[g.rhs])
    # the paper's rule: the transpose of a lower-triangular matrix is upper triangular
    p = mom.mom_equation_plan_transposed([(9, 9, mom.LOWER_TRI), (9, 9, mom.LOWER_TRI)], [True, True])
    assert p.result_desc().property == mom.UPPER_TRI and p.parenthesization() == "(0^T*1^T)"
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan_transposed([(7, 30, 0), (7, 40, 0)], [False, False])
    assert e.value.status == mom.ERR_SHAPE_MISMATCH
    assert mom.mom_equation_plan_transposed([(7, 30, 0), (7, 40, 0)], [True, False]).result_desc().rows == 30


# ---- sums of several chains ---------------------------------------------------------------------------

def assert_same_sum_plan(chains, transposed=None, names=None, variant=mom.VARIANT_3XTF32):
    want = op.plan_sum(chains, transposed or (), names or ())
    got = mom.mom_equation_plan_sum(chains, transposed, names, variant)
    assert got.parenthesization() == want.paren
    assert got.flops() == (want.mul_flops, want.add_flops)
    assert got.reused_products() == want.reused
    rd = got.result_desc()
    assert (rd.rows, rd.cols, rd.property) == (want.result_desc.rows, want.result_desc.cols, want.result_desc.prop)
    steps = got.steps()
    assert len(steps) == len(want.steps)
    for g, w in zip(steps, want.steps):
        assert (g.lhs, g.rhs, g.out, g.m, g.n, g.k) == (w.lhs, w.rhs, w.out, w.m, w.n, w.k)
        assert (g.lhs_property, g.rhs_property, g.out_property, g.useful_mults) == (w.lhs_prop, w.rhs_prop, w.out_prop, w.mults)
    return got, want


def test_random_sums_of_chains_match_the_oracle():
    shared = 0
    for seed in range(400):
        eq = wl.random_sum_equation(seed)
        got, want = assert_same_sum_plan(eq.descs(), eq.transposed, eq.names)
        shared += want.reused > 0
        assert_same_sum_plan(eq.descs(), eq.transposed, None)        # nothing known to be shared
    assert shared >= 20
    for seed in range(200):                                          # with Diagonal factors
        eq = wl.random_sum_equation(seed, diagonal=True)
        assert_same_sum_plan(eq.descs(), eq.transposed, eq.names)


def test_gram_products_match_the_oracle():
    grams = shared = 0
    for seed in range(400):
        eq = wl.random_gram_sum(seed)
        got, want = assert_same_sum_plan(eq.descs(), eq.transposed, eq.names)
        grams += any(s.gram for s in want.steps)
        shared += want.reused > 0
        for g, w in zip(got.steps(), want.steps):
            assert (g.kind == mom.KIND_GRAM) == w.gram
            if w.gram:
                assert g.lhs == g.rhs and g.rhs_transposed != g.lhs_transposed
        assert_same_sum_plan(eq.descs(), eq.transposed, None)          # without names there is no Gram product
    assert grams >= 250 and shared >= 40
    A, S = (10, 4, mom.GENERAL), (10, 10, mom.SYMMETRIC)
    got, want = assert_same_sum_plan([[A, A], [S]], [[False, True], [False]], [[0, 0], [1]])
    assert got.parenthesization() == "(0*1^T)+2" and got.flops() == (2 * 220, 100) and got.result_desc().property == mom.SYMMETRIC
    got, _ = assert_same_sum_plan([[A, A]], [[False, True]], None)
    assert got.flops()[0] == 2 * 400 and got.result_desc().property == mom.GENERAL
    eq = wl.config_gram()
    got, want = assert_same_sum_plan(eq.descs(), eq.transposed, eq.names)
    n, k = 4096, 2048
    assert got.parenthesization() == "((0*1)*(2^T*3^T))+4" and want.mults == n * k * k + k * n * (n + 1) // 2
    assert [s.kind for s in got.steps()] == [mom.KIND_GG, mom.KIND_GRAM] and got.result_desc().property == mom.SYMMETRIC


def test_sum_plan_shares_a_product_between_chains():
    G = mom.GENERAL
    a, b, c = (8, 50, G), (50, 8, G), (8, 100, G)
    got, want = assert_same_sum_plan([[a, b, c], [a, b, c]], None, [[0, 1, 2], [0, 1, 3]])
    assert got.reused_products() == 1 and got.num_steps() == 3
    assert got.parenthesization() == "((0*1)*2)+((3*4)*5)"
    # a shared run of three factors saves its two products
    d = (100, 7, G)
    got, _ = assert_same_sum_plan([[a, b, a, (50, 300, G)], [a, b, a, (50, 300, G)]], None, [[0, 1, 0, 2], [0, 1, 0, 3]])
    assert got.reused_products() >= 1


def test_sum_plan_of_one_chain_equals_the_chain_plan():
    for seed in range(60):
        eq = wl.random_equation(seed, max_len=7, max_dim=40, allow_add=False)
        one = mom.mom_equation_plan(eq.descs())
        many = mom.mom_equation_plan_sum([eq.descs()])
        assert one.parenthesization() == many.parenthesization() and one.flops() == many.flops()


@pytest.mark.parametrize("chains,names,status,code", [
    ([], None, mom.ERR_INVALID_ARG, "invalid_arg"),
    ([[(4, 5, 0)], [(5, 4, 0)]], None, mom.ERR_SHAPE_MISMATCH, "shape_mismatch"),
    ([[(4, 5, 0), (4, 5, 0)]], None, mom.ERR_SHAPE_MISMATCH, "shape_mismatch"),
    ([[(4, 4, 0)], [(4, 4, 1)]], [[0], [0]], mom.ERR_INVALID_ARG, "invalid_arg"),
    ([[(4, 4, 0)], []], None, mom.ERR_INVALID_ARG, None),
])
def test_sum_plan_errors(chains, names, status, code):
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan_sum(chains, None, names)
    assert e.value.status == status
    if code is not None:
        with pytest.raises(op.OracleError) as oe:
            op.plan_sum(chains, (), names or ())
        assert oe.value.code == code


# ---- nested expressions -------------------------------------------------------------------------------

def assert_same_expression_plan(expr, operands, variant=mom.VARIANT_3XTF32):
    want = op.plan_expr(expr, operands)
    got = mom.mom_expression_plan(expr, operands, variant)
    assert got.parenthesization() == want.paren
    assert got.flops() == (want.mul_flops, want.add_flops)
    assert (got.temporaries(), got.reused_products()) == (want.temporaries, want.reused)
    rd = got.result_desc()
    assert (rd.rows, rd.cols, rd.property) == (want.result_desc.rows, want.result_desc.cols, want.result_desc.prop)
    assert [(s.m, s.n, s.k, s.lhs_property, s.rhs_property, s.out_property, s.useful_mults) for s in got.steps()] == list(want.products)
    return got, want


def test_random_expressions_match_the_oracle():
    nested = 0
    for seed in range(500):
        ex = wl.random_expression(seed)
        _, want = assert_same_expression_plan(ex.expr, ex.descs())
        nested += want.temporaries > 0
    assert nested >= 100
    for seed in range(200):                                          # with Diagonal operands
        ex = wl.random_expression(seed, diagonal=True)
        assert_same_expression_plan(ex.expr, ex.descs())


def test_expression_plan_examples():
    G, L = mom.GENERAL, mom.LOWER_TRI
    ops = [(10, 10, G)] * 3
    got, _ = assert_same_expression_plan(("mul", [0, ("add", [1, 2])]), ops)
    assert got.parenthesization() == "(0*[1+2])" and got.num_steps() == 1 and got.temporaries() == 1
    # the same nested sum twice is one temporary; a product of the temporary is shared like any other
    e = ("add", [("mul", [0, ("add", [1, 2]), 0]), ("mul", [0, ("add", [1, 2]), 1])])
    got, want = assert_same_expression_plan(e, ops)
    assert got.temporaries() == 1
    # flattening and transposes
    got, _ = assert_same_expression_plan(("t", ("mul", [("mul", [0, 1]), ("t", 2)])), ops)
    assert got.parenthesization() == "(2*(1^T*0^T))"
    assert_same_expression_plan(("mul", [0, ("add", [1, 2])]), [(10, 10, L)] * 3)
    assert_same_expression_plan(wl.config_expression().expr, wl.config_expression().descs())


@pytest.mark.parametrize("expr,operands,status,code", [
    (("mul", [0, ("add", [1, 2])]), [(4, 5, 0), (5, 6, 0), (6, 5, 0)], mom.ERR_SHAPE_MISMATCH, "shape_mismatch"),
    (("mul", [0, 7]), [(4, 5, 0)], mom.ERR_INVALID_ARG, "invalid_arg"),
    (("add", []), [(4, 5, 0)], mom.ERR_INVALID_ARG, "invalid_arg"),
    (("add", [0, ("t", 0)]), [(4, 5, 0)], mom.ERR_SHAPE_MISMATCH, "shape_mismatch"),
])
def test_expression_plan_errors(expr, operands, status, code):
    with pytest.raises(mom.MomError) as e:
        mom.mom_expression_plan(expr, operands)
    assert e.value.status == status
    with pytest.raises(op.OracleError) as oe:
        op.plan_expr(expr, operands)
    assert oe.value.code == code


def test_expression_node_arrays_are_validated():
    ops = mom._desc_array([(4, 4, 0)])
    handle = ctypes.c_void_p()
    lib = mom._lib
    cyc = (mom.ExprNode * 1)(mom.ExprNode(mom.EXPR_TRANSPOSE, 0, 0, 1))          # a node that is its own child
    kids = (ctypes.c_int32 * 1)(0)
    assert lib.mom_expression_plan(ops, 1, cyc, 1, kids, 1, 0, 0, ctypes.byref(handle)) == mom.ERR_INVALID_ARG
    bad = (mom.ExprNode * 1)(mom.ExprNode(mom.EXPR_MUL, 0, 0, 3))                # children out of range
    assert lib.mom_expression_plan(ops, 1, bad, 1, kids, 1, 0, 0, ctypes.byref(handle)) == mom.ERR_INVALID_ARG
    unk = (mom.ExprNode * 1)(mom.ExprNode(9, 0, 0, 1))
    assert lib.mom_expression_plan(ops, 1, unk, 1, kids, 1, 0, 0, ctypes.byref(handle)) == mom.ERR_INVALID_ARG
    leaf = (mom.ExprNode * 1)(mom.ExprNode(mom.EXPR_OPERAND, 0, 0, 0))
    assert lib.mom_expression_plan(ops, 1, leaf, 1, kids, 0, 5, 0, ctypes.byref(handle)) == mom.ERR_INVALID_ARG
    assert lib.mom_expression_plan(ops, 1, leaf, 1, kids, 0, 0, 0, ctypes.byref(handle)) == mom.OK
    lib.mom_plan_destroy(handle)


def test_size_limits_of_the_library():
    D = lambda r, c: (r, c, wl.GENERAL)
    # every kernel indexes with 32-bit integers: larger dimensions are refused when the plan is made
    big = 2 ** 31
    with pytest.raises(mom.MomError) as e:
        mom.mom_matrix_desc(big, 8)
    assert e.value.status == mom.ERR_LIMIT
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan([D(8, big), D(big, 8)], [], mom.VARIANT_3XTF32)
    assert e.value.status == mom.ERR_LIMIT
    # the plane-fed tcgen05 kernel's tile table keeps a tile's first row in 24 bits: a taller (or wider) product goes to
    # the warp-level kernel (default variant) or the FFMA kernel (forced variant)
    tall = 2 ** 24
    for m, n in ((tall, 64), (64, tall), (tall - 1024 + 4, 64)):
        for variant, want in ((mom.VARIANT_3XTF32, 2), (mom.VARIANT_3XTF32_FORCE, 0)):
            plan = mom.mom_equation_plan([D(m, 64), D(64, n)], [], variant)
            assert plan.step(0).uses_tensor_cores == want
    plan = mom.mom_equation_plan([D(tall - 1024, 64), D(64, 64)], [], mom.VARIANT_3XTF32)
    assert plan.step(0).uses_tensor_cores == 1           # m*n*k is above the size rule and the rows fit the table


def test_planning_from_several_threads():
    # planning is a pure function of its arguments: the same plans whether made one by one or from eight threads at once
    import threading
    eqs = [wl.random_equation(seed, max_len=9, max_dim=50) for seed in range(64)]
    want = [(p.parenthesization(), p.flops()) for p in (mom.mom_equation_plan(e.descs(), e.add_descs(), mom.VARIANT_3XTF32) for e in eqs)]
    got = [[None] * len(eqs) for _ in range(8)]
    def work(slot):
        for rep in range(5):
            for i, e in enumerate(eqs):
                p = mom.mom_equation_plan(e.descs(), e.add_descs(), mom.VARIANT_3XTF32)
                got[slot][i] = (p.parenthesization(), p.flops())
                del p                                      # destroys the plan (no device state was ever created)
    threads = [threading.Thread(target=work, args=(s,)) for s in range(8)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert all(g == want for g in got)


def test_packed_container_matches_the_oracle_definition():
    # integer work: the library's closed forms against the oracle's row-by-row sums, bit for bit
    from oracle import packed as pk
    for n in list(range(1, 41)) + [63, 64, 65, 200, 333]:
        for prop in (wl.LOWER_TRI, wl.UPPER_TRI, wl.STRICT_LOWER, wl.STRICT_UPPER, wl.UNIT_LOWER, wl.UNIT_UPPER):
            oracle_prop = pk.LOWER_TRI if prop in (wl.LOWER_TRI, wl.STRICT_LOWER, wl.UNIT_LOWER) else pk.UPPER_TRI
            assert mom.mom_packed_elements(n, prop) == pk.elements(n, oracle_prop)
            for i in sorted({0, 1, 2, 3, 4, n // 2, n - 2, n - 1} & set(range(n))):
                off, first, end = mom.mom_packed_row(n, prop, i)
                assert off == pk.row_offset(n, oracle_prop, i) and (first, end) == pk.row_range(n, oracle_prop, i)
    for prop in (wl.GENERAL, wl.IDENTITY, wl.DIAGONAL, wl.SYMMETRIC):
        with pytest.raises(mom.MomError) as e:
            mom.mom_packed_elements(8, prop)
        assert e.value.status == mom.ERR_PROPERTY
    with pytest.raises(mom.MomError) as e:
        mom.mom_packed_row(8, wl.LOWER_TRI, 8)
    assert e.value.status == mom.ERR_INVALID_ARG
    # the input generator's packing agrees with the oracle's
    rng = np.random.default_rng(1)
    for n in (1, 5, 8, 13, 64):
        a = rng.standard_normal((n, n)).astype(np.float32)
        assert np.array_equal(wl.pack_triangle(np.tril(a), True), pk.pack(np.tril(a), pk.LOWER_TRI))
        assert np.array_equal(wl.pack_triangle(np.triu(a), False), pk.pack(np.triu(a), pk.UPPER_TRI))


def test_storage_changes_neither_the_plan_nor_its_costs():
    P = mom.STORAGE_PACKED
    for seed in range(60):
        eq = wl.random_equation(seed, max_len=6, max_dim=40)
        descs = eq.descs()
        storage = [P if d[2] in (wl.LOWER_TRI, wl.UPPER_TRI) and seed % 2 == 0 else 0 for d in descs]
        got = mom.mom_equation_plan_stored(descs, None, storage, eq.add_descs(), None, None, 0, mom.VARIANT_3XTF32)
        want = op.plan(descs, eq.add_descs())
        assert got.parenthesization() == want.paren and got.flops() == (want.mul_flops, want.add_flops)
        rd = got.result_desc()
        assert got.result_elements() == rd.rows * rd.cols
    # sizes: the packed X of L*L, and the workspace the storage layer adds where no kernel reads the container in place
    n = 200
    dense = mom.mom_equation_plan([(n, n, wl.LOWER_TRI), (n, n, wl.LOWER_TRI)], [], mom.VARIANT_FFMA)
    packed = mom.mom_equation_plan_stored([(n, n, wl.LOWER_TRI), (n, n, wl.LOWER_TRI)], None, [P, P], (), None, None, P, mom.VARIANT_FFMA)
    assert packed.result_elements() == mom.mom_packed_elements(n, wl.LOWER_TRI) == n * (n + 4) // 2
    assert packed.workspace_bytes(1) >= dense.workspace_bytes(1) + 3 * n * n * 4       # two dense copies and a dense X
    assert packed.host_staging_bytes(1) < dense.host_staging_bytes(1) + 3 * n * n * 4


def test_kernel_choice_of_the_default_variant():
    # three tensor-core kernels by size and shape: warp-level (2), one-launch tcgen05 with the split in shared memory (3),
    # plane-fed tcgen05 (1)
    G = wl.GENERAL
    kind = lambda m, k, n, t=(False, False): mom.mom_equation_plan_transposed([(k, m, G) if t[0] else (m, k, G), (n, k, G) if t[1] else (k, n, G)], t, (), None,
                                                                          mom.VARIANT_3XTF32).step(0).uses_tensor_cores
    assert [kind(n, n, n) for n in (256, 384, 448, 512, 768, 1024, 1536, 1792, 2048, 2560)] == [2, 2, 3, 3, 3, 3, 3, 3, 3, 1]
    assert kind(4096, 128, 4096) == 1                        # 2 * 10^9 multiplications, but 1024 tiles: many waves
    assert kind(2048, 512, 2048) == 3                        # 256 tiles of 128 x 128, but one wave of CTA pairs
    assert kind(900, 1200, 100) == 3 and kind(256, 2048, 64) == 2 and kind(128, 4096, 128) == 2       # small work; a result of one tile
    assert kind(512, 512, 510) == 2                        # rows TMA cannot address
    assert kind(640, 640, 640, (True, False)) == 3 and kind(640, 640, 640, (False, True)) == 3     # transposed operands are read as stored
    assert kind(642, 640, 640, (True, False)) == 2         # ... when their rows are 16-byte addressable (A stored 640 x 642)
    assert kind(1024, 1024, 1024, (True, False)) == 3 and kind(2560, 2560, 2560, (True, False)) == 1   # the plane kernel reads them through its split pass


def test_independent_subtrees_of_small_products_are_marked_to_run_side_by_side():
    G = wl.GENERAL
    five = wl.config_five_general()
    p = mom.mom_equation_plan(five.descs(), (), mom.VARIANT_3XTF32)
    assert p.parenthesization() == "((0*(1*2))*(3*4))"
    steps = p.steps()
    assert [(s.lhs, s.rhs) for s in steps] == [(1, 2), (0, 5), (3, 4), (6, 7)]
    assert p.concurrent_steps() == (2, 3, 3)               # (3*4) beside (0*(1*2)); the last product waits for both
    # the buffers of both subtrees are alive together: nothing is shared between them
    sizes = [256 * 64 * 4, 1024 * 64 * 4, 64 * 512 * 4]
    assert p.workspace_bytes() >= sum(sizes)
    # a right-nested chain has no such pair; large products are left in order (each fills the GPU by itself); nor does the FFMA variant pair
    assert mom.mom_equation_plan(wl.config_paper_chain().descs(), (), mom.VARIANT_3XTF32).concurrent_steps()[2] == -1
    big = [(512, 8192, G), (8192, 4096, G), (4096, 8192, G), (8192, 512, G)]
    p = mom.mom_equation_plan(big, (), mom.VARIANT_3XTF32)
    assert p.parenthesization() == "((0*1)*(2*3))" and p.concurrent_steps()[2] == -1
    assert mom.mom_equation_plan(five.descs(), (), mom.VARIANT_FFMA).concurrent_steps()[2] == -1
    # a pair below the root: ((0*1)*(2*3))*4
    deep = [(200, 40, G), (40, 200, G), (200, 40, G), (40, 200, G), (200, 8, G)]
    p = mom.mom_equation_plan(deep, (), mom.VARIANT_3XTF32)
    if p.parenthesization() == "(((0*1)*(2*3))*4)":
        assert p.concurrent_steps() == (1, 2, 2)
