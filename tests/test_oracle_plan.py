"""Pins for the plan oracle: what the paper and plain arithmetic fix about parenthesization.

Each test compares `oracle.plan` with something that is NOT `oracle.plan`: a value the paper
prints, hand arithmetic, a brute-force count, or the textbook matrix-chain recurrence written here.
"""
import itertools

import numpy as np
import pytest

from conftest import golden
from oracle import plan as op
from oracle.plan import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I, DIAGONAL as D, Desc
import workloads as wl


def general_chain(dims):
    return [(dims[i], dims[i + 1], G) for i in range(len(dims) - 1)]


def textbook_matrix_chain(dims):
    """Minimum scalar multiplications for general matrices with boundary dims p0..pn (classic O(n^3) DP)."""
    n = len(dims) - 1
    cost = [[0] * n for _ in range(n)]
    for length in range(2, n + 1):
        for i in range(0, n - length + 1):
            j = i + length - 1
            cost[i][j] = min(cost[i][k] + cost[k + 1][j] + dims[i] * dims[k + 1] * dims[j + 1]
                             for k in range(i, j))
    return cost[0][n - 1]


# ---------------------------------------------------------------- the paper's printed example
def test_section4_chain_matches_the_paper():
    g = golden("section4_chain.txt")
    dims = [int(x) for x in g["dims"].split()]
    p = op.plan(general_chain(dims))
    assert p.paren == g["chosen"]
    # hand arithmetic for the chosen tree: A3*A4, then A2*(..), then A1*(..)
    assert p.mults == 900 * 1200 * 100 + 1100 * 900 * 100 + 800 * 1100 * 100 == 295_000_000
    assert p.mul_flops == 590_000_000
    # the initial left-nested tree the paper starts from is worse
    left_nested = 800 * 1100 * 900 + 800 * 900 * 1200 + 800 * 1200 * 100
    assert left_nested == 1_752_000_000 > p.mults
    assert [(s.lhs, s.rhs, s.out) for s in p.steps] == [(2, 3, 4), (1, 4, 5), (0, 5, 6)]
    assert [(s.m, s.n, s.k) for s in p.steps] == [(900, 100, 1200), (1100, 100, 900), (800, 100, 1100)]


def test_listing2_product_is_typed_lower_triangular():
    g = golden("listing2_types.txt")
    n = int(g["n"])
    names = {v: k for k, v in wl.PROPERTY_NAMES.items()}
    p = op.plan([(n, n, names[g["lhs_property"]]), (n, n, names[g["rhs_property"]])])
    assert p.result_desc == Desc(n, n, names[g["result_property"]])
    assert p.paren == "(0*1)"
    # sum_{l} (#rows i >= l) * (#cols j <= l) = sum_{l=0}^{4} (5-l)(l+1) = 5+8+9+8+5
    assert p.mults == 35 and p.mul_flops == 70


# ---------------------------------------------------------------- cost model
@pytest.mark.parametrize("pa,pb", list(itertools.product([G, L, U, D], repeat=2)))
def test_closed_form_mults_equal_brute_force_count(pa, pb):
    for n in range(1, 8):
        shapes = [(n, n, n)]
        if pa == G:
            shapes.append((n + 2, n, n))
        if pb == G:
            shapes.append((n, n, n + 3))
        if pa == G and pb == G:
            shapes.append((n + 1, n + 4, n + 2))
        for (m, k, c) in shapes:
            if pa != G and m != k:
                continue
            if pb != G and k != c:
                continue
            a, b = Desc(m, k, pa), Desc(k, c, pb)
            assert op.product_mults(a, b) == op.brute_force_mults(a, b), (a, b)


def test_brute_force_count_against_dense_indicator_product():
    # the count of useful multiplications equals the sum of entries of S(A) * S(B) (0/1 matrices)
    for pa, pb in itertools.product([G, L, U, D], repeat=2):
        n = 6
        sa = np.array([[op.in_structure(pa, i, j) for j in range(n)] for i in range(n)], dtype=np.int64)
        sb = np.array([[op.in_structure(pb, i, j) for j in range(n)] for i in range(n)], dtype=np.int64)
        assert int((sa @ sb).sum()) == op.product_mults(Desc(n, n, pa), Desc(n, n, pb))


def test_structural_nonzeros():
    for prop in (G, L, U, I, D):
        for n in (1, 2, 5, 9):
            d = Desc(n, n, prop)
            assert op.structural_nonzeros(d) == op.brute_force_nonzeros(d)
    assert op.structural_nonzeros(Desc(3, 7, G)) == 21


def test_identity_costs_nothing_and_join_rules():
    assert op.product_mults(Desc(4, 4, I), Desc(4, 9, G)) == 0
    assert op.product_mults(Desc(9, 4, G), Desc(4, 4, I)) == 0
    assert op.join(L, L) == L and op.join(U, U) == U
    assert op.join(L, U) == G and op.join(U, L) == G
    assert op.join(G, L) == G and op.join(U, G) == G
    assert op.join(I, L) == L and op.join(U, I) == U and op.join(I, I) == I
    # join is associative and commutative, so a sub-chain's property does not depend on its tree
    assert op.join(D, D) == D and op.join(D, L) == L and op.join(U, D) == U and op.join(D, G) == G
    assert op.join(I, D) == D and op.join(D, I) == D
    for a, b, c in itertools.product([G, L, U, I, D], repeat=3):
        assert op.join(op.join(a, b), c) == op.join(a, op.join(b, c))
        assert op.join(a, b) == op.join(b, a)


def test_product_structure_rule_matches_boolean_products():
    # the structure of a product of 0/1 structure matrices is inside the joined property's structure,
    # and fills it completely
    n = 5
    for pa, pb in itertools.product([G, L, U, I, D], repeat=2):
        sa = np.array([[op.in_structure(pa, i, j) for j in range(n)] for i in range(n)], dtype=np.int64)
        sb = np.array([[op.in_structure(pb, i, j) for j in range(n)] for i in range(n)], dtype=np.int64)
        got = (sa @ sb) > 0
        want = np.array([[op.in_structure(op.join(pa, pb), i, j) for j in range(n)] for i in range(n)])
        assert np.array_equal(got, want), (pa, pb)


# ---------------------------------------------------------------- enumeration
def test_number_of_trees_is_catalan():
    expect = [1, 1, 2, 5, 14, 42, 132, 429]
    for r in range(1, 9):
        assert sum(1 for _ in op.all_trees(0, r - 1)) == expect[r - 1] == op.catalan(r)


def test_all_general_chains_reduce_to_the_textbook_dp():
    rng = np.random.default_rng(7)
    for _ in range(60):
        n = int(rng.integers(1, 8))
        dims = [int(x) for x in rng.integers(1, 60, size=n + 1)]
        p = op.plan(general_chain(dims))
        assert p.mults == textbook_matrix_chain(dims)
        assert sum(s.mults for s in p.steps) == p.mults
        assert len(p.steps) == n - 1


def test_chosen_tree_is_a_minimum_under_brute_force_costs():
    # independent re-evaluation: cost every tree with brute-force counts on tiny shapes
    rng = np.random.default_rng(11)
    for _ in range(25):
        n = int(rng.integers(2, 6))
        cur = int(rng.integers(1, 6))
        chain = []
        for _ in range(n):
            kind = int(rng.integers(0, 4))
            if kind == 0:
                chain.append((cur, cur, L))
            elif kind == 1:
                chain.append((cur, cur, U))
            else:
                nxt = int(rng.integers(1, 6))
                chain.append((cur, nxt, G))
                cur = nxt
        descs = [Desc(*c) for c in chain]

        def brute(tree):
            if isinstance(tree, int):
                return descs[tree], 0
            _, lt, rt = tree
            dl, cl = brute(lt)
            dr, cr = brute(rt)
            return Desc(dl.rows, dr.cols, op.join(dl.prop, dr.prop)), cl + cr + op.brute_force_mults(dl, dr)

        best = min(brute(t)[1] for t in op.all_trees(0, n - 1))
        assert op.plan(chain).mults == best


# ---------------------------------------------------------------- identity simplification
def test_identity_operands_vanish():
    p = op.plan([(64, 64, I), (64, 64, L)])
    assert (p.paren, p.mults, len(p.steps)) == ("1", 0, 0)
    assert p.result_desc == Desc(64, 64, L)
    p = op.plan([(64, 64, L), (64, 64, I)])
    assert (p.paren, p.mults, len(p.steps)) == ("0", 0, 0)
    p = op.plan([(8, 8, I), (8, 8, I), (8, 8, I)])
    assert (p.paren, p.mults, len(p.steps)) == ("I", 0, 0)
    assert p.result_desc == Desc(8, 8, I)


def test_inserting_identities_changes_neither_cost_nor_tree_shape():
    base = [(30, 30, L), (30, 12, G), (12, 12, U), (12, 40, G)]
    p0 = op.plan(base)
    for pos in range(len(base) + 1):
        dim = base[pos][0] if pos < len(base) else base[-1][1]
        chain = base[:pos] + [(dim, dim, I)] + base[pos:]
        p1 = op.plan(chain)
        assert p1.mults == p0.mults
        relabel = p0.paren
        # shift original indices >= pos by one
        out, num = "", ""
        for ch in relabel + " ":
            if ch.isdigit():
                num += ch
            else:
                if num:
                    v = int(num)
                    out += str(v + 1 if v >= pos else v)
                    num = ""
                out += ch
        assert p1.paren == out.strip()


# ---------------------------------------------------------------- ties and the benchmark's plans
def test_tie_break_prefers_smallest_preorder_split_list():
    n = 8192
    chain = [(n, n, L), (n, n, G), (n, n, U), (n, n, G)]
    tri_gen = n * (n * (n + 1) // 2)
    gen_gen = n * n * n
    p = op.plan(chain)
    assert p.mults == 2 * tri_gen + gen_gen == 1_099_578_736_640
    assert p.paren == "(0*(1*(2*3)))"      # every one of the 5 trees costs the same
    # a three-way all-equal general chain: split after the first operand wins
    assert op.plan([(4, 4, G)] * 3).paren == "(0*(1*2))"


def test_benchmark_configuration_plans():
    p = op.plan(wl.config_tiny().descs())
    # (L*A)*B : 32*64*65/2 + 64*32*48 ;  L*(A*B) : 64*32*48 + 48*64*65/2
    assert (p.paren, p.mults) == ("((0*1)*2)", 66_560 + 98_304)
    assert 98_304 + 48 * 64 * 65 // 2 == 198_144 > p.mults

    p = op.plan(wl.config_five_general().descs())
    # (M2*M3): 256*2048*64 ; M1*(..): 1024*256*64 ; (M4*M5): 64*1024*512 ; product: 1024*64*512
    assert p.paren == "((0*(1*2))*(3*4))"
    assert p.mults == 256 * 2048 * 64 + 1024 * 256 * 64 + 64 * 1024 * 512 + 1024 * 64 * 512 == 117_440_512

    eq = wl.config_property_heavy()
    p = op.plan(eq.descs(), eq.add_descs())
    n = 4096
    assert p.paren == "(0*(1*3))" and p.kept == (0, 1, 3)
    assert p.mults == 2 * n * (n * (n + 1) // 2) == 68_736_253_952
    assert p.add_flops == n * n
    assert p.result_desc == Desc(n, n, G)
    # the alternative (L*U)*B: sum of squares for L*U, then a full general product
    assert n * (n + 1) * (2 * n + 1) // 6 + n ** 3 == 91_634_358_272 > p.mults

    eq = wl.config_batched()
    p = op.plan(eq.descs(), eq.add_descs())
    assert (p.paren, p.mults) == ("(0*(1*2))", 64 * 64 * 16 + 16 * 64 * 65 // 2)
    assert p.mults == 98_816 and p.add_flops == 1024


# ---------------------------------------------------------------- Add terms and errors
def test_sum_property():
    assert op.plan([(4, 4, L), (4, 4, L)], [(4, 4, L)]).result_desc.prop == L
    assert op.plan([(4, 4, L), (4, 4, L)], [(4, 4, U)]).result_desc.prop == G
    assert op.plan([(4, 4, L), (4, 4, L)], [(4, 4, I)]).result_desc.prop == L
    assert op.plan([(4, 4, I)], [(4, 4, I)]).result_desc.prop == D       # I + I = 2I: a diagonal matrix
    assert op.plan([(4, 4, D)], [(4, 4, I)]).result_desc.prop == D
    assert op.plan([(4, 4, D)], [(4, 4, L)]).result_desc.prop == L
    assert op.plan([(4, 4, D), (4, 4, U)], [(4, 4, D)]).result_desc.prop == U
    assert op.plan([(4, 4, L)], [(4, 4, D), (4, 4, U)]).result_desc.prop == G
    assert op.plan([(4, 4, D)], []).result_desc.prop == D
    assert op.plan([(4, 4, U)], [(4, 4, D)]).add_flops == 4
    assert op.plan([(4, 4, I)], [(4, 4, U), (4, 4, I)]).result_desc.prop == U
    assert op.plan([(4, 4, I)], []).result_desc.prop == I
    assert op.plan([(4, 4, U)], [(4, 4, G)]).add_flops == 16
    assert op.plan([(4, 4, U)], [(4, 4, L), (4, 4, I)]).add_flops == 10 + 4


@pytest.mark.parametrize("chain,add,code", [
    ([], [], "invalid_arg"),
    ([(0, 3, G)], [], "invalid_arg"),
    ([(3, 4, L)], [], "property"),
    ([(3, 4, I)], [], "property"),
    ([(3, 4, D)], [], "property"),
    ([(3, 3, 10)], [], "property"),
    ([(3, 4, 6)], [], "property"),
    ([(3, 4, 9)], [], "property"),
    ([(3, 4, G), (5, 3, G)], [], "shape_mismatch"),
    ([(3, 4, G)], [(3, 5, G)], "shape_mismatch"),
])
def test_invalid_equations_are_rejected(chain, add, code):
    with pytest.raises(op.OracleError) as e:
        op.plan(chain, add)
    assert e.value.code == code


# ---------------------------------------------------------------- Transpose (paper Table 1; Section 2 inference rule)
def test_transposed_operands_take_the_transposed_type():
    # the rule the paper prints: lowerTriangular(A) -> upperTriangular(A^T)
    assert op.transpose_desc(Desc(5, 5, L)) == Desc(5, 5, U)
    assert op.transpose_desc(Desc(5, 5, U)) == Desc(5, 5, L)
    assert op.transpose_desc(Desc(3, 7, G)) == Desc(7, 3, G)
    assert op.transpose_desc(Desc(4, 4, I)) == Desc(4, 4, I)
    # L^T * L^T is upperTri; L^T * L is general; structure of S(A^T) is the mirrored structure
    assert op.plan([(6, 6, L), (6, 6, L)], chain_transposed=[True, True]).result_desc == Desc(6, 6, U)
    assert op.plan([(6, 6, L), (6, 6, L)], chain_transposed=[True, False]).result_desc == Desc(6, 6, G)
    for prop in (G, L, U, I):
        tp = op.transpose_desc(Desc(5, 5, prop)).prop
        for i in range(5):
            for j in range(5):
                assert op.in_structure(tp, i, j) == op.in_structure(prop, j, i)


def test_transposes_change_shapes_costs_and_the_string():
    # A (7 x 30) stored, used as A^T (30 x 7): the chain A^T * B * C with B 7 x 40, C 40 x 3
    p = op.plan([(7, 30, G), (7, 40, G), (40, 3, G)], chain_transposed=[True, False, False])
    assert p.paren == "(0^T*(1*2))"
    assert p.mults == 7 * 40 * 3 + 30 * 7 * 3
    assert p.result_desc == Desc(30, 3, G)
    # a plan with transposes equals the plan of the explicitly transposed descriptors (up to the printed marks)
    q = op.plan([(30, 7, G), (7, 40, G), (40, 3, G)])
    assert q.mults == p.mults and q.paren == p.paren.replace("^T", "")
    with pytest.raises(op.OracleError):
        op.plan([(7, 30, G), (7, 40, G)])                        # without the transpose the shapes do not chain
    # Add terms may be transposed too
    p = op.plan([(4, 9, G)], [(9, 4, G)], add_transposed=[True])
    assert p.result_desc == Desc(4, 9, G) and p.add_flops == 36
    assert op.plan([(5, 5, L)], [(5, 5, U)], add_transposed=[True]).result_desc.prop == L
