"""GPU parity: every product kind, epilogue and plan shape against the fp64 oracle, through the C ABI."""
import itertools

import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2208_10391_b200 as mom
import workloads as wl
from workloads import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I, Operand, Equation
from gpu_util import run_equation, check_against_oracle, run_expression, check_expression_against_oracle, stratified_rows, TOL

pytestmark = pytest.mark.gpu

VARIANTS = [mom.VARIANT_FFMA, mom.VARIANT_3XTF32_FORCE, mom.VARIANT_3XTF32_WARP, mom.VARIANT_3XTF32_INLINE]
VNAME = {mom.VARIANT_FFMA: "ffma", mom.VARIANT_3XTF32_FORCE: "tc", mom.VARIANT_3XTF32: "auto", mom.VARIANT_3XTF32_WARP: "warp",
         mom.VARIANT_3XTF32_INLINE: "inline"}


def both(eq, variant, **kw):
    x, plan, (chain, add) = run_equation(eq, variant)
    return check_against_oracle(eq, x, plan, chain, add, **kw), x, plan


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("pa,pb", list(itertools.product([G, L, U], repeat=2)))
@pytest.mark.parametrize("n", [1, 5, 64, 200, 332])
def test_every_property_pair(pa, pb, n, variant):
    # square n x n operands; 200 and 332 are multiples of 4 that leave ragged tiles in every tile size used
    eq = Equation(f"pair_{pa}{pb}_{n}", 100 + n, (Operand(n, n, pa, "normal" if pa == G else "uniform"),
                                                  Operand(n, n, pb, "normal" if pb == G else "uniform")))
    both(eq, variant)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("m,k,n", [(64, 32, 48), (300, 520, 260), (129, 257, 65), (8, 2048, 16), (1000, 4, 12)])
def test_rectangular_general_products(m, k, n, variant):
    eq = Equation(f"gg_{m}x{k}x{n}", 7, (Operand(m, k, G, "normal"), Operand(k, n, G, "normal")))
    both(eq, variant)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("pt", [L, U])
@pytest.mark.parametrize("side", ["left", "right"])
def test_triangular_times_rectangular(pt, side, variant):
    if side == "left":
        eq = Equation("tg", 8, (Operand(392, 392, pt), Operand(392, 136, G, "normal")))
    else:
        eq = Equation("gt", 9, (Operand(136, 392, G, "normal"), Operand(392, 392, pt)))
    both(eq, variant)


@pytest.mark.parametrize("pa,pb", [(G, G), (L, G), (U, G), (G, L), (G, U), (L, L), (U, L)])
def test_split_k_products(pa, pb):
    # few output tiles and a long contraction: the tensor-core kernel runs k-slices on different CTAs and a
    # small kernel adds the partial sums (and applies the Add terms and the structure mask)
    n = 640
    shapes = {(G, G): ((256, 2048), (2048, 64)), (L, G): ((n, n), (n, 136)), (U, G): ((n, n), (n, 136)),
              (G, L): ((72, n), (n, n)), (G, U): ((72, n), (n, n)), (L, L): ((n, n), (n, n)), (U, L): ((n, n), (n, n))}
    (am, ak), (bk, bn) = shapes[(pa, pb)]
    add = (Operand(am, bn, G, "normal"), Operand(am, bn, I)) if am == bn else (Operand(am, bn, G, "normal"),)
    eq = Equation(f"splitk_{pa}{pb}", 60, (Operand(am, ak, pa, "normal" if pa == G else "uniform"),
                                           Operand(bk, bn, pb, "normal" if pb == G else "uniform")), add)
    both(eq, mom.VARIANT_3XTF32_FORCE)
    both(eq, mom.VARIANT_3XTF32_WARP)       # the warp-level kernel splits the contraction over a thread-block cluster
    # the same product as the inner step of a chain whose next step is a tensor-core step too
    eq = Equation(f"splitk_chain_{pa}{pb}", 61, (Operand(200, am, G, "normal"), Operand(am, ak, pa, "normal" if pa == G else "uniform"),
                                                 Operand(bk, bn, pb, "normal" if pb == G else "uniform")))
    both(eq, mom.VARIANT_3XTF32_FORCE)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_listing2_exact_values(variant):
    # paper Listing 2: 5x5 lowerTri filled with ones times itself; every value is a small integer
    eq = wl.config_listing2()
    _, x, plan = both(eq, variant)
    want = np.array([[max(i - j + 1, 0) for j in range(5)] for i in range(5)], dtype=np.float32)
    assert np.array_equal(x, want)
    assert plan.result_desc().property == L


@pytest.mark.parametrize("variant", VARIANTS + [mom.VARIANT_3XTF32], ids=VNAME.get)
def test_config_tiny_and_identity_checks(variant):
    both(wl.config_tiny(), variant)
    for eq in (wl.config_tiny_identity_left(), wl.config_tiny_identity_right()):
        x, plan, (chain, add) = run_equation(eq, variant)
        assert plan.num_steps() == 0 and plan.flops() == (0, 0)
        src = [c for c in chain if c is not None][0]
        assert np.array_equal(x, src)          # A*I = A and I*A = A, bit for bit


@pytest.mark.parametrize("variant", VARIANTS + [mom.VARIANT_3XTF32], ids=VNAME.get)
def test_config_five_general(variant):
    both(wl.config_five_general(), variant)


@pytest.mark.parametrize("variant", VARIANTS + [mom.VARIANT_3XTF32], ids=VNAME.get)
def test_paper_section4_chain(variant):
    both(wl.config_paper_chain(), variant)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("n", [256, 520])
def test_config_property_heavy_small(n, variant):
    both(wl.config_property_heavy(n=n), variant)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("n", [384, 776])
def test_config_large_square_small(n, variant):
    both(wl.config_large_square(n=n), variant)


INLINE_SHAPES = [
    # (m, k, n, left property, right property, Add terms): the one-launch tcgen05 kernel that splits in shared memory
    (128, 32, 64, G, G, 0), (100, 36, 100, G, G, 1), (900, 1200, 100, G, G, 0), (256, 2048, 64, G, G, 2),      # k split over a cluster
    (64, 1024, 512, G, G, 0), (1024, 64, 512, G, G, 1), (1000, 260, 76, G, G, 0), (1, 4, 4, G, G, 0),
    (520, 520, 520, L, G, 1), (520, 520, 136, U, G, 0), (300, 392, 392, G, L, 0), (300, 392, 392, G, U, 2),
    (392, 392, 392, L, L, 1), (392, 392, 392, U, U, 0), (392, 392, 392, L, U, 0), (392, 392, 392, U, L, 1),
    (1024, 1024, 1024, G, G, 0), (1536, 1152, 1280, G, G, 1),
    (128, 4096, 128, G, G, 1), (100, 4100, 60, G, G, 0),            # one or two tiles, long contraction: clusters of 16 CTAs
    # more than one wave of 128 x 128 tiles but at most one wave of 256 x 256 tiles: the launcher takes the CTA-pair form
    # (A halves in both CTAs' tensor memory, each CTA half of B, the leader issues cta_group::2 MMAs)
    (2048, 64, 2048, G, G, 1), (1800, 100, 1900, G, G, 0), (1536, 1536, 2048, L, G, 1), (1536, 2048, 2048, G, U, 0),
    (2048, 2048, 2048, L, L, 1),
]


@pytest.mark.parametrize("m,k,n", [(256, 2048, 64), (100, 4099, 44), (64, 8192, 32), (130, 2052, 70)])
def test_warp_level_kernel_with_sixteen_k_slices(m, k, n):
    # very few output tiles and a contraction of 2048 or more: the warp-level kernel splits k over clusters of 16 CTAs (the
    # non-portable cluster size) that add their partial tiles through distributed shared memory; ragged m, n and k
    eq = Equation(f"warp16_{m}x{k}x{n}", 77, (Operand(m, k, G, "normal", 1.0 / np.sqrt(k)), Operand(k, n, G, "normal")),
                  (Operand(m, n, G, "normal"),))
    x, plan, (chain, terms_h) = run_equation(eq, mom.VARIANT_3XTF32_WARP)
    assert plan.step(0).uses_tensor_cores == 2 and plan.last_launch_count() == 1
    check_against_oracle(eq, x, plan, chain, terms_h)


@pytest.mark.parametrize("m,k,n,pa,pb,terms", INLINE_SHAPES)
def test_inline_split_tensor_core_kernel(m, k, n, pa, pb, terms):
    # every launch shape of the kernel: 64- and 128-column tiles, 1 to 8 k-slices per tile (cluster), CTA pairs, ragged edges in
    # m, n and k, triangular factors (structural k-ranges, masked triangular results), fused Add terms incl. Identity
    dist = lambda p: "uniform" if p != G else "normal"
    add = [Operand(m, n, G, "normal")] * min(terms, 1) + ([Operand(m, n, I)] if terms == 2 and m == n else
                                                          [Operand(m, n, G, "normal")] if terms == 2 else [])
    eq = Equation(f"inline_{m}x{k}x{n}_{pa}{pb}", 75, (Operand(m, k, pa, dist(pa), 1.0 / np.sqrt(k)), Operand(k, n, pb, dist(pb))), tuple(add))
    x, plan, (chain, terms_h) = run_equation(eq, mom.VARIANT_3XTF32_INLINE)
    assert plan.step(0).uses_tensor_cores == 3 and plan.last_launch_count() == 1
    check_against_oracle(eq, x, plan, chain, terms_h)


def test_subtrees_side_by_side_on_two_streams():
    # chains whose chosen tree multiplies two products: the right subtree runs on the plan's side stream beside the left one.
    # Same values as the plan computed in order (the forced variants keep the plain order), within the bound of the oracle,
    # also when the same plan is executed again and again on the same workspace.
    rng = np.random.default_rng(11)
    found = 0
    for trial in range(60):
        n = int(rng.integers(4, 7))
        dims = [int(rng.choice([8, 24, 64, 136, 264, 520])) for _ in range(n + 1)]
        props = [G] * n
        eq = Equation(f"side_{trial}", 500 + trial, tuple(Operand(dims[i], dims[i + 1], props[i], "normal", 1.0 / np.sqrt(dims[i + 1])) for i in range(n)))
        plan = mom.mom_equation_plan(eq.descs(), (), mom.VARIANT_3XTF32)
        if plan.concurrent_steps()[2] < 0 or plan.workspace_bytes() == 0:
            continue
        found += 1
        chain, add = wl.generate(eq)
        x, plan, _ = run_equation(eq, mom.VARIANT_3XTF32, chain, add)
        check_against_oracle(eq, x, plan, chain, add)
        dchain = [torch.from_numpy(a).cuda() for a in chain]
        outs = torch.full((20,) + x.shape, float("nan"), dtype=torch.float32, device="cuda")
        wsb = plan.workspace_bytes(1)
        ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
        for i in range(20):
            plan.execute([t.data_ptr() for t in dchain], [], outs[i].data_ptr(), ws.data_ptr(), wsb, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        o = outs.cpu().numpy()
        assert all(np.array_equal(o[i], x) for i in range(20))
    assert found >= 10


@pytest.mark.parametrize("case", ["LG", "GU_plus_C", "chain"])
def test_pair_kernel_ragged_shapes(case):
    # big enough for the CTA-pair tensor-core kernel (256-row tiles), with edges that are not multiples of the tile
    m, k, n = 3336, 3064, 3592
    if case == "LG":
        eq = Equation("pair_LG", 70, (Operand(m, m, L), Operand(m, n, G, "normal", 0.02)))
    elif case == "GU_plus_C":
        eq = Equation("pair_GU", 71, (Operand(m, n, G, "normal", 0.02), Operand(n, n, U)), (Operand(m, n, G, "normal"),))
    else:
        eq = Equation("pair_chain", 72, (Operand(m, m, U), Operand(m, k, G, "normal", 0.02), Operand(k, k, L), Operand(k, n, G, "normal", 0.02)))
    x, plan, (chain, add) = run_equation(eq, mom.VARIANT_3XTF32)
    assert all(s.uses_tensor_cores == 1 for s in plan.steps())
    # one row in every 32-row slab: every pair-tile row and every epilogue warp's slab is compared
    check_against_oracle(eq, x, plan, chain, add, rows=stratified_rows(m, 3, extra=[0, 127, 128, 255, 256, m - 1]))


@pytest.mark.parametrize("pa,pb", list(itertools.product([G, L, U], repeat=2)))
def test_pair_kernel_whole_output(pa, pb):
    # the smallest products the CTA-pair kernel takes (48 pair tiles of 256 x 256), every property pair, compared with
    # the oracle on the WHOLE output: every tile, every k-range of the tile table, every epilogue slab
    m, n = 2048, 1536
    if pa != G and pb != G:
        m = n = 2048                                      # both factors are square
    k = m if pa != G else n if pb != G else 1152
    op = lambda r, c, p: Operand(r, c, p, "normal", 0.05) if p == G else Operand(r, c, p)
    eq = Equation(f"pair_full_{pa}{pb}", 73, (op(m, k, pa), op(k, n, pb)), (Operand(m, n, G, "normal"),) if pa == G else ())
    x, plan, (chain, add) = run_equation(eq, mom.VARIANT_3XTF32_FORCE)
    assert plan.step(0).uses_tensor_cores == 1 and (m // 256) * (n // 256) >= 48
    check_against_oracle(eq, x, plan, chain, add)


@pytest.mark.parametrize("variant", [mom.VARIANT_3XTF32, mom.VARIANT_FFMA], ids=VNAME.get)
def test_config_property_heavy_full_size_sampled_rows(variant):
    eq = wl.config_property_heavy()
    x, plan, (chain, add) = run_equation(eq, variant)
    check_against_oracle(eq, x, plan, chain, add, rows=stratified_rows(4096, 0, extra=[0, 127, 128, 4095]))


@pytest.mark.parametrize("variant", [mom.VARIANT_3XTF32], ids=VNAME.get)
def test_config_large_square_full_size_sampled_rows(variant):
    eq = wl.config_large_square()
    x, plan, (chain, add) = run_equation(eq, variant)
    # 256 rows, one in every 32-row slab: all 32 pair-tile rows and all 256 epilogue-warp slabs of X
    check_against_oracle(eq, x, plan, chain, add, rows=stratified_rows(8192, 1, extra=[0, 127, 128, 8191]))


@pytest.mark.parametrize("variant", VARIANTS + [mom.VARIANT_3XTF32], ids=VNAME.get)
def test_config_batched(variant):
    eq = wl.config_batched(batch=37)
    both(eq, variant)
    eq = wl.config_batched()                      # the full 4096 instances, a sample of them checked
    x, plan, (chain, add) = run_equation(eq, variant)
    check_against_oracle(eq, x, plan, chain, add, instances=[0, 1, 63, 64, 2047, 4095])


@pytest.mark.parametrize("variant", [mom.VARIANT_FFMA, mom.VARIANT_3XTF32], ids=VNAME.get)
@pytest.mark.parametrize("n", [1, 5, 8, 12, 16, 24, 27, 32])
def test_batched_small_chains(n, variant):
    # plans of the form M1*(M2*(M3*B)) with a narrow B, batched: the fused shared-memory kernel
    for chain, add in [
        ((Operand(64, 64, L), Operand(64, 64, G), Operand(64, n, G)), (Operand(64, n, G),)),
        ((Operand(40, 72, G, "normal"), Operand(72, 72, U), Operand(72, 52, G), Operand(52, n, G)), ()),
        ((Operand(36, 36, U), Operand(36, n, G)), (Operand(36, n, G), Operand(36, n, G))),
        ((Operand(100, 20, G), Operand(20, n, G)), ()),
        ((Operand(28, 26, G), Operand(26, 26, L), Operand(26, 4 * ((n + 3) // 4), G)), ()),      # k = 26: not a multiple of 4
    ]:
        eq = Equation(f"narrow_n{n}", 40 + n, chain, add, batch=45)
        plan = mom.mom_equation_plan(eq.descs(), eq.add_descs(), variant)
        both(eq, variant)


BATCHED_CHAINS = {
    # name: (chain of (rows, cols, property), Add terms, instances): right-nested plans with a right end of 8 or 16 columns
    "LAB_plus_C": (((64, 64, L), (64, 64, G), (64, 16, G)), ((64, 16, G),), 300),
    "UAB": (((64, 64, U), (64, 64, G), (64, 16, G)), (), 257),
    "one_product_n8": (((48, 32, G), (32, 8, G)), ((48, 8, G), (48, 8, G)), 513),
    "four_products": (((32, 64, G), (64, 64, L), (64, 48, G), (48, 48, U), (48, 16, G)), ((32, 16, G),), 260),
    "square_result": (((16, 16, L), (16, 16, L)), ((16, 16, I), (16, 16, L)), 1000),
    "upper_right_end": (((64, 16, G), (16, 16, U), (16, 16, U)), (), 256),
    "mixed_heights": (((16, 48, G), (48, 64, G), (64, 64, L), (64, 8, G)), ((16, 8, G), (16, 8, G), (16, 8, G)), 333),
}


@pytest.mark.parametrize("variant", [mom.VARIANT_3XTF32], ids=VNAME.get)
@pytest.mark.parametrize("name", sorted(BATCHED_CHAINS))
def test_batched_right_nested_chains(name, variant):
    # many instances of M_S*(...(M_1*B)) with whole 16-row blocks: the kernel that gives two warps to each instance and
    # streams the factors through registers; every instance compared with the oracle
    chain, add, batch = BATCHED_CHAINS[name]
    dist = lambda p: "uniform" if p != G else "normal"
    eq = Equation(f"batched_chain_{name}", 50, tuple(Operand(r, c, p, dist(p)) for r, c, p in chain),
                  tuple(Operand(r, c, p, dist(p)) for r, c, p in add), batch=batch)
    _, x, plan = both(eq, variant)
    assert plan.last_launch_count() == 1
    # fewer instances than the kernel is worth: the one-CTA-per-instance kernel gives the same values within the bound
    small = Equation(f"batched_chain_{name}_few", 50, eq.chain, eq.add, batch=7)
    both(small, variant)


def test_batched_chain_with_padding_and_poisoned_gaps():
    # instance strides larger than the matrices, NaNs in the gaps: nothing outside an instance is read or written
    eq = wl.config_batched(batch=384)
    chain, add = wl.generate(eq)
    plan = mom.mom_equation_plan(eq.descs(), eq.add_descs(), mom.VARIANT_3XTF32)
    pad = 12
    def padded(a):
        flat = np.full((a.shape[0], a[0].size + pad), np.nan, dtype=np.float32)
        flat[:, :a[0].size] = a.reshape(a.shape[0], -1)
        return torch.from_numpy(flat).cuda()
    dc, da = [padded(a) for a in chain], [padded(a) for a in add]
    out = torch.full((384, 64 * 16 + pad), float("nan"), dtype=torch.float32, device="cuda")
    plan.execute_batched([t.data_ptr() for t in dc], [t.shape[1] for t in dc], [t.data_ptr() for t in da],
                         [t.shape[1] for t in da], out.data_ptr(), out.shape[1], 384, None, 0,
                         torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    o = out.cpu().numpy()
    assert np.isnan(o[:, 64 * 16:]).all()
    check_against_oracle(eq, o[:, :64 * 16].reshape(384, 64, 16), plan, chain, add)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_batched_with_padding_between_instances(variant):
    eq = wl.config_batched(batch=5)
    chain, add = wl.generate(eq)
    plan = mom.mom_equation_plan(eq.descs(), eq.add_descs(), variant)
    pad = 8
    def padded(a):
        flat = np.full((a.shape[0], a[0].size + pad), np.nan, dtype=np.float32)
        flat[:, :a[0].size] = a.reshape(a.shape[0], -1)
        return torch.from_numpy(flat).cuda()
    dc, da = [padded(a) for a in chain], [padded(a) for a in add]
    out = torch.full((5, 64 * 16 + pad), float("nan"), dtype=torch.float32, device="cuda")
    wsb = plan.workspace_bytes(5)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")
    plan.execute_batched([t.data_ptr() for t in dc], [t.shape[1] for t in dc], [t.data_ptr() for t in da],
                         [t.shape[1] for t in da], out.data_ptr(), out.shape[1], 5, ws.data_ptr() if wsb else None, wsb,
                         torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    o = out.cpu().numpy()
    assert np.isnan(o[:, 64 * 16:]).all()          # padding untouched
    x = o[:, :64 * 16].reshape(5, 64, 16)
    check_against_oracle(eq, x, plan, chain, add)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_add_terms_and_result_structure(variant):
    n = 72
    # L*L + L stays lowerTri (upper part +0.0f); L*L + U becomes general; Identity term adds ones on the diagonal
    for terms in ([Operand(n, n, L)], [Operand(n, n, U)], [Operand(n, n, I)], [Operand(n, n, L), Operand(n, n, I), Operand(n, n, L)]):
        eq = Equation("ll_plus", 21, (Operand(n, n, L), Operand(n, n, L)), tuple(terms))
        both(eq, variant)
    # more Add terms than one launch fuses
    eq = Equation("many_terms", 22, (Operand(40, 24, G), Operand(24, 56, G)), tuple(Operand(40, 56, G, "normal") for _ in range(11)))
    both(eq, variant)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_zero_step_plans(variant):
    n = 33
    for chain, add in [((Operand(n, n, I),), ()), ((Operand(n, n, I), Operand(n, n, I)), (Operand(n, n, U),)),
                       ((Operand(n, n, I), Operand(n, n, U), Operand(n, n, I)), (Operand(n, n, U), Operand(n, n, I))),
                       ((Operand(n, 2 * n, G),), (Operand(n, 2 * n, G),)),
                       ((Operand(n, n, L),), tuple(Operand(n, n, L) for _ in range(10)))]:
        eq = Equation("zero_step", 23, chain, add)
        both(eq, variant)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_random_equations(variant):
    for seed in range(40):
        eq = wl.random_equation(1000 + seed, max_len=5, max_dim=40, dim_multiple=4 if seed % 2 else 1)
        both(eq, variant)


def test_host_entry_point_uploads_large_triangles_by_blocks():
    # triangular operands of 1024 rows or more cross the bus only up to (from) their diagonal blocks of 256 rows;
    # the device copy is completed with zeros, so the result is the device entry point's, bit for bit
    n = 1288                                 # not a multiple of the block
    eq = Equation("host_tri", 90, (Operand(n, n, L), Operand(n, n, G, "normal", 0.03), Operand(n, n, U)), (Operand(n, n, G, "normal"),))
    chain, add = wl.generate(eq)
    xd, plan, _ = run_equation(eq, mom.VARIANT_3XTF32, chain, add, via="device")
    xh, _, _ = run_equation(eq, mom.VARIANT_3XTF32, chain, add, via="host")
    assert np.array_equal(xd, xh)
    full = 4 * n * n * 4
    blocks = [(r0, min(n, r0 + 256)) for r0 in range(0, n, 256)]
    lower = sum((r1 - r0) * r1 for r0, r1 in blocks) * 4
    upper = sum((r1 - r0) * (n - r0) for r0, r1 in blocks) * 4
    assert plan.host_upload_bytes(1) == full - 2 * n * n * 4 + lower + upper < 0.85 * full
    # a stale staging area must not leak into the zero-filled part: run once more after poisoning is done by run_equation
    xh2, _, _ = run_equation(eq, mom.VARIANT_FFMA, chain, add, via="host")
    xd2, _, _ = run_equation(eq, mom.VARIANT_FFMA, chain, add, via="device")
    assert np.array_equal(xd2, xh2)


def test_host_entry_point_copies_the_first_rows_back_early():
    # from 2048 rows on, a plane-kernel product that writes X runs as two launches in the host entry point (rows up to a
    # multiple of 256 near 40 % first) and the first rows travel back during the second launch; same bits as one launch
    for n, add in ((2312, ()), (2304, (Operand(2304, 2304, G, "normal"),))):
        eq = Equation(f"host_parts_{n}", 91, (Operand(n, n, L), Operand(n, n, G, "normal", 0.02)), add)
        chain, terms = wl.generate(eq)
        xd, plan, _ = run_equation(eq, mom.VARIANT_3XTF32, chain, terms, via="device")
        xh, plan_h, _ = run_equation(eq, mom.VARIANT_3XTF32, chain, terms, via="host")
        assert np.array_equal(xd, xh)
        assert plan_h.last_launch_count() == plan.last_launch_count() + 1
        check_against_oracle(eq, xh, plan_h, chain, terms, rows=stratified_rows(n, 8))


def test_host_entry_point_starts_on_the_first_rows_of_a_left_operand_still_on_its_way():
    # L*A*U*B (the benchmark's shape): the product A*(U*B) lies inside the plan and reads the stored general A as its
    # left factor; in the host entry point A travels in two pieces and the product runs as two launches, each
    # splitting its own rows of A (one launch and one split pass more), then the product that writes X as two
    # launches as well.  Same bits as the device entry point's single launches.
    for n in (2312, 2048):
        eq = wl.config_large_square(n=n)
        chain, terms = wl.generate(eq)
        xd, plan, _ = run_equation(eq, mom.VARIANT_3XTF32, chain, terms, via="device")
        xh, plan_h, _ = run_equation(eq, mom.VARIANT_3XTF32, chain, terms, via="host")
        assert plan.parenthesization() == "(0*(1*(2*3)))"
        assert np.array_equal(xd, xh)
        assert plan_h.last_launch_count() == plan.last_launch_count() + 3
        xh2, _, _ = run_equation(eq, mom.VARIANT_3XTF32, chain, terms, via="host")       # events and pieces are reusable
        assert np.array_equal(xd, xh2)
        check_against_oracle(eq, xh, plan_h, chain, terms, rows=stratified_rows(n, 9))
    # two chains write X one after the other: the first one's rows are not final when its product ends, so nothing is
    # copied back early; the stored A is the left factor of both roots: A*(U*B) + A*L
    n = 2048
    g = Operand(n, n, G, "normal", 0.02)
    ex = wl.Expression("two_uses", 92, (g, Operand(n, n, U), g, Operand(n, n, L)), ("add", [("mul", [0, 1, 2]), ("mul", [0, 3])]))
    xd, plan_d, arrays = run_expression(ex, mom.VARIANT_3XTF32, via="device")
    xh, plan_h, _ = run_expression(ex, mom.VARIANT_3XTF32, via="host")
    assert np.array_equal(xd, xh) and plan_h.last_launch_count() == plan_d.last_launch_count()
    check_expression_against_oracle(ex, xh, plan_h, arrays, sample_rows=stratified_rows(n, 10))


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_host_entry_point_matches_device_entry_point(variant):
    for eq in (wl.config_tiny(), wl.config_batched(batch=9), wl.config_property_heavy(n=264)):
        chain, add = wl.generate(eq)
        xd, plan, _ = run_equation(eq, variant, chain, add, via="device")
        xh, _, _ = run_equation(eq, variant, chain, add, via="host")
        assert np.array_equal(xd, xh)
        check_against_oracle(eq, xh, plan, chain, add)


def test_argument_errors_are_reported_before_any_launch():
    # large enough not to run as one fused shared-memory kernel, so that it needs a workspace
    eq = Equation("errors", 5, (Operand(200, 200, L), Operand(200, 200, G), Operand(200, 48, G)))
    chain, _ = wl.generate(eq)
    plan = mom.mom_equation_plan(eq.descs(), (), mom.VARIANT_FFMA)
    assert plan.workspace_bytes() > 0
    d = [torch.from_numpy(a).cuda() for a in chain]
    out = torch.zeros(200 * 48 + 4, dtype=torch.float32, device="cuda")
    ws = torch.empty(plan.workspace_bytes(), dtype=torch.uint8, device="cuda")
    ptrs = [t.data_ptr() for t in d]
    def status(**kw):
        args = dict(chain=ptrs, out=out.data_ptr(), ws=ws.data_ptr(), wsb=plan.workspace_bytes())
        args.update(kw)
        try:
            plan.execute(args["chain"], [], args["out"], args["ws"], args["wsb"], 0)
        except mom.MomError as e:
            return e.status
        return mom.OK
    assert status(chain=[ptrs[0], None, ptrs[2]]) == mom.ERR_INVALID_ARG
    assert status(chain=[ptrs[0] + 4, ptrs[1], ptrs[2]]) == mom.ERR_ALIGNMENT
    assert status(out=out.data_ptr() + 4) == mom.ERR_ALIGNMENT
    assert status(wsb=plan.workspace_bytes() - 1) == mom.ERR_WORKSPACE_TOO_SMALL
    assert status(ws=None) == mom.ERR_WORKSPACE_TOO_SMALL
    assert status() == mom.OK
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)


# ---------------------------------------------------------------- Transpose (paper Table 1; Section 2 inference rule)
TRANSPOSE_CASES = {
    "At_B": (((200, 136, G), (200, 264, G)), (True, False), (), ()),
    "A_Bt": (((136, 200, G), (264, 200, G)), (False, True), (), ()),
    "At_Bt_plus_Ct": (((200, 136, G), (264, 200, G)), (True, True), ((264, 136, G),), (True,)),
    "Lt_G": (((328, 328, L), (328, 72, G)), (True, False), (), ()),
    "G_Ut": (((72, 328, G), (328, 328, U)), (False, True), (), ()),
    "Lt_L": (((264, 264, L), (264, 264, L)), (True, False), (), ()),
    "Lt_Lt_plus_Ut": (((264, 264, L), (264, 264, L)), (True, True), ((264, 264, L),), (True,)),
    "chain": (((96, 200, G), (96, 96, U), (328, 96, G), (328, 40, G)), (True, True, True, False), ((200, 40, G), (40, 200, G)), (False, True)),
    "zero_step": (((56, 120, G),), (True,), ((56, 120, G), (120, 56, G)), (True, False)),
    "zero_step_Lt": (((64, 64, L),), (True,), ((64, 64, I),), (False,)),
    "tiny_fused": (((64, 64, L), (32, 64, G), (48, 32, G)), (True, True, True), ((64, 48, G),), (False,)),
    "odd_sizes": (((33, 21, G), (33, 33, U), (33, 18, G)), (True, True, False), ((18, 21, G),), (True,)),
}


@pytest.mark.parametrize("variant", VARIANTS + [mom.VARIANT_3XTF32], ids=VNAME.get)
@pytest.mark.parametrize("name", sorted(TRANSPOSE_CASES))
def test_transposed_operands(name, variant):
    chain, ct, add, at = TRANSPOSE_CASES[name]
    dist = lambda p: "uniform" if p != G else "normal"
    eq = Equation(f"transpose_{name}", 80, tuple(Operand(r, c, p, dist(p)) for r, c, p in chain),
                  tuple(Operand(r, c, p, dist(p)) for r, c, p in add), chain_t=ct, add_t=at)
    _, x, plan = both(eq, variant)
    if name == "Lt_Lt_plus_Ut":
        assert plan.result_desc().property == U       # (L^T)(L^T) + (L)^T... every summand is upper triangular


@pytest.mark.parametrize("variant", [mom.VARIANT_FFMA, mom.VARIANT_3XTF32], ids=VNAME.get)
def test_transposed_operands_batched(variant):
    eq = Equation("transpose_batched", 81, (Operand(64, 64, L), Operand(48, 64, G), Operand(48, 16, G)), (Operand(16, 64, G),),
                  batch=40, chain_t=(True, True, False), add_t=(True,))
    both(eq, variant)


def test_transposed_operands_large_sampled_rows():
    # large enough for the CTA-pair kernel: X = L^T * B^T + C with L stored lower triangular (used as upper)
    m, n = 3336, 3592
    eq = Equation("transpose_pair", 82, (Operand(m, m, L), Operand(n, m, G, "normal", 0.02)), (Operand(m, n, G, "normal"),),
                  chain_t=(True, True))
    x, plan, (chain, add) = run_equation(eq, mom.VARIANT_3XTF32)
    assert plan.step(0).uses_tensor_cores == 1 and plan.step(0).lhs_property == U
    check_against_oracle(eq, x, plan, chain, add, rows=stratified_rows(m, 4))


def test_config_transposed_full_size_sampled_rows():
    eq = wl.config_transposed()
    x, plan, (chain, add) = run_equation(eq, mom.VARIANT_3XTF32)
    assert plan.parenthesization() == "(0^T*(1*(2^T*3)))"
    check_against_oracle(eq, x, plan, chain, add, rows=stratified_rows(4096, 6))


INLINE_TRANSPOSED = [
    # (m, k, n, left property as used, right property as used, A stored transposed, B stored transposed, Add terms)
    (640, 640, 640, G, G, True, False, 0), (640, 640, 640, G, G, False, True, 1), (640, 640, 640, G, G, True, True, 0),
    (900, 1200, 100, G, G, False, True, 0), (256, 2048, 64, G, G, True, False, 1), (520, 520, 392, U, G, True, False, 0),
    (392, 520, 520, G, L, False, True, 1), (392, 392, 392, U, L, True, True, 0), (1024, 1024, 1024, G, G, True, True, 1),
    (100, 36, 100, G, G, True, True, 0), (1000, 260, 76, G, G, True, False, 0),
]


@pytest.mark.parametrize("m,k,n,pa,pb,ta,tb,terms", INLINE_TRANSPOSED)
def test_inline_kernel_reads_transposed_operands_as_stored(m, k, n, pa, pb, ta, tb, terms):
    # A stored k x m and / or B stored n x k: the one-launch tcgen05 kernel loads the stored tiles and its transform warps read
    # them the other way round (A: a thread gathers its row from a column of the raw boxes; B: the raw tile is K-major already)
    flip = {L: U, U: L, G: G}
    dist = lambda p: "uniform" if p != G else "normal"
    a_op = Operand(k, m, flip[pa], dist(pa), 1.0 / np.sqrt(k)) if ta else Operand(m, k, pa, dist(pa), 1.0 / np.sqrt(k))
    b_op = Operand(n, k, flip[pb], dist(pb)) if tb else Operand(k, n, pb, dist(pb))
    add = (Operand(m, n, G, "normal"),) * terms
    eq = Equation(f"inline_t_{m}x{k}x{n}_{pa}{pb}_{int(ta)}{int(tb)}", 76, (a_op, b_op), add, chain_t=(ta, tb), add_t=(False,) * terms)
    x, plan, (chain, terms_h) = run_equation(eq, mom.VARIANT_3XTF32_INLINE)
    assert plan.step(0).uses_tensor_cores == 3 and plan.last_launch_count() == 1
    assert plan.step(0).lhs_property == pa and plan.step(0).rhs_property == pb
    check_against_oracle(eq, x, plan, chain, terms_h)
