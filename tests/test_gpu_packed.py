"""Packed triangular storage on the GPU: operands read from, and results written to, the packed container, against
the fp64 oracle on the unpacked matrices (paper Section 2, "Matrix Attribute": containers other than the dense buffer
are the paper's future work; the container is defined in oracle/packed.py and include/mom.h)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2208_10391_b200 as mom
import workloads as wl
from workloads import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, IDENTITY as I, Operand, Equation
from oracle import packed as pk
from oracle import plan as op
from gpu_util import check_against_oracle, stratified_rows, CANARY

pytestmark = pytest.mark.gpu

D, P = mom.STORAGE_DENSE, mom.STORAGE_PACKED
VARIANTS = [mom.VARIANT_3XTF32, mom.VARIANT_FFMA, mom.VARIANT_3XTF32_FORCE, mom.VARIANT_3XTF32_WARP, mom.VARIANT_3XTF32_INLINE]
VNAME = {mom.VARIANT_FFMA: "ffma", mom.VARIANT_3XTF32_FORCE: "tc", mom.VARIANT_3XTF32: "auto", mom.VARIANT_3XTF32_WARP: "warp", mom.VARIANT_3XTF32_INLINE: "inline"}
LOWER_KINDS = (wl.LOWER_TRI, wl.STRICT_LOWER, wl.UNIT_LOWER)


def is_lower(prop):
    return prop in LOWER_KINDS


def run_stored(eq, variant, chain_s, add_s=None, result_s=D, via="device"):
    """Plan with storage flags, hand packed operands over packed, return (X dense, X as written, plan, host arrays)."""
    chain, add = wl.generate(eq)
    add_s = list(add_s or [D] * len(add))
    plan = mom.mom_equation_plan_stored(eq.descs(), eq.chain_t, chain_s, eq.add_descs(), eq.add_t, add_s, result_s, variant)
    rd = plan.result_desc()
    batch = eq.batch
    stored = lambda a, o, s: a if s == D or a is None else wl.pack_triangle(a, is_lower(o.prop))
    hc = [stored(a, o, s) for a, o, s in zip(chain, eq.chain, chain_s)]
    ha = [stored(a, o, s) for a, o, s in zip(add, eq.add, add_s)]
    n_x = plan.result_elements()
    assert n_x == (pk.elements(rd.rows, pk.LOWER_TRI if is_lower(rd.property) else pk.UPPER_TRI) if result_s == P else rd.rows * rd.cols)
    stream = torch.cuda.current_stream().cuda_stream
    if via == "host":
        stage_bytes = plan.host_staging_bytes(batch)
        staging = torch.full((max(stage_bytes, 256),), 255, dtype=torch.uint8, device="cuda")
        pc = [None if a is None else torch.from_numpy(a).pin_memory() for a in hc]
        pa = [None if a is None else torch.from_numpy(a).pin_memory() for a in ha]
        out = torch.full((batch * n_x,), float("nan"), dtype=torch.float32).pin_memory()
        plan.execute_host([None if t is None else t.data_ptr() for t in pc], [None if t is None else t.data_ptr() for t in pa],
                          out.data_ptr(), batch, staging.data_ptr(), stage_bytes, stream)
        raw = out.numpy().reshape(batch, n_x).copy()
    else:
        dc = [None if a is None else torch.from_numpy(a).cuda() for a in hc]
        da = [None if a is None else torch.from_numpy(a).cuda() for a in ha]
        wsb = plan.workspace_bytes(batch)
        ws = torch.full((max(wsb, 256),), 255, dtype=torch.uint8, device="cuda")           # NaN patterns
        guarded = torch.full((batch * n_x + 2 * CANARY,), float("nan"), dtype=torch.float32, device="cuda")
        guarded[:CANARY] = 12345.0
        guarded[-CANARY:] = 12345.0
        out = guarded[CANARY:CANARY + batch * n_x]
        cp = [None if t is None else t.data_ptr() for t in dc]
        ap = [None if t is None else t.data_ptr() for t in da]
        if batch > 1:
            plan.execute_batched(cp, [0 if t is None else t[0].numel() for t in dc], ap, [0 if t is None else t[0].numel() for t in da],
                                 out.data_ptr(), n_x, batch, ws.data_ptr() if wsb else None, wsb, stream)
        else:
            plan.execute(cp, ap, out.data_ptr(), ws.data_ptr() if wsb else None, wsb, stream)
        torch.cuda.synchronize()
        assert plan.device_status() == (0, 0)
        g = guarded.cpu().numpy()
        assert np.all(g[:CANARY] == 12345.0) and np.all(g[-CANARY:] == 12345.0), "wrote outside the output buffer"
        raw = g[CANARY:CANARY + batch * n_x].reshape(batch, n_x).copy()
    assert not np.isnan(raw).any(), "part of the output was never written"
    if result_s == P:
        o_prop = pk.LOWER_TRI if is_lower(rd.property) else pk.UPPER_TRI
        x = np.stack([pk.unpack(r, rd.rows, o_prop) for r in raw])
        # the container's padding (next to the diagonal, past the last column) holds +0.0f: packing the unpacked matrix
        # gives back the very bits that were written
        for b in range(batch):
            assert np.array_equal(pk.pack(x[b], o_prop).view(np.uint32), raw[b].view(np.uint32))
    else:
        x = raw.reshape(batch, rd.rows, rd.cols)
    return (x if batch > 1 else x[0]), raw, plan, (chain, add)


def check(eq, variant, chain_s, add_s=None, result_s=D, via="device", rows=None):
    x, raw, plan, (chain, add) = run_stored(eq, variant, chain_s, add_s, result_s, via)
    # storage changes neither the plan nor the values: same parenthesization and FLOPs as the oracle's dense plan
    check_against_oracle(eq, x, plan, chain, add, rows=rows)
    return x, plan


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("n", [5, 64, 200, 332])
def test_packed_operands_every_pair(n, variant):
    for pa, pb in [(L, G), (U, G), (G, L), (G, U), (L, L), (U, U), (L, U), (U, L)]:
        eq = Equation(f"packed_{pa}{pb}_{n}", 300 + n, (Operand(n, n, pa, "normal" if pa == G else "uniform"),
                                                       Operand(n, n, pb, "normal" if pb == G else "uniform")))
        check(eq, variant, [P if pa != G else D, P if pb != G else D])


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
@pytest.mark.parametrize("n", [1, 6, 72, 264])
def test_packed_result_and_terms(n, variant):
    # L*L + L (+ I) stays lower triangular: operands, a term and X all packed; U*U likewise
    for tri in (L, U):
        eq = Equation(f"packed_x_{tri}_{n}", 310 + n, (Operand(n, n, tri), Operand(n, n, tri)), (Operand(n, n, tri), Operand(n, n, I)))
        check(eq, variant, [P, P], [P, D], P)
        check(eq, variant, [D, P], [D, D], P)
        check(eq, variant, [P, D], [P, D], D)


@pytest.mark.parametrize("variant", VARIANTS, ids=VNAME.get)
def test_packed_in_chains_with_transposes_and_kinds(variant):
    SL, UU = wl.STRICT_LOWER, wl.UNIT_UPPER
    n = 136
    # a packed lower triangle used transposed, strict and unit kinds in the ordinary triangle's container, a zero-step plan
    eq = Equation("packed_t", 320, (Operand(n, n, L), Operand(n, 72, G, "normal"), Operand(72, 72, U)), (Operand(n, 72, G, "normal"),),
                  chain_t=(True, False, False))
    check(eq, variant, [P, D, P])
    eq = Equation("packed_kinds", 321, (Operand(n, n, SL, "normal"), Operand(n, n, SL, "normal")), (Operand(n, n, L),))
    check(eq, variant, [P, P], [P], P)
    eq = Equation("packed_unit", 322, (Operand(n, n, UU, "normal"), Operand(n, n, UU, "normal")))
    x, plan = check(eq, variant, [P, D], None, P)
    assert plan.result_desc().property == UU
    eq = Equation("packed_zero_step", 323, (Operand(n, n, I), Operand(n, n, L)), (Operand(n, n, L),))
    check(eq, variant, [D, P], [P], P)
    check(eq, variant, [D, P], [D], D)


def test_packed_storage_is_refused_where_it_has_no_meaning():
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan_stored([(8, 8, G), (8, 8, L)], None, [P, D])
    assert e.value.status == mom.ERR_PROPERTY                      # a general matrix has no packed container
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan_stored([(8, 8, L), (8, 8, U)], None, [P, P], (), None, None, P)
    assert e.value.status == mom.ERR_PROPERTY                      # L*U is general: X cannot be packed
    with pytest.raises(mom.MomError) as e:
        mom.mom_equation_plan_stored([(8, 8, L), (8, 8, L)], None, [2, 0])
    assert e.value.status == mom.ERR_INVALID_ARG


def test_large_packed_operands_and_result_on_the_tensor_core_kernel():
    # L*L at 2048 on the CTA-pair kernel: both operands are read from their containers by the operand-split pass and X
    # is written packed by the product kernel's epilogue (tiles above the diagonal are not written at all): no
    # unpacking or packing pass, no extra workspace
    n = 2048
    eq = Equation("packed_LL_2048", 330, (Operand(n, n, L), Operand(n, n, L)), (Operand(n, n, L),))
    dense = mom.mom_equation_plan(eq.descs(), eq.add_descs(), mom.VARIANT_3XTF32_FORCE)      # the same kernel on dense storage
    x, raw, plan, (chain, add) = run_stored(eq, mom.VARIANT_3XTF32, [P, P], [D], P)
    assert plan.step(0).uses_tensor_cores == 1
    assert plan.workspace_bytes(1) == dense.workspace_bytes(1)
    assert plan.last_launch_count() == 2                            # one pass splitting both operands, one product
    check_against_oracle(eq, x, plan, chain, add)
    # a packed term needs its dense copy (one unpacking pass); U*B with a packed U and a dense, general X
    x, raw, plan, (chain, add) = run_stored(eq, mom.VARIANT_3XTF32, [P, P], [P], P)
    assert plan.last_launch_count() == 3
    check_against_oracle(eq, x, plan, chain, add, rows=stratified_rows(n, 1))
    eq = Equation("packed_UB_2048", 331, (Operand(n, n, U), Operand(n, 1536, G, "normal", 0.05)))
    x, plan = check(eq, mom.VARIANT_3XTF32, [P, D])
    assert plan.last_launch_count() == 2
    # through the host entry point: the containers cross the bus as they are
    eq = Equation("packed_host", 332, (Operand(1288, 1288, L), Operand(1288, 1288, L)), (Operand(1288, 1288, L),))
    xd, _, plan_d, _ = run_stored(eq, mom.VARIANT_3XTF32, [P, P], [P], P, via="device")
    xh, _, plan_h, _ = run_stored(eq, mom.VARIANT_3XTF32, [P, P], [P], P, via="host")
    assert np.array_equal(xd, xh)
    packed = 4 * pk.elements(1288, pk.LOWER_TRI)
    assert plan_h.host_upload_bytes(1) == 3 * packed


@pytest.mark.parametrize("variant", [mom.VARIANT_3XTF32, mom.VARIANT_FFMA], ids=VNAME.get)
def test_batched_equations_with_packed_triangles(variant):
    # the benchmark's batched shape with L_i packed: 2176 instead of 4096 entries per instance; with enough instances
    # the batched-chain kernel reads the containers in place (no workspace at all), with few the operands are unpacked
    for batch in (300, 9):
        eq = wl.config_batched(batch=batch)
        x, plan = check(eq, variant, [P, D, D])
        if variant == mom.VARIANT_3XTF32 and batch >= 256:
            assert plan.workspace_bytes(batch) == 0 and plan.last_launch_count() == 1
    eq = Equation("packed_batched_U", 340, (Operand(48, 48, U), Operand(48, 64, G), Operand(64, 64, L), Operand(64, 8, G)), (Operand(48, 8, G),), batch=260)
    check(eq, variant, [P, D, P, D])
    eq = Equation("packed_batched_x", 341, (Operand(16, 16, L), Operand(16, 16, L)), (Operand(16, 16, L),), batch=400)
    check(eq, variant, [P, P], [P], P)
