"""Helpers for the GPU parity tests: device buffers through PyTorch, calls through the C ABI."""
from __future__ import annotations

import numpy as np
import torch

import paper_2208_10391_b200 as mom
from oracle import plan as op
from oracle import values as ov
import workloads as wl

TOL = 1e-5          # normwise bound ||X - X_ref||_F / || |M1|...|Mn| + sum|Ti| ||_F stated for this method
CANARY = 64         # guard floats on each side of the output buffer


def stratified_rows(m: int, seed: int, slab: int = 32, extra=()):
    """One row out of every `slab` consecutive rows (drawn at random inside the slab), plus `extra` rows.

    The tensor-core kernels write the output in tiles of 128 or 256 rows, each epilogue warp a slab of 32 rows:
    with one row per slab every tile row and every warp's slab of a large output is compared with the oracle,
    at a cost the oracle can afford (m / 32 vector-matrix chains).
    """
    rng = np.random.default_rng(seed)
    rows = [min(m - 1, r0 + int(rng.integers(0, slab))) for r0 in range(0, m, slab)]
    rows += [r for r in extra if 0 <= r < m]
    return np.unique(np.array(rows, dtype=np.int64))


def to_device(arrs):
    return [None if a is None else torch.from_numpy(a).cuda() for a in arrs]


def run_equation(eq: wl.Equation, variant: int, chain=None, add=None, via: str = "device"):
    """Plan and evaluate `eq` on the GPU; returns (X as numpy f32, plan, (chain, add) host arrays)."""
    if chain is None:
        chain, add = wl.generate(eq)
    plan = mom.mom_equation_plan_transposed(eq.descs(), eq.chain_t, eq.add_descs(), eq.add_t, variant)
    rd = plan.result_desc()
    batch = eq.batch
    shape = (batch, rd.rows, rd.cols) if batch > 1 else (rd.rows, rd.cols)
    n_out = int(np.prod(shape))
    stream = torch.cuda.current_stream().cuda_stream
    if via == "host":
        stage_bytes = plan.host_staging_bytes(batch)
        staging = torch.full((max(stage_bytes, 256),), 255, dtype=torch.uint8, device="cuda")   # NaN patterns: nothing stale may be read
        pinned = [None if a is None else torch.from_numpy(a).pin_memory() for a in chain]
        pinned_add = [None if a is None else torch.from_numpy(a).pin_memory() for a in add]
        out = torch.full((n_out,), float("nan"), dtype=torch.float32).pin_memory()
        plan.execute_host([None if t is None else t.data_ptr() for t in pinned],
                          [None if t is None else t.data_ptr() for t in pinned_add],
                          out.data_ptr(), batch, staging.data_ptr(), stage_bytes, stream)
        x = out.numpy().reshape(shape).copy()
    else:
        dchain, dadd = to_device(chain), to_device(add)
        ws_bytes = plan.workspace_bytes(batch)
        ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
        guarded = torch.full((n_out + 2 * CANARY,), float("nan"), dtype=torch.float32, device="cuda")
        guarded[:CANARY] = 12345.0
        guarded[-CANARY:] = 12345.0
        out = guarded[CANARY:CANARY + n_out]
        assert out.data_ptr() % 16 == 0
        cp = [None if t is None else t.data_ptr() for t in dchain]
        ap = [None if t is None else t.data_ptr() for t in dadd]
        if batch > 1:
            cs = [0 if t is None else t[0].numel() for t in dchain]
            as_ = [0 if t is None else t[0].numel() for t in dadd]
            plan.execute_batched(cp, cs, ap, as_, out.data_ptr(), rd.rows * rd.cols, batch,
                                 ws.data_ptr() if ws_bytes else None, ws_bytes, stream)
        else:
            plan.execute(cp, ap, out.data_ptr(), ws.data_ptr() if ws_bytes else None, ws_bytes, stream)
        torch.cuda.synchronize()
        assert plan.device_status() == (0, 0), "a device-side wait timed out"
        g = guarded.cpu().numpy()
        assert np.all(g[:CANARY] == 12345.0) and np.all(g[-CANARY:] == 12345.0), "wrote outside the output buffer"
        x = g[CANARY:CANARY + n_out].reshape(shape).copy()
    assert plan.last_launch_count() >= 1
    return x, plan, (chain, add)


def check_against_oracle(eq: wl.Equation, x: np.ndarray, plan, chain, add, rows=None, instances=None, tol: float = TOL):
    """Element-wise parity with the fp64 oracle; returns the worst normwise error seen."""
    want = op.plan(eq.descs(), eq.add_descs(), eq.chain_t, eq.add_t)
    assert plan.parenthesization() == want.paren
    assert plan.flops() == (want.mul_flops, want.add_flops)
    prop = plan.result_desc().property
    assert prop == want.result_desc.prop
    assert not np.isnan(x).any(), "part of the output was never written"
    worst = 0.0
    insts = range(eq.batch) if instances is None else instances
    for b in (insts if eq.batch > 1 else [None]):
        c = [None if a is None else (a if b is None else a[b]) for a in chain]
        t = [None if a is None else (a if b is None else a[b]) for a in add]
        xb = x if b is None else x[b]
        c, cd = ov.transposed_operands(c, eq.descs(), eq.chain_t)
        t, td = ov.transposed_operands(t, eq.add_descs(), eq.add_t)
        x_ref, d = ov.evaluate(c, cd, t, td, rows=rows)
        got = xb if rows is None else xb[rows]
        err = ov.normwise_error(got, x_ref, d)
        assert err <= tol, f"normwise error {err:.3e} > {tol:.1e} ({eq.name}, instance {b})"
        worst = max(worst, err)
        # entries outside the result's structure: exactly +0.0f (all 32 bits clear)
        mask = ov.off_structure_mask(xb.shape[0], xb.shape[1], prop)
        assert np.all(xb.view(np.uint32)[mask] == 0), "off-structure entries must be +0.0f"
        assert ov.unit_diagonal_exactly_one(xb, prop), "the diagonal of a unit triangular result must be exactly 1"
    return worst


def run_sum_equation(eq: wl.SumEquation, variant: int, use_names: bool = True, poison_out: bool = True):
    """Plan and evaluate a sum of chains on the GPU; returns (X, plan, per-chain host arrays)."""
    arrays = wl.generate_sum(eq)
    plan = mom.mom_equation_plan_sum(eq.descs(), eq.transposed, eq.names if use_names else None, variant)
    rd = plan.result_desc()
    n_out = rd.rows * rd.cols
    stream = torch.cuda.current_stream().cuda_stream
    dev = {}
    ptrs = []
    for chain, names in zip(arrays, eq.names):
        for a, nm in zip(chain, names):
            if a is None:
                ptrs.append(None)
                continue
            if nm not in dev:
                dev[nm] = torch.from_numpy(a).cuda()
            ptrs.append(dev[nm].data_ptr())
    ws_bytes = plan.workspace_bytes(1)
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    guarded = torch.full((n_out + 2 * CANARY,), float("nan") if poison_out else 7.0, dtype=torch.float32, device="cuda")
    guarded[:CANARY] = 12345.0
    guarded[-CANARY:] = 12345.0
    out = guarded[CANARY:CANARY + n_out]
    plan.execute(ptrs, [], out.data_ptr(), ws.data_ptr() if ws_bytes else None, ws_bytes, stream)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0), "a device-side wait timed out"
    g = guarded.cpu().numpy()
    assert np.all(g[:CANARY] == 12345.0) and np.all(g[-CANARY:] == 12345.0), "wrote outside the output buffer"
    return g[CANARY:CANARY + n_out].reshape(rd.rows, rd.cols).copy(), plan, arrays


def check_sum_against_oracle(eq: wl.SumEquation, x: np.ndarray, plan, arrays, use_names: bool = True, rows=None,
                             tol: float = TOL):
    want = op.plan_sum(eq.descs(), eq.transposed, eq.names if use_names else ())
    assert plan.parenthesization() == want.paren
    assert plan.flops() == (want.mul_flops, want.add_flops)
    assert plan.reused_products() == want.reused
    prop = plan.result_desc().property
    assert prop == want.result_desc.prop
    assert not np.isnan(x).any(), "part of the output was never written"
    used_a, used_d = [], []
    for chain, descs, flags in zip(arrays, eq.descs(), eq.transposed):
        a, d = ov.transposed_operands(chain, descs, flags)
        used_a.append(a)
        used_d.append(d)
    x_ref, den = ov.evaluate_sum(used_a, used_d, rows=rows)
    got = x if rows is None else x[rows]
    err = ov.normwise_error(got, x_ref, den)
    assert err <= tol, f"normwise error {err:.3e} > {tol:.1e} ({eq.name})"
    mask = ov.off_structure_mask(x.shape[0], x.shape[1], prop)
    assert np.all(x.view(np.uint32)[mask] == 0), "off-structure entries must be +0.0f"
    assert ov.unit_diagonal_exactly_one(x, prop), "the diagonal of a unit triangular result must be exactly 1"
    return err


def run_expression(ex: wl.Expression, variant: int, via: str = "device"):
    """Plan and evaluate a nested expression on the GPU; returns (X, plan, operand host arrays)."""
    arrays = wl.generate_expression(ex)
    plan = mom.mom_expression_plan(ex.expr, ex.descs(), variant)
    rd = plan.result_desc()
    n_out = rd.rows * rd.cols
    stream = torch.cuda.current_stream().cuda_stream
    if via == "host":
        stage_bytes = plan.host_staging_bytes(1)
        staging = torch.empty(max(stage_bytes, 256), dtype=torch.uint8, device="cuda")
        pinned = [None if a is None else torch.from_numpy(a).pin_memory() for a in arrays]
        out = torch.full((n_out,), float("nan"), dtype=torch.float32).pin_memory()
        plan.execute_host([None if t is None else t.data_ptr() for t in pinned], [], out.data_ptr(), 1,
                          staging.data_ptr(), stage_bytes, stream)
        return out.numpy().reshape(rd.rows, rd.cols).copy(), plan, arrays
    dev = to_device(arrays)
    ws_bytes = plan.workspace_bytes(1)
    ws = torch.full((max(ws_bytes, 256) // 4,), float("nan"), dtype=torch.float32, device="cuda")
    guarded = torch.full((n_out + 2 * CANARY,), float("nan"), dtype=torch.float32, device="cuda")
    guarded[:CANARY] = 12345.0
    guarded[-CANARY:] = 12345.0
    out = guarded[CANARY:CANARY + n_out]
    plan.execute([None if t is None else t.data_ptr() for t in dev], [], out.data_ptr(),
                 ws.data_ptr() if ws_bytes else None, ws_bytes, stream)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0), "a device-side wait timed out"
    g = guarded.cpu().numpy()
    assert np.all(g[:CANARY] == 12345.0) and np.all(g[-CANARY:] == 12345.0), "wrote outside the output buffer"
    return g[CANARY:CANARY + n_out].reshape(rd.rows, rd.cols).copy(), plan, arrays


def check_expression_against_oracle(ex: wl.Expression, x: np.ndarray, plan, arrays, tol: float = TOL, sample_rows=None):
    want = op.plan_expr(ex.expr, ex.descs())
    assert plan.parenthesization() == want.paren
    assert plan.flops() == (want.mul_flops, want.add_flops)
    assert (plan.temporaries(), plan.reused_products()) == (want.temporaries, want.reused)
    prop = plan.result_desc().property
    assert prop == want.result_desc.prop
    assert not np.isnan(x).any(), "part of the output was never written"
    x_ref, den = ov.evaluate_expr(ex.expr, arrays, ex.descs())
    if sample_rows is not None:
        err = ov.normwise_error(x[sample_rows], x_ref[sample_rows], den[sample_rows])
    else:
        err = ov.normwise_error(x, x_ref, den)
    assert err <= tol, f"normwise error {err:.3e} > {tol:.1e} ({ex.name})"
    mask = ov.off_structure_mask(x.shape[0], x.shape[1], prop)
    assert np.all(x.view(np.uint32)[mask] == 0), "off-structure entries must be +0.0f"
    assert ov.unit_diagonal_exactly_one(x, prop), "the diagonal of a unit triangular result must be exactly 1"
    return err
