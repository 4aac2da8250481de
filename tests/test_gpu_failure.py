"""Failure detection on the device: a bounded wait that runs out is reported, cleared, and breaks nothing.

The product kernels never spin forever: every wait on a barrier gives up after a time limit, records
MOM_ERR_DEVICE_TIMEOUT with a detail word in the plan's status block, and the CTA leaves.  Here that route is
driven end to end without breaking any product kernel: the library's self-test kernel waits, with the same wait
routine, on a barrier nothing ever signals, with a limit of a few milliseconds.
"""
import time

import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2208_10391_b200 as mom
import workloads as wl
from gpu_util import run_equation, check_against_oracle

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_cleared_and_leaves_the_plan_usable():
    eq = wl.config_property_heavy(n=520)
    x0, plan, (chain, add) = run_equation(eq, mom.VARIANT_3XTF32_FORCE)      # ends with device_status() == (0, 0)
    stream = torch.cuda.current_stream().cuda_stream
    detail = (7 << 24) | (3 << 16) | 0x1234
    t0 = time.perf_counter()
    plan.probe_wait_timeout(5.0, detail, stream)
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert 0.004 <= waited < 1.0, f"the wait should give up after about 5 ms, took {waited * 1e3:.1f} ms"
    assert plan.device_status() == (mom.ERR_DEVICE_TIMEOUT, detail)
    assert plan.device_status() == (0, 0)                                    # reading cleared it
    # the context and the plan work as before: same bits as the first run, still within the bound
    x1, _, _ = run_equation(eq, mom.VARIANT_3XTF32_FORCE, chain, add)
    dchain = [None if a is None else torch.from_numpy(a).cuda() for a in chain]
    dadd = [None if a is None else torch.from_numpy(a).cuda() for a in add]
    out = torch.full((520, 520), float("nan"), dtype=torch.float32, device="cuda")
    wsb = plan.workspace_bytes(1)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")
    plan.execute([None if t is None else t.data_ptr() for t in dchain], [None if t is None else t.data_ptr() for t in dadd],
                 out.data_ptr(), ws.data_ptr() if wsb else None, wsb, stream)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    x2 = out.cpu().numpy()
    assert np.array_equal(x0, x1) and np.array_equal(x0, x2)
    check_against_oracle(eq, x2, plan, chain, add)


def test_only_the_first_failure_is_kept_and_a_fresh_plan_can_run_the_self_test():
    eq = wl.config_tiny()
    plan = mom.mom_equation_plan(eq.descs(), eq.add_descs(), mom.VARIANT_3XTF32)   # never executed: no device state yet
    stream = torch.cuda.current_stream().cuda_stream
    plan.probe_wait_timeout(2.0, 111, stream)
    plan.probe_wait_timeout(2.0, 222, stream)
    torch.cuda.synchronize()
    assert plan.device_status() == (mom.ERR_DEVICE_TIMEOUT, 111)              # the first failure's detail word stays
    assert plan.device_status() == (0, 0)
    with pytest.raises(mom.MomError) as e:
        plan.probe_wait_timeout(0.0, 1, stream)
    assert e.value.status == mom.ERR_INVALID_ARG
    with pytest.raises(mom.MomError):
        plan.probe_wait_timeout(5000.0, 1, stream)                            # limits above one second are refused
    x, plan2, (chain, add) = run_equation(eq, mom.VARIANT_3XTF32)
    check_against_oracle(eq, x, plan2, chain, add)


@pytest.mark.parametrize("name", ["five_general", "paper_chain", "square_640", "tri_chain"])
def test_back_to_back_executions_give_the_same_bits(name):
    # The small-product kernels are launched so that a product's prologue overlaps the previous product's tail (programmatic
    # dependent launch): a product must still see everything its predecessors wrote.  300 executions enqueued back to back, each
    # into its own output: all bit-identical, and the first one within the bound of the oracle.
    eq = {"five_general": wl.config_five_general(), "paper_chain": wl.config_paper_chain(), "square_640": wl.config_square_product(640),
          "tri_chain": wl.Equation("tri_chain", 77, (wl.Operand(520, 520, wl.LOWER_TRI), wl.Operand(520, 520, wl.GENERAL, "normal", 0.05),
                                                     wl.Operand(520, 520, wl.UPPER_TRI), wl.Operand(520, 136, wl.GENERAL, "normal")),
                                   (wl.Operand(520, 136, wl.GENERAL, "normal"),))}[name]
    chain, add = wl.generate(eq)
    plan = mom.mom_equation_plan(eq.descs(), eq.add_descs(), mom.VARIANT_3XTF32)
    rd = plan.result_desc()
    dchain = [None if a is None else torch.from_numpy(a).cuda() for a in chain]
    dadd = [None if a is None else torch.from_numpy(a).cuda() for a in add]
    reps = 300
    outs = torch.full((reps, rd.rows, rd.cols), float("nan"), dtype=torch.float32, device="cuda")
    wsb = plan.workspace_bytes(1)
    ws = torch.full((max(wsb, 256),), 255, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    cp = [None if t is None else t.data_ptr() for t in dchain]
    ap = [None if t is None else t.data_ptr() for t in dadd]
    for i in range(reps):
        plan.execute(cp, ap, outs[i].data_ptr(), ws.data_ptr() if wsb else None, wsb, stream)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    x = outs.cpu().numpy()
    check_against_oracle(eq, x[0], plan, chain, add)
    same = (x.view(np.uint32) == x[0].view(np.uint32)).reshape(reps, -1).all(axis=1)
    assert same.all(), f"executions {np.nonzero(~same)[0][:10].tolist()} differ from the first"
