"""The allocation-free product entry point against the ordinary execute path.

`mom_product_3xtf32_noalloc` serves callers that cannot allocate device memory at the point where they
need a product (a component living inside an application that owns all device memory, or a loop that must
not touch an allocator) and have no workspace to lend: its scratch is an array built into the library.
This file is collected last on purpose, so that a run that stops at the first failure has already run every
other test.  Each case makes two calls in a row because all calls share the one array: the second call sees
whatever the first left behind (other shapes, other structure) and must still be right.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import paper_2208_10391_b200 as mom
import workloads as wl
from workloads import GENERAL as G, LOWER_TRI as L, UPPER_TRI as U, Operand, Equation
from gpu_util import TOL
from oracle import values as ov

pytestmark = pytest.mark.gpu


def _reference(eq, chain):
    """The same product through mom_equation_execute (tensor-core kernel forced), with a caller workspace."""
    plan = mom.mom_equation_plan(eq.descs(), (), mom.VARIANT_3XTF32_FORCE)
    assert plan.step(0).uses_tensor_cores == 1
    d = [torch.from_numpy(a).cuda() for a in chain]
    rd = plan.result_desc()
    out = torch.full((rd.rows, rd.cols), float("nan"), dtype=torch.float32, device="cuda")
    wsb = plan.workspace_bytes()
    ws = torch.empty(wsb, dtype=torch.uint8, device="cuda")
    plan.execute([t.data_ptr() for t in d], [], out.data_ptr(), ws.data_ptr(), wsb, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    return out.cpu().numpy(), rd.property


def _no_alloc(eq, chain, out, status):
    a, b = (torch.from_numpy(x).cuda() for x in chain)
    (m, k, pa), (_, n, pb) = eq.descs()
    out.fill_(float("nan"))
    status.zero_()
    torch.cuda.synchronize()
    mom.mom_product_3xtf32_noalloc(m, n, k, pa, pb, a.data_ptr(), b.data_ptr(), out.data_ptr(), status.data_ptr(),
                                   torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[:2] == [0, 0], "a device-side wait timed out"
    return out[: m * n].cpu().numpy().reshape(m, n)


def _check(eq, out, status):
    chain, _ = wl.generate(eq)
    want, prop = _reference(eq, chain)
    got = _no_alloc(eq, chain, out, status)
    x_ref, d = ov.evaluate(chain, eq.descs())
    assert ov.normwise_error(got, x_ref, d) <= TOL                       # against the oracle
    assert ov.normwise_error(got, want.astype(np.float64), d) <= TOL     # against the existing entry point
    mask = ov.off_structure_mask(got.shape[0], got.shape[1], prop)
    assert np.all(got.view(np.uint32)[mask] == 0)


def test_two_calls_in_a_row_match_the_execute_path():
    # buffers are allocated up front by the test; the calls under test allocate nothing
    out = torch.empty(1024 * 1024, dtype=torch.float32, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    first = Equation("noalloc_LL", 31, (Operand(1024, 1024, L), Operand(1024, 1024, L)))          # fills the array to its limit
    second = Equation("noalloc_GG", 32, (Operand(392, 520, G, "normal"), Operand(520, 136, G, "normal")))
    third = Equation("noalloc_UG", 33, (Operand(264, 264, U), Operand(264, 776, G, "normal")))
    _check(first, out, status)
    _check(second, out, status)
    _check(third, out, status)
    _check(first, out, status)


def test_sizes_beyond_the_built_in_array_are_rejected():
    # every call below must be refused before anything is enqueued: the tiny buffer is never touched
    a = torch.zeros(16, dtype=torch.float32, device="cuda")
    def status(m, n, k, pa=G, pb=G):
        try:
            mom.mom_product_3xtf32_noalloc(m, n, k, pa, pb, a.data_ptr(), a.data_ptr(), a.data_ptr(), None, 0)
        except mom.MomError as e:
            return e.status
        return mom.OK
    assert status(1024, 1028, 1024) == mom.ERR_LIMIT            # planes would need more than 16 MiB
    assert status(8192, 8192, 8192) == mom.ERR_LIMIT
    assert status(64, 64, 62) == mom.ERR_INVALID_ARG            # k not a multiple of 4
    assert status(64, 32, 48, L, G) == mom.ERR_PROPERTY         # triangular operand must be square
    assert status(0, 4, 4) == mom.ERR_INVALID_ARG
