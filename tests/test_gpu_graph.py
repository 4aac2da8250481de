"""mom_equation_execute inside a CUDA graph: once a plan has run (every allocation happens in the first call), its launches,
its second stream and its events can be captured by the caller and replayed; a replay gives the bits of the plain call."""
import numpy as np
import pytest
import torch

import paper_2208_10391_b200 as mom
import workloads as wl
from gpu_util import check_against_oracle, to_device

pytestmark = pytest.mark.gpu


def _setup(eq, variant):
    chain, add = wl.generate(eq)
    plan = mom.mom_equation_plan_transposed(eq.descs(), eq.chain_t, eq.add_descs(), eq.add_t, variant)
    rd = plan.result_desc()
    dchain, dadd = to_device(chain), to_device(add)
    shape = (eq.batch, rd.rows, rd.cols) if eq.batch > 1 else (rd.rows, rd.cols)
    out = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
    wsb = plan.workspace_bytes(eq.batch)
    ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")
    cp = [None if t is None else t.data_ptr() for t in dchain]
    ap = [None if t is None else t.data_ptr() for t in dadd]

    def run(stream):
        if eq.batch > 1:
            plan.execute_batched(cp, [0 if t is None else t[0].numel() for t in dchain], ap,
                                 [0 if t is None else t[0].numel() for t in dadd], out.data_ptr(), rd.rows * rd.cols,
                                 eq.batch, ws.data_ptr() if wsb else None, wsb, stream)
        else:
            plan.execute(cp, ap, out.data_ptr(), ws.data_ptr() if wsb else None, wsb, stream)
    return plan, run, out, (chain, add), (dchain, dadd, ws)


CASES = [
    ("five_general", lambda: wl.config_five_general(), mom.VARIANT_3XTF32),          # warp-level kernel, two streams, clusters of 16
    ("section4", lambda: wl.config_paper_chain(), mom.VARIANT_3XTF32),               # one-launch tcgen05 kernel, dependent launches
    ("tiny", lambda: wl.config_tiny(), mom.VARIANT_3XTF32),                          # fused small-equation kernel
    ("batched", lambda: wl.config_batched(batch=300), mom.VARIANT_3XTF32),           # batched-chain kernel
    ("plane_fed", lambda: wl.config_property_heavy(n=512), mom.VARIANT_3XTF32_FORCE),  # operand splits + plane-fed tcgen05 kernel
    ("pair_form", lambda: wl.Equation("GG_2048x64x2048", 15, (wl.Operand(2048, 64, wl.GENERAL, "normal"),
                                                              wl.Operand(64, 2048, wl.GENERAL, "normal"))), mom.VARIANT_3XTF32),
    ("ffma", lambda: wl.config_property_heavy(n=256), mom.VARIANT_FFMA),
]


@pytest.mark.parametrize("name,make,variant", CASES, ids=[c[0] for c in CASES])
def test_execute_can_be_captured_and_replayed(name, make, variant):
    eq = make()
    plan, run, out, (chain, add), keep = _setup(eq, variant)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        run(stream.cuda_stream)                              # the first call allocates (tile tables, streams, events)
        run(stream.cuda_stream)
        stream.synchronize()
        want = out.clone()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            run(stream.cuda_stream)
        for _ in range(3):
            out.fill_(float("nan"))
            graph.replay()
            stream.synchronize()
            assert torch.equal(out, want)
        # replays back to back, then a plain call again: the plan is still usable outside the graph
        for _ in range(50):
            graph.replay()
        run(stream.cuda_stream)
        stream.synchronize()
        assert torch.equal(out, want)
    assert plan.device_status() == (0, 0)
    check_against_oracle(eq, out.cpu().numpy(), plan, chain, add, instances=(0, eq.batch - 1) if eq.batch > 1 else None)
