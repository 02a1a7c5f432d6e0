"""End-to-end steps on host buffers (the call `bench.py` times for its `e2e` figure): the pipelined form, which
overlaps the copies of neighbouring steps with the kernels, must give the bits of the plain step by step form."""
import pytest
import torch

import paper_2608_28158_b200 as H
from workloads import make_inputs
from parity_util import config_case, plan_of, to_physical

pytestmark = pytest.mark.gpu


def test_pipelined_host_steps_equal_eager_steps():
    cfg, fo, _ = config_case("cfg1")
    plan = plan_of(fo).upload()
    Hh, dk, dv = cfg["H"], cfg["dk"], cfg["dv"]
    steps = []
    for seed in (21, 22, 23, 24, 25):
        phys = to_physical(plan, make_inputs(fo.n_tokens, Hh, dk, dv, cfg["dtype"], seed), device="cpu")
        steps.append({n: x.pin_memory() for n, x in phys.items()})
    ws = H.Workspace(plan, Hh, dk, dv, steps[0]["q"].dtype, 0)
    # eager reference, one step at a time
    want = []
    for host_in in steps:
        dev = {n: x.cuda() for n, x in host_in.items()}
        out = H.run_fwd_bwd(plan, ws, dev["q"], dev["k"], dev["v"], dev["g"], dev["dO"])
        H.harts_la_check(ws.dev_status)
        want.append({n: x.cpu() for n, x in out.items()})
    like_in = {n: x.cuda() for n, x in steps[0].items()}
    like_out = {n: torch.empty_like(x, device="cuda") for n, x in want[0].items()}
    pipe = H.HostPipeline(plan, ws, like_in, like_out)
    got = [{n: torch.empty_like(x).pin_memory() for n, x in want[0].items()} for _ in steps]
    for host_in, host_out in zip(steps, got):
        pipe.step(host_in, host_out)
    pipe.finish()
    H.harts_la_check(ws.dev_status)
    for k, (g, w) in enumerate(zip(got, want)):
        for n in w:
            assert torch.equal(g[n], w[n]), (k, n)
    # the unpipelined form of the same call
    dev_in = {n: torch.empty_like(x) for n, x in like_in.items()}
    host_out = {n: torch.empty_like(x).pin_memory() for n, x in want[0].items()}
    H.run_fwd_bwd_host(plan, ws, steps[2], dev_in, like_out, host_out)
    for n in host_out:
        assert torch.equal(host_out[n], want[2][n]), n
