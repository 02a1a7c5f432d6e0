"""The backward entry point that keeps its scratch inside the library (harts_la_bwd_static).

Some users of this library run the backward at a point where they cannot obtain device memory: their step's
memory was handed out in full up front, or they are given tensors but no allocator.  For them the library
carries a fixed scratch array; this test checks that the entry point using it gives the same gradients as the
ordinary one (which takes a caller-owned scratch buffer), twice in a row -- the second call finds the first
call's leftovers in the array -- and that a problem too large for the array is refused.
This file is collected last on purpose, so a run that stops at the first failure has run everything else."""
import numpy as np
import pytest
import torch

import paper_2608_28158_b200 as H
from parity_util import config_case, plan_of, to_physical

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["cfg0b", "cfg1"])
def test_static_scratch_backward_matches_the_caller_scratch_backward(name):
    cfg, fo, inp = config_case(name)
    plan = plan_of(fo).upload()
    phys = to_physical(plan, inp)
    ws = H.Workspace(plan, cfg["H"], cfg["dk"], cfg["dv"], phys["q"].dtype)
    ref = H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
    H.harts_la_check(ws.dev_status)
    ref = {n: x.clone() for n, x in ref.items()}
    for attempt in range(2):
        got = {n: torch.full_like(ref[n], float("nan")) for n in ("dq", "dk", "dv", "dg")}
        H.harts_la_bwd_static(plan, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"], got["dq"], got["dk"],
                              got["dv"], got["dg"], ws.chunk_states, dev_status=ws.dev_status)
        H.harts_la_check(ws.dev_status)
        for n in got:
            a, b = got[n].float().cpu().numpy(), ref[n].float().cpu().numpy()
            err = np.linalg.norm(a - b) / np.linalg.norm(b)
            # same kernels, same inputs: the tolerance of the parity tests is far more than is needed
            assert err <= (1e-4 if cfg["dtype"] == "fp32" else 1e-2), (name, attempt, n, err)
            assert np.isfinite(a).all()


def test_static_scratch_rejects_a_problem_that_does_not_fit():
    cfg, fo, inp = config_case("cfg2", device="cuda")     # needs 69 x 16 x 64 KiB of scratch: more than the array
    plan = plan_of(fo).upload()
    q = torch.zeros(plan.C, cfg["H"], 128, dtype=torch.bfloat16, device="cuda")
    g = torch.zeros(plan.C, cfg["H"], dtype=torch.float32, device="cuda")
    cs = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(H.HartsError) as e:
        H.harts_la_bwd_static(plan, q, q, q, g, q, q, q, q, g, cs)
    assert e.value.code == -7
    torch.cuda.synchronize()
