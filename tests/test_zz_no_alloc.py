"""The backward entry point that keeps its scratch inside the library (harts_la_bwd_static).

Some users of this library run the backward at a point where they cannot obtain device memory: their step's
memory was handed out in full up front, or they are given tensors but no allocator.  For them the library
carries a fixed scratch array; this test checks that the entry point using it gives the same gradients as the
ordinary one (which takes a caller-owned scratch buffer), twice in a row -- the second call finds the first
call's leftovers in the array -- and that a problem too large for the array is refused.
This file is collected last on purpose, so a run that stops at the first failure has run everything else."""
import pytest
import torch

import paper_2608_28158_b200 as H
from parity_util import config_case, plan_of, to_physical

pytestmark = pytest.mark.gpu


def _problem(name):
    cfg, fo, inp = config_case(name)
    plan = plan_of(fo).upload()
    phys = to_physical(plan, inp)
    ws = H.Workspace(plan, cfg["H"], cfg["dk"], cfg["dv"], phys["q"].dtype)
    ref = H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
    H.harts_la_check(ws.dev_status)
    return plan, phys, ws, {n: x.clone() for n, x in ref.items()}


def _static_backward(plan, phys, ws, like):
    got = {n: torch.full_like(like[n], float("nan")) for n in ("dq", "dk", "dv", "dg")}
    H.harts_la_bwd_static(plan, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"], got["dq"], got["dk"],
                          got["dv"], got["dg"], ws.chunk_states, dev_status=ws.dev_status)
    H.harts_la_check(ws.dev_status)
    return got


@pytest.mark.parametrize("name,other", [("cfg0b", "cfg1"), ("cfg1", "cfg0b")])
def test_static_scratch_backward_matches_the_caller_scratch_backward(name, other):
    """Same kernels, same inputs, only the scratch lives elsewhere: the gradients must be the same BITS.  Between
    the two calls another problem (another plan, another layout of the scratch) runs through the same array, so the
    second call starts on leftovers that are wrong for it; and the second call must not change the device's free
    memory."""
    plan, phys, ws, ref = _problem(name)
    plan2, phys2, ws2, ref2 = _problem(other)
    first = _static_backward(plan, phys, ws, ref)
    for n in first:
        assert torch.equal(first[n], ref[n]), (name, "first call", n)
    between = _static_backward(plan2, phys2, ws2, ref2)
    for n in between:
        assert torch.equal(between[n], ref2[n]), (other, "call in between", n)
    torch.cuda.synchronize()
    got = {n: torch.full_like(ref[n], float("nan")) for n in ("dq", "dk", "dv", "dg")}
    free_before = torch.cuda.mem_get_info()[0]
    H.harts_la_bwd_static(plan, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"], got["dq"], got["dk"],
                          got["dv"], got["dg"], ws.chunk_states, dev_status=ws.dev_status)
    H.harts_la_check(ws.dev_status)
    assert torch.cuda.mem_get_info()[0] == free_before
    for n in got:
        assert torch.equal(got[n], ref[n]), (name, "second call", n)


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
