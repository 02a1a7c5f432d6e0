"""The failure path of the bounded device-side waits, exercised without faulting or hanging anything: a tiny kernel
waits (limit: one millisecond) on a barrier nothing arrives at, then on a flag nobody sets.  The wait must run out, the CTA's latch must make the
next wait return at once, harts_la_check must report the time-out, and the context must stay usable: a normal
forward+backward afterwards gives the same bits as one before."""
import pytest
import torch

import paper_2608_28158_b200 as H
from parity_util import config_case, plan_of, to_physical

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    cfg, fo, inp = config_case("cfg1")
    plan = plan_of(fo).upload()
    phys = to_physical(plan, inp)
    ws = H.Workspace(plan, cfg["H"], cfg["dk"], cfg["dv"], phys["q"].dtype)
    before = H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
    H.harts_la_check(ws.dev_status)
    before = {n: x.clone() for n, x in before.items()}

    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    report = torch.full((8,), -1, dtype=torch.int32, device="cuda")
    H.harts_la_selftest_timeout(status, report)
    with pytest.raises(H.HartsError) as e:
        H.harts_la_check(status)
    assert e.value.code == -4                                   # HARTS_ETIMEOUT
    first_ok, second_ok, us_first, us_second, saw_latch = report[:5].tolist()
    print("selftest report:", report[:5].tolist())
    assert first_ok == 0 and second_ok == 0 and saw_latch == 1
    assert 900 <= us_first <= 100_000                           # ran for about the limit, not for the default half second
    assert us_second <= 100                                     # the latch: no second spin
    # the flag wait of the one-launch forms: runs out after its limit and latches; with the status word already set
    # (another CTA gave up) it returns at once and latches too
    flag_bits, us_flag, us_flag_status = report[5:8].tolist()
    assert flag_bits == 4 + 8 and 900 <= us_flag <= 100_000 and us_flag_status <= 100

    after = H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
    H.harts_la_check(ws.dev_status)                             # this workspace's own status word is still clean
    for n in after:
        assert torch.equal(after[n], before[n]), n
