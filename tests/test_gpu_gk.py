"""GPU parity of the per-channel-decay path (harts_la_gk_fwd / harts_la_gk_bwd, the Diag(gamma) term of Eq. 1)
through the C ABI against its fp64 trajectory-wise oracle, per tensor (relative Frobenius error) and per row.

Tolerances: fp32 inputs (fp32 arithmetic on the CUDA cores): 1e-4 (fast exponential, fp32 accumulation over 64-row
chunks).  bf16 inputs: outputs 5e-3, gradients 1e-2 -- the operands q~ = q e^{b}, k~ = k e^{b_n-b}, the scores and the
stored chunk states are rounded to bf16 as in the scalar-gate kernels; with d = 128 the dense products run on the
tensor cores (bf16 operands, fp32 accumulation), with d = 64 on the CUDA cores."""
import numpy as np
import pytest
import torch

import paper_2608_28158_b200 as H
from oracle import gk_oracle as go
from workloads import config_forest, make_forest, make_gk, make_inputs
from parity_util import plan_of, rel_err, row_err, to_physical

pytestmark = pytest.mark.gpu
TOL = {"fp32": dict(o=1e-4, dq=1e-4, dk=1e-4, dv=1e-4, dg=1e-4),
       "bf16": dict(o=5e-3, dq=1e-2, dk=1e-2, dv=1e-2, dg=1e-2)}
ROW_MULT = 3.0
DT = {"fp32": torch.float32, "bf16": torch.bfloat16}


def run_gk(fo, heads, d, dtype, seed, strong_every=0, backward=True, flags=0, raw=False, strong_shift=7.0):
    inp = make_inputs(fo.n_tokens, heads, d, d, dtype, seed)
    inp["g"] = make_gk(fo.n_tokens, heads, d, seed, strong_every=strong_every, strong_shift=strong_shift)
    plan = plan_of(fo).upload()
    phys = to_physical(plan, inp)
    cs_bytes, sc_bytes = H.harts_la_gk_workspace_bytes(plan.tables, heads, d, d, 0 if dtype == "fp32" else 1)
    slots = torch.full((max(plan.n_slots, 1) * heads * d * d,), float("nan"), device="cuda")
    cs = torch.empty(cs_bytes, dtype=torch.uint8, device="cuda")
    scratch = torch.empty(sc_bytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    out = {"o": torch.full_like(phys["v"], float("nan"))}
    H.harts_la_gk_fwd(plan, 0, phys["q"], phys["k"], phys["v"], phys["g"], out["o"], slots, cs, flags=flags,
                      dev_status=status)
    if backward:
        out.update(dq=torch.full_like(phys["q"], float("nan")), dk=torch.full_like(phys["k"], float("nan")),
                   dv=torch.full_like(phys["v"], float("nan")), dg=torch.full_like(phys["g"], float("nan")))
        H.harts_la_gk_bwd(plan, 0, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"], out["dq"], out["dk"],
                          out["dv"], out["dg"], cs, scratch, flags=flags, dev_status=status)
    H.harts_la_check(status)
    rows = torch.as_tensor(plan.row_of_token.astype(np.int64), device="cuda")
    got = {n: x[rows].float().cpu().numpy() for n, x in out.items()}
    if raw:
        return plan, got
    ref = go.forest_eval(fo, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"] if backward else None)
    assert ref["copy_gap"] < 1e-9
    errs = {}
    for n in got:
        errs[n] = rel_err(got[n], ref[n])
        errs[n + ".row"] = row_err(got[n], ref[n])
        assert np.isfinite(got[n]).all(), n
    return plan, errs


def check(errs, dtype):
    for n, e in errs.items():
        base = n.split(".")[0]
        assert e <= TOL[dtype][base] * (ROW_MULT if n.endswith(".row") else 1.0), (n, e, errs)


@pytest.mark.parametrize("name,dtype,d,heads", [("cfg0", "fp32", 64, 1), ("cfg0b", "fp32", 64, 2), ("cfg0b", "bf16", 64, 2),
                                                ("cfg0b", "bf16", 128, 2), ("cfg1", "bf16", 128, 1)])
def test_configs_against_the_oracle(name, dtype, d, heads):
    plan, errs = run_gk(config_forest(name), heads, d, dtype, 11)
    print(name, dtype, d, errs)
    check(errs, dtype)


def test_edge_forests_and_random_forests():
    import random
    from test_gpu_parity import edge_forests
    from test_plan_oracle import random_tree
    rnd = random.Random(5)
    forests = list(edge_forests().values())
    forests += [make_forest([random_tree(rnd, rnd.randint(1, 10), rnd.choice([5, 70, 300])) for _ in range(rnd.randint(1, 3))])
                for _ in range(10)]
    for n, fo in enumerate(forests):
        dtype, d = (("fp32", 64), ("bf16", 128), ("bf16", 64))[n % 3]
        plan, errs = run_gk(fo, 1 + n % 2, d, dtype, 30 + n)
        check(errs, dtype)


def test_gates_far_outside_the_usual_range_do_not_overflow():
    """Every 8th channel decays by about e^-4 per token (e^-250 over a chunk): a kernel that factorised
    e^{b_t} e^{-b_j} from the chunk start would overflow here; this one evaluates e^{b_t-b_j} directly."""
    plan, errs = run_gk(config_forest("cfg0b"), 2, 64, "fp32", 3, strong_every=8)
    print(errs)
    check(errs, "fp32")
    plan, errs = run_gk(config_forest("cfg0b"), 1, 128, "bf16", 3, strong_every=8)
    check(errs, "bf16")
    # The tensor-core kernels take the pairs inside a 16-row block as a dense product while no channel decays by more
    # than 2^100 over the block, and by the exact per-pair path otherwise.  Gates of about -4 per token sit right at that
    # limit (a mixture of both kinds of chunks); gates of about -9 per token (e^-570 per chunk) are all beyond it; mild
    # gates with two such channels test the decision per chunk.
    for shift, every in ((12.0, 8), (12.0, 64), (9.0, 3)):
        plan, errs = run_gk(config_forest("cfg0b"), 2, 128, "bf16", 4, strong_every=every, strong_shift=shift)
        check(errs, "bf16")
    plan, errs = run_gk(config_forest("cfg1"), 1, 128, "bf16", 6, strong_every=16, strong_shift=8.0)
    check(errs, "bf16")


def test_bench_size_sampled_parity():
    """The benchmark's workload for this path -- cfg2's forest, 16 heads, d = 128, bf16, all rounds in one launch per
    pass, every chunk on the dense-diagonal path -- with the oracle on two whole trees x three heads."""
    from workloads import CONFIGS
    fo = config_forest("cfg2")
    heads, d = CONFIGS["cfg2"]["H"], 128
    inp = make_inputs(fo.n_tokens, heads, d, d, "bf16", 21, device="cuda")
    inp["g"] = make_gk(fo.n_tokens, heads, d, 21, device="cuda")
    plan = plan_of(fo).upload()
    phys = to_physical(plan, inp)
    cs_bytes, sc_bytes = H.harts_la_gk_workspace_bytes(plan.tables, heads, d, d, 1)
    slots = torch.full((max(plan.n_slots, 1) * heads * d * d,), float("nan"), device="cuda")
    cs = torch.empty(cs_bytes, dtype=torch.uint8, device="cuda")
    scratch = torch.empty(sc_bytes, dtype=torch.uint8, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    out = {n: torch.full_like(phys[m], float("nan")) for n, m in (("o", "v"), ("dq", "q"), ("dk", "k"), ("dv", "v"), ("dg", "g"))}
    H.harts_la_gk_fwd(plan, 0, phys["q"], phys["k"], phys["v"], phys["g"], out["o"], slots, cs, dev_status=status)
    H.harts_la_gk_bwd(plan, 0, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"], out["dq"], out["dk"], out["dv"],
                      out["dg"], cs, scratch, dev_status=status)
    H.harts_la_check(status)
    rows = torch.as_tensor(plan.row_of_token.astype(np.int64), device="cuda")
    trees, hs = [1, 6], [0, heads // 2, heads - 1]
    base = fo.token_base()
    tok = np.concatenate([np.arange(base[fo.tree_node_ptr[t]], base[fo.tree_node_ptr[t + 1]]) for t in trees])
    sub = fo.subset(trees)
    ti, hi = torch.as_tensor(tok, device="cuda"), torch.as_tensor(hs, device="cuda")
    pick = {n: x[ti][:, hi].cpu() for n, x in inp.items()}
    ref = go.forest_eval(sub, pick["q"], pick["k"], pick["v"], pick["g"], pick["dO"])
    errs = {}
    for n, x in out.items():
        assert torch.isfinite(x.float()).all(), n
        got = x[rows][ti][:, hi].float().cpu().numpy()
        errs[n] = rel_err(got, ref[n])
        errs[n + ".row"] = row_err(got, ref[n])
    print("cfg2 gk", errs)
    check(errs, "bf16")


def test_tensor_core_path_agrees_with_the_cuda_core_path():
    """bf16, d = 128: the same call with HARTS_FLAG_FMA_KERNELS runs the CUDA-core kernels (pair sums over whole
    chunks, no anchored operands, fp32 products).  Two different decompositions of the same sums, same bf16 roundings of
    the inputs and states: they must agree to within the oracle tolerance (each is within it of the oracle, so twice of it is what the triangle
    inequality alone would give), on forests with several rounds, shared
    slots and replayed rows, three heads, with strongly decaying channels mixed in."""
    import random
    from test_plan_oracle import random_tree
    rnd = random.Random(17)
    forests = [config_forest("cfg0b"), config_forest("cfg1")]
    forests += [make_forest([random_tree(rnd, rnd.randint(2, 12), rnd.choice([40, 200, 600])) for _ in range(2)])
                for _ in range(4)]
    for n, fo in enumerate(forests):
        heads = 1 if fo.n_tokens > 10000 else 3
        _, tc = run_gk(fo, heads, 128, "bf16", 50 + n, strong_every=8 * (n % 2), raw=True)
        _, cc = run_gk(fo, heads, 128, "bf16", 50 + n, strong_every=8 * (n % 2), raw=True, flags=H.HARTS_FLAG_FMA_KERNELS)
        for name in tc:
            assert rel_err(tc[name], cc[name]) <= 1.0 * TOL["bf16"][name], (n, name, rel_err(tc[name], cc[name]))


def test_all_rounds_in_one_launch_give_the_bits_of_one_launch_per_round():
    """bf16, d = 128, several rounds: round 0 runs all rounds in one launch per pass (tickets and flags between the
    CTAs); with HARTS_FLAG_ROUND_LAUNCHES every round is a launch of its own.  Same arithmetic, same bits -- on forests
    with shared slots, replayed rows and three rounds, two heads."""
    import random
    from test_plan_oracle import random_tree
    rnd = random.Random(23)
    forests = [config_forest("cfg0b"), config_forest("cfg1")]
    forests += [make_forest([random_tree(rnd, rnd.randint(3, 14), rnd.choice([40, 200, 700])) for _ in range(rnd.randint(1, 3))])
                for _ in range(8)]
    multi = 0
    for n, fo in enumerate(forests):
        plan, one = run_gk(fo, 2, 128, "bf16", 70 + n, raw=True)
        _, per = run_gk(fo, 2, 128, "bf16", 70 + n, raw=True, flags=H.HARTS_FLAG_ROUND_LAUNCHES)
        for name in one:
            assert np.array_equal(one[name], per[name]), (n, name)
        multi += int(plan.n_rounds > 1)
    assert multi >= 6


def test_equal_channels_agree_with_the_scalar_gate_kernels():
    """With every channel's gate equal, the per-channel kernels and the scalar-gate fp32 kernels compute the same
    function (different code): outputs within fp32 accumulation error of each other."""
    fo = config_forest("cfg0b")
    inp = make_inputs(fo.n_tokens, 1, 64, 64, "fp32", 9)
    plan = plan_of(fo).upload()
    phys = to_physical(plan, inp)
    ws = H.Workspace(plan, 1, 64, 64, torch.float32)
    ref = H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
    gk = phys["g"][:, :, None].expand(-1, -1, 64).contiguous()
    cs_bytes, sc_bytes = H.harts_la_gk_workspace_bytes(plan.tables, 1, 64, 64, 0)
    slots = torch.zeros(max(plan.n_slots, 1) * 64 * 64, device="cuda")
    cs = torch.empty(cs_bytes, dtype=torch.uint8, device="cuda")
    scratch = torch.empty(sc_bytes, dtype=torch.uint8, device="cuda")
    o, dq, dk, dv = (torch.empty_like(phys[n]) for n in ("v", "q", "k", "v"))
    dgk = torch.empty_like(gk)
    H.harts_la_gk_fwd(plan, 0, phys["q"], phys["k"], phys["v"], gk, o, slots, cs)
    H.harts_la_gk_bwd(plan, 0, phys["q"], phys["k"], phys["v"], gk, phys["dO"], dq, dk, dv, dgk, cs, scratch)
    torch.cuda.synchronize()
    for a, b in ((o, ref["o"]), (dq, ref["dq"]), (dk, ref["dk"]), (dv, ref["dv"]), (dgk.sum(dim=2), ref["dg"])):
        assert rel_err(a.cpu().numpy(), b.cpu().numpy()) <= 1e-4


def test_unsupported_shapes_are_refused():
    fo = config_forest("cfg0")
    plan = plan_of(fo).upload()
    q = torch.zeros(plan.C, 1, 96, device="cuda")
    with pytest.raises(H.HartsError) as e:
        H.harts_la_gk_fwd(plan, 0, q, q, q, q, torch.empty_like(q), torch.zeros(16, device="cuda"), None)
    assert e.value.code == -3
    torch.cuda.synchronize()
