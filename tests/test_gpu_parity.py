"""GPU parity: the CUDA path (through the C ABI) against the fp64 trajectory-wise oracle, element
by element on the same seeded inputs.  Tolerances (relative Frobenius error per tensor): bf16
inputs with fp32 accumulation 5e-3 for outputs and 1e-2 for gradients; the fp32 configuration is
held to 1e-4 (fp32 accumulation over 64-row chunks plus the fast exponential)."""
import numpy as np
import pytest
import torch

import paper_2608_28158_b200 as H
from workloads import make_forest, make_inputs
from parity_util import compare, config_case, oracle_subset, plan_of, rel_err, run_gpu, to_physical

pytestmark = pytest.mark.gpu

TOL = {"fp32": dict(o=1e-4, dq=1e-4, dk=1e-4, dv=1e-4, dg=1e-4),
       "bf16": dict(o=5e-3, dq=1e-2, dk=1e-2, dv=1e-2, dg=1e-2)}


# Besides the Frobenius tolerance per tensor, every single (token, head) row is held to ROW_MULT times that tolerance (observed worst rows: 0.9x for o, 0.5x for dq, dk, dv, 1.5x for dg)
# (relative to the larger of its own norm and the tensor's RMS row norm): the Frobenius error is an RMS over rows, the
# worst of 10^5..10^6 rows of independent bf16 roundings lies a few standard deviations above it.
ROW_MULT = 2.0


def check(errs, dtype):
    for n, e in errs.items():
        base = n.split(".")[0]
        assert e <= TOL[dtype][base] * (ROW_MULT if n.endswith(".row") else 1.0), (n, e, errs)


@pytest.mark.parametrize("name", ["cfg0", "cfg0b", "cfg1"])
def test_small_configs_full_parity(name):
    cfg, fo, inp = config_case(name)
    plan, out = run_gpu(fo, inp)
    tok, ref = oracle_subset(fo, inp, list(range(fo.n_trees)), list(range(cfg["H"])))
    assert ref["copy_gap"] < 1e-9
    errs = compare(out, tok, list(range(cfg["H"])), ref, rows=True)
    print(name, errs)
    check(errs, cfg["dtype"])


@pytest.mark.parametrize("name,trees", [("cfg2", [0, 5]), ("cfg3", [3, 17, 31]), ("cfg4", [0, 63])])
def test_large_configs_sampled_parity(name, trees):
    # full-size launch on the GPU; the oracle evaluates whole trees for three heads
    cfg, fo, inp = config_case(name, device="cuda")
    plan, out = run_gpu(fo, inp)
    heads = [0, cfg["H"] // 2, cfg["H"] - 1]
    tok, ref = oracle_subset(fo, inp, trees, heads)
    errs = compare(out, tok, heads, ref, rows=True)
    print(name, "C", plan.C, "R", plan.R, "rounds", plan.n_rounds, "seqs", plan.n_seq, errs)
    check(errs, cfg["dtype"])
    for x in out.values():
        assert torch.isfinite(x.float()).all()


@pytest.mark.parametrize("name", ["cfg0", "cfg0b", "cfg1"])
def test_compact_equals_trajectory_wise_on_gpu(name):
    # same kernels on the expanded forest (one zero-state sequence per leaf): outputs at m(s) agree.
    cfg, fo, inp = config_case(name)
    _, out = run_gpu(fo, inp, backward=False)
    (ptr, par, off, ln), src = H.expand_trajectories(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len)
    src_t = torch.as_tensor(src)
    exp_inp = {n: x[src_t] for n, x in inp.items()}
    exp_fo = make_forest([([-1], [0], [int(l)]) for l in ln])
    _, exp_out = run_gpu(exp_fo, exp_inp, backward=False)
    a = exp_out["o"].float().cpu().numpy()
    b = out["o"][src_t.cuda()].float().cpu().numpy()
    # the chunk grid of a replay-started branch coincides with the trajectory's own grid and the exported boundary
    # states are exact fp32 copies, so the two runs take the same floating-point path
    print(name, "compact vs trajectory-wise: max abs diff", float(np.abs(a - b).max()), "rel", rel_err(a, b))
    assert np.array_equal(a, b)


def edge_forests():
    return {
        "one_token": make_forest([([-1], [0], [1])]),
        "exact_chunk": make_forest([([-1, 0, 0], [0, 64, 64], [64, 64, 1])]),
        "two_chunks_and_tail": make_forest([([-1, 0, 0, 2], [0, 128, 100, 63], [129, 5, 200, 64])]),
        "many_tiny": make_forest([([-1] + [0] * 40, [0] + [1 + (7 * i) % 90 for i in range(40)],
                                   [90] + [1 + i % 5 for i in range(40)])] * 3),
        "nested_in_chunk": make_forest([([-1, 0, 1, 2, 3, 0], [0, 10, 5, 3, 2, 10], [10, 7, 6, 4, 70, 130])]),
    }


@pytest.mark.parametrize("case", list(edge_forests()))
@pytest.mark.parametrize("dtype,d", [("fp32", 64), ("bf16", 128)])
def test_edge_cases(case, dtype, d):
    fo = edge_forests()[case]
    inp = make_inputs(fo.n_tokens, 2, d, d, dtype, 17)
    plan, out = run_gpu(fo, inp)
    tok, ref = oracle_subset(fo, inp, list(range(fo.n_trees)), [0, 1])
    errs = compare(out, tok, [0, 1], ref, rows=True)
    print(case, dtype, errs)
    check(errs, dtype)


def random_forest_cases(n_cases=36, seed=2024):
    """Seeded forests of the kinds that random testing needs to meet: forks nested inside one chunk, replay spans that
    cross several ancestor segments, several consumers of one exported state, chains of short branches, long roots."""
    import random
    from test_plan_oracle import random_tree
    rnd = random.Random(seed)
    cases = []
    for i in range(n_cases):
        max_len = rnd.choice([5, 40, 70, 200, 700])
        trees = [random_tree(rnd, rnd.randint(1, 12), max_len) for _ in range(rnd.randint(1, 4))]
        cases.append((make_forest(trees), rnd.choice([1, 2, 3, 4]), 500 + i))
    return cases


def test_random_forests_through_the_tensor_core_kernels():
    """36 seeded random forests (1-4 heads, bf16, d = 128: the tcgen05 kernels) against the oracle, per tensor and
    per row; also checks that the set covers the structures it is meant to cover."""
    nested = multi_seg_replay = shared_slot = multi_round = 0
    for fo, heads, seed in random_forest_cases():
        inp = make_inputs(fo.n_tokens, heads, 128, 128, "bf16", seed)
        plan, out = run_gpu(fo, inp)
        tok, ref = oracle_subset(fo, inp, list(range(fo.n_trees)), list(range(heads)))
        errs = compare(out, tok, list(range(heads)), ref, rows=True)
        check(errs, "bf16")
        rp = np.diff(plan.seq_replay_ptr)
        for i in np.nonzero(rp > 0)[0]:
            r = plan.replay_row[plan.seq_replay_ptr[i]:plan.seq_replay_ptr[i + 1]]
            multi_seg_replay += int((np.diff(r) != 1).any())          # replayed rows from more than one row range
        nested += int((np.diff(plan.rg_ptr) > 1).any())               # a row replayed by several sequences
        shared_slot += int((np.diff(plan.slot_cons_ptr) > 1).any())
        multi_round += int(plan.n_rounds >= 3)
    print("coverage:", nested, multi_seg_replay, shared_slot, multi_round)
    assert nested >= 5 and multi_seg_replay >= 5 and shared_slot >= 5 and multi_round >= 2


def test_all_rounds_in_one_launch_give_the_bits_of_one_launch_per_round():
    """Problems with few (sequence, head) items per CTA run all rounds in one launch: the CTAs draw the
    items from a ticket counter and the sequences wait for each other through flags instead of kernel boundaries.  Outputs, gradients, exported states
    and chunk states must equal, bit for bit, those of one launch per round -- on forests with several consumers per
    boundary, replayed first chunks and three rounds."""
    import random
    from test_plan_oracle import random_tree
    rnd = random.Random(3)
    # cfg2 x 16 heads: 1,104 items, several per CTA (the ticket counter and the per-item flags at work)
    cases = [(config_case("cfg1")[1], 1, 5), (config_case("cfg2")[1], 16, 6)]
    cases += [(make_forest([random_tree(rnd, rnd.randint(3, 14), rnd.choice([40, 200, 700])) for _ in range(rnd.randint(1, 3))]),
               rnd.choice([1, 2]), 60 + i) for i in range(14)]
    one_launch = shared = 0
    for fo, heads, seed in cases:
        inp = make_inputs(fo.n_tokens, heads, 128, 128, "bf16", seed)
        plan = plan_of(fo).upload()
        phys = to_physical(plan, inp)
        got = {}
        for name, flags in (("rounds", H.HARTS_FLAG_ROUND_LAUNCHES), ("one", 0)):
            ws = H.Workspace(plan, heads, 128, 128, phys["q"].dtype, flags)
            ws.slots.fill_(float("nan"))
            ws.chunk_states.zero_()
            out = H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
            H.harts_la_check(ws.dev_status)
            n_state = plan.n_chunks * heads * 128 * 128 * 2
            got[name] = dict(out, slots=ws.slots[:plan.n_slots * heads * 128 * 128].clone(),
                             states=ws.chunk_states[:n_state].clone())
        for n in got["one"]:
            assert torch.equal(got["one"][n], got["rounds"][n]), (n, fo.n_tokens, heads)
        if 1 < plan.n_rounds <= 32 and plan.n_seq * heads <= 8 * 148:
            one_launch += 1
            shared += int((np.diff(plan.slot_cons_ptr) > 1).any())
    assert one_launch >= 8 and shared >= 3, (one_launch, shared)


def test_rounds_issued_one_by_one_match_round_zero():
    cfg, fo, inp = config_case("cfg0b")
    plan = plan_of(fo).upload()
    phys = to_physical(plan, inp)
    ws = H.Workspace(plan, 1, 64, 64, torch.float32)
    ref = H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
    ref = {n: x.clone() for n, x in ref.items()}
    ws2 = H.Workspace(plan, 1, 64, 64, torch.float32)
    o = torch.zeros_like(phys["v"])
    dq, dk, dv, dg = (torch.zeros_like(phys[n]) for n in ("q", "k", "v", "g"))
    for r in range(1, plan.n_rounds + 1):
        H.harts_la_fwd(plan, r, phys["q"], phys["k"], phys["v"], phys["g"], o, ws2.slots, ws2.chunk_states)
    for r in range(plan.n_rounds, 0, -1):
        H.harts_la_bwd(plan, r, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"], dq, dk, dv, dg,
                       ws2.chunk_states, ws2.scratch)
    torch.cuda.synchronize()
    for n, x in (("o", o), ("dq", dq), ("dk", dk), ("dv", dv), ("dg", dg)):
        assert torch.equal(x, ref[n]), n


def test_hand_built_tables_drive_one_packed_call():
    # Eq. 16 without the planner: two sequences in one call, the second starts from a caller-provided state in a slot
    # and the first exports its boundary after chunk 0 into another slot.
    import ctypes
    H_, d, n0, n1 = 2, 128, 150, 70
    inp = make_inputs(n0 + n1, H_, d, d, "bf16", 23)
    dev = {n: x.cuda() for n, x in inp.items()}
    i32 = lambda *v: torch.tensor(v, dtype=torch.int32, device="cuda")  # noqa: E731
    arrays = dict(seq_own_begin=i32(0, n0, n0 + n1), seq_init_slot=i32(-1, 1), seq_replay_ptr=i32(0, 0, 0),
                  replay_row=i32(0), seq_req_ptr=i32(0, 1, 1), slot_chunk=i32(1), seq_chunk_ptr=i32(0, 3, 5),
                  slot_cons_ptr=i32(0, 0), slot_cons_seq=i32(0), rg_row=i32(0), rg_ptr=i32(0), rg_entry=i32(0))
    tb = H.binding.Tables()
    tb.chunk, tb.n_rows, tb.n_replay, tb.n_seq, tb.n_slots, tb.n_chunks, tb.n_rg_rows = 64, n0 + n1, 0, 2, 2, 5, 0
    for n, a in arrays.items():
        setattr(tb, n, a.data_ptr())
    S0 = torch.randn(H_, d, d, device="cuda") * 0.1
    slots = torch.zeros(2, H_, d, d, device="cuda")
    slots[1] = S0
    o = torch.empty_like(dev["v"])
    H.harts_la_fwd_seqs(tb, 0, 2, dev["q"], dev["k"], dev["v"], dev["g"], o, slots, None)
    torch.cuda.synchronize()
    # fp64 token recurrence for both sequences
    q, k, v, g = (inp[n].double().numpy() for n in ("q", "k", "v", "g"))
    ref = np.zeros((n0 + n1, H_, d))
    S = np.zeros((H_, d, d))
    for t in range(n0):
        if t == 64:
            exported = S.copy()
        S = np.exp(g[t])[:, None, None] * S + k[t][:, :, None] * v[t][:, None, :]
        ref[t] = np.einsum("hi,hij->hj", q[t], S)
    S = S0.double().cpu().numpy()
    for t in range(n0, n0 + n1):
        S = np.exp(g[t])[:, None, None] * S + k[t][:, :, None] * v[t][:, None, :]
        ref[t] = np.einsum("hi,hij->hj", q[t], S)
    assert rel_err(o.float().cpu().numpy(), ref) < 5e-3
    assert rel_err(slots[0].cpu().numpy(), exported) < 5e-3


def test_bad_hand_built_tables_are_caught_on_the_device_and_nothing_is_dereferenced():
    """HARTS_FLAG_CHECK_TABLES: a replay row far outside the tensors, an initial-state slot that does not exist, a
    boundary request past the sequence's end.  The validation kernel records HARTS_EINVAL, the kernels of the call do
    not run (the outputs keep their fill value), nothing faults; the same tables without the mistake pass the check
    and give the bits of an unchecked run."""
    H_, d, n0, n1 = 2, 128, 150, 70
    inp = make_inputs(n0 + n1, H_, d, d, "bf16", 23)
    dev = {n: x.cuda() for n, x in inp.items()}
    i32 = lambda *v: torch.tensor(v, dtype=torch.int32, device="cuda")  # noqa: E731

    def tables(replay_row=5, init_slot=0, slot_chunk=1):
        # sequence 0: 150 rows from the zero state, exports the state after its first chunk into slot 0;
        # sequence 1: replays row `replay_row`, then its 70 own rows, from slot `init_slot`
        arrays = dict(seq_own_begin=i32(0, n0, n0 + n1), seq_init_slot=i32(-1, init_slot), seq_replay_ptr=i32(0, 0, 1),
                      replay_row=i32(replay_row), seq_req_ptr=i32(0, 1, 1), slot_chunk=i32(slot_chunk),
                      seq_chunk_ptr=i32(0, 3, 5), slot_cons_ptr=i32(0, 1), slot_cons_seq=i32(1), rg_row=i32(5),
                      rg_ptr=i32(0, 1), rg_entry=i32(0))
        tb = H.binding.Tables()
        tb.chunk, tb.n_rows, tb.n_replay, tb.n_seq, tb.n_slots, tb.n_chunks, tb.n_rg_rows = 64, n0 + n1, 1, 2, 1, 5, 1
        for n, a in arrays.items():
            setattr(tb, n, a.data_ptr())
        return tb, arrays

    def forward(tb, flags):
        status = torch.zeros(4, dtype=torch.int32, device="cuda")
        slots = torch.zeros(1, H_, d, d, device="cuda")
        o = torch.full_like(dev["v"], 7.0)
        H.harts_la_fwd_seqs(tb, 0, 1, dev["q"], dev["k"], dev["v"], dev["g"], o, slots, None, flags, status)
        H.harts_la_fwd_seqs(tb, 1, 2, dev["q"], dev["k"], dev["v"], dev["g"], o, slots, None, flags, status)
        return o, status

    good, keep = tables()
    o_ref, st = forward(good, 0)
    H.harts_la_check(st)
    o_chk, st = forward(good, H.HARTS_FLAG_CHECK_TABLES)
    H.harts_la_check(st)
    assert torch.equal(o_ref, o_chk)
    for kwargs, table in ((dict(replay_row=10 ** 9), 4), (dict(init_slot=3), 2), (dict(slot_chunk=3), 6)):
        bad, keep = tables(**kwargs)
        o, st = forward(bad, H.HARTS_FLAG_CHECK_TABLES)
        with pytest.raises(H.HartsError) as e:
            H.harts_la_check(st)
        assert e.value.code == -1 and int(st[1]) == table, (kwargs, st.tolist())
        # the call that held the bad entry, and every later call on this status word, left the outputs alone
        lo_ = 0 if table == 6 else n0
        assert bool((o[lo_:] == 7.0).all())
    torch.cuda.synchronize()


def test_errors_are_reported_without_launching():
    cfg, fo, inp = config_case("cfg0")
    plan = plan_of(fo).upload()
    phys = to_physical(plan, inp)
    ws = H.Workspace(plan, 1, 64, 64, torch.float32)
    o = torch.empty_like(phys["v"])
    # misaligned pointer
    bad = torch.empty(phys["q"].numel() + 1, dtype=torch.float32, device="cuda")[1:].view_as(phys["q"])
    with pytest.raises(H.HartsError) as e:
        H.harts_la_fwd(plan, 0, bad, phys["k"], phys["v"], phys["g"], o, ws.slots, ws.chunk_states)
    assert e.value.code == -1
    # unsupported head dimension
    q96 = torch.zeros(plan.C, 1, 96, device="cuda")
    with pytest.raises(H.HartsError) as e:
        H.harts_la_fwd(plan, 0, q96, q96, q96, phys["g"], torch.empty_like(q96), ws.slots, ws.chunk_states)
    assert e.value.code == -3
    # round out of range
    with pytest.raises(H.HartsError) as e:
        H.harts_la_fwd(plan, 9, phys["q"], phys["k"], phys["v"], phys["g"], o, ws.slots, ws.chunk_states)
    assert e.value.code == -1
    torch.cuda.synchronize()


def test_repeated_runs_are_bit_identical():
    """No float atomics anywhere: hand-off gradients and replayed-row gradients are summed in table order, so every
    run of the same plan on the same inputs gives the same bits.  A race between the kernels' warp roles (MMA issue,
    TMA, row preparation, element-wise passes) would show up as a run that differs."""
    import random
    from test_plan_oracle import random_tree
    rnd = random.Random(77)
    forests = [config_case("cfg2")[1]]
    forests += [make_forest([random_tree(rnd, rnd.randint(3, 40), rnd.choice([100, 700, 3000])) for _ in range(rnd.randint(1, 6))])
                for _ in range(4)]
    for k, fo in enumerate(forests):
        Hh = 16 if k == 0 else rnd.choice([1, 2, 4])
        inp = make_inputs(fo.n_tokens, Hh, 128, 128, "bf16", 40 + k)
        plan = plan_of(fo).upload()
        phys = to_physical(plan, inp)
        ws = H.Workspace(plan, Hh, 128, 128, phys["q"].dtype, 0)
        first = None
        for _ in range(12):
            out = H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
            H.harts_la_check(ws.dev_status)
            if first is None:
                first = {n: x.clone() for n, x in out.items()}
                assert all(bool(torch.isfinite(x.float()).all()) for x in first.values())
            else:
                for n in out:
                    assert torch.equal(out[n], first[n]), (k, n)


def test_a_whole_step_can_be_captured_in_a_cuda_graph():
    """The calls only enqueue work on the caller's stream (no allocation, no synchronisation), so all rounds of a
    forward+backward step can be captured once and replayed; the replay gives the same bits as the eager step."""
    cfg, fo, inp = config_case("cfg1")
    plan = plan_of(fo).upload()
    phys = to_physical(plan, inp)
    ws = H.Workspace(plan, cfg["H"], cfg["dk"], cfg["dv"], phys["q"].dtype, 0)
    out = H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
    ref = {n: x.clone() for n, x in out.items()}
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"], out=out, stream=s)   # warm-up
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=s):
            H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"], out=out, stream=s)
    torch.cuda.synchronize()
    for x in out.values():
        x.zero_()
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    H.harts_la_check(ws.dev_status)
    for n in out:
        assert torch.equal(out[n], ref[n]), n
