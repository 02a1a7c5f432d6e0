"""GPU parity of the compact-to-semantic log-probability (Eqs. 17, 19) through the C ABI against the fp64 oracle.

Tolerances: lse and lambda are fp32 results of an fp32 sum over V terms with ex2/lg2 approximations of relative
error 2^-22: |error| <= 2e-5 absolute on values of magnitude ~10-20.  dz is rounded once to the logit dtype:
relative Frobenius error <= 5e-3 for bf16 (one rounding, 2^-9 at most per element) and 1e-5 for fp32."""
import numpy as np
import pytest
import torch

import paper_2608_28158_b200 as H
from oracle import logp_oracle as lo
from workloads import config_forest, make_forest, make_logits, make_logp_grad

pytestmark = pytest.mark.gpu
DZ_TOL = {"bf16": 5e-3, "fp32": 1e-5}


def _dev(a, dtype=None):
    return torch.as_tensor(np.ascontiguousarray(a)).to("cuda", dtype=dtype)


def _run(z_dev, m, y, g, n_rows, V, with_status=True):
    """z_dev [n_rows, ld] device (may be a strided view); m, y host int32; g host fp32.  Returns lse, lambda, dz."""
    md, yd = _dev(m, torch.int32), _dev(y, torch.int32)
    lse = torch.full((n_rows,), float("nan"), device="cuda")
    lam = torch.full((len(m),), float("nan"), device="cuda")
    status = torch.zeros(2, dtype=torch.int32, device="cuda") if with_status else None
    H.harts_logp_fwd(z_dev, md, yd, lse, lam, V=V, dev_status=status)
    ptr, pos = H.harts_logp_csr(n_rows, m)
    dz = torch.full_like(z_dev, float("nan"))
    H.harts_logp_bwd(z_dev, yd, _dev(ptr), _dev(pos), lse, _dev(g, torch.float32), dz, V=V, dev_status=status)
    if with_status:
        H.harts_la_check(status)
    torch.cuda.synchronize()
    return lse, lam, dz


def _rel(x, ref, g):
    """Relative Frobenius error of dz.  Every term of Eq. 19 is g_s times an O(1) factor, so ||g|| is the scale
    the error is held to when the terms cancel (V = 1: onehot - softmax = 0 exactly)."""
    return float(np.linalg.norm(x - ref) / max(np.linalg.norm(ref), np.linalg.norm(g), 1e-30))


def _forest_case(name, V, dtype, seed):
    fo = config_forest(name) if isinstance(name, str) else name
    C = fo.n_tokens
    data = make_logits(C, V, dtype, seed)
    plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64)
    rot = plan.row_of_token.astype(np.int64)
    tok = data["token_id"].numpy()
    m, y, _ = H.harts_logp_positions(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, tok,
                                     plan.row_of_token)
    m0, y0, _ = lo.positions(fo, tok)
    g = make_logp_grad(len(m), seed).numpy()
    z_phys = torch.empty_like(data["z"])
    z_phys[torch.as_tensor(rot)] = data["z"]
    return fo, data["z"].double().numpy(), z_phys.cuda(), rot, (m, y), (m0, y0), g


@pytest.mark.parametrize("name,V,dtype", [("cfg0", 1000, "bf16"), ("cfg0b", 4104, "bf16"), ("cfg0", 1000, "fp32"),
                                          ("cfg0b", 157184, "bf16")])
def test_tree_parity(name, V, dtype):
    fo, z64, z_dev, rot, (m, y), (m0, y0), g = _forest_case(name, V, dtype, 3)
    lse, lam, dz = _run(z_dev, m, y, g, fo.n_tokens, V)
    lam_ref, lse_ref = lo.mapped_logp(z64, m0, y0)
    dz_ref = lo.mapped_logp_grad(z64, m0, y0, g.astype(np.float64))
    assert np.abs(lse.cpu().numpy()[rot] - lse_ref).max() <= 2e-5
    assert np.abs(lam.cpu().numpy() - lam_ref).max() <= 2e-5
    got = dz.float().cpu().numpy().astype(np.float64)[rot]
    assert _rel(got, dz_ref, g) <= DZ_TOL[dtype]
    # rows that no active position reuses are exactly zero
    idle = np.ones(fo.n_tokens, bool)
    idle[m0[g != 0]] = False
    assert not got[idle].any() and not dz_ref[idle].any()


@pytest.mark.parametrize("dtype,V,ld,shift", [("bf16", 1003, 1003, 0), ("bf16", 1003, 1008, 3), ("fp32", 1001, 1001, 0),
                                              ("bf16", 5, 5, 1), ("fp32", 1, 1, 0), ("bf16", 2051, 2064, 0)])
def test_ragged_rows_and_misaligned_starts(dtype, V, ld, shift):
    """Any V, any row stride, any starting offset: the scalar head and tail paths and the unaligned z/dz pair."""
    rng = np.random.default_rng(7)
    C, P = 37, 90
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    store = torch.zeros(C * ld + 16, dtype=dt)
    z = store[shift:shift + C * ld].view(C, ld)
    z[:, :V] = make_logits(C, V, dtype, 5)["z"]
    m = rng.integers(0, C, P).astype(np.int32)
    y = rng.integers(0, V, P).astype(np.int32)
    g = make_logp_grad(P, 1).numpy()
    sd = store.cuda()
    z_dev = sd[shift:shift + C * ld].view(C, ld)
    lse, lam, dz = _run(z_dev, m, y, g, C, V)
    z64 = z[:, :V].double().numpy()
    lam_ref, lse_ref = lo.mapped_logp(z64, m, y)
    dz_ref = lo.mapped_logp_grad(z64, m, y, g.astype(np.float64))
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 2e-5
    assert np.abs(lam.cpu().numpy() - lam_ref).max() <= 2e-5
    assert _rel(dz[:, :V].float().cpu().numpy().astype(np.float64), dz_ref, g) <= DZ_TOL[dtype]


def test_shared_targets_masked_words_and_idle_rows():
    """Several positions with the same (row, target); -inf logits (masked words); a row whose positions all have
    g = 0; a row nobody reuses; no positions at all."""
    V, C = 520, 6
    z = make_logits(C, V, "bf16", 9)["z"]
    z[1, 100:300] = float("-inf")
    m = np.array([0, 0, 0, 1, 1, 2, 2, 4, 4, 4], np.int32)
    y = np.array([7, 7, 9, 5, 5, 1, 2, 519, 519, 0], np.int32)
    g = np.array([0.5, -0.25, 1.0, 2.0, 1.0, 0.0, 0.0, 1.0, -1.0, 0.0], np.float32)
    lse, lam, dz = _run(z.cuda(), m, y, g, C, V)
    z64 = z.double().numpy()
    zf = np.clip(z64, -500, None)                           # exp(-500) ~ 1e-217 stands in for exp(-inf) = 0
    lam_ref, lse_ref = lo.mapped_logp(zf, m, y)
    dz_ref = lo.mapped_logp_grad(zf, m, y, g.astype(np.float64))
    got = dz.float().cpu().numpy().astype(np.float64)
    assert np.abs(lse.cpu().numpy() - lse_ref).max() <= 2e-5 and np.abs(lam.cpu().numpy() - lam_ref).max() <= 2e-5
    assert _rel(got, dz_ref, g) <= 5e-3
    assert not got[2].any() and not got[3].any() and not got[5].any()
    assert not got[1, 100:300].any()                         # masked words get no gradient
    # row 4: the two weights on word 519 cancel, w = 0: the row is all zeros although it was processed
    assert not got[4].any()
    lse0, lam0, dz0 = _run(z.cuda(), np.zeros(0, np.int32), np.zeros(0, np.int32), np.zeros(0, np.float32), C, V)
    assert lam0.numel() == 0 and not dz0.float().cpu().numpy().any()
    assert np.abs(lse0.cpu().numpy() - lse_ref).max() <= 2e-5


def test_vocabulary_shards_combine_to_the_unsharded_result():
    """Three uneven shards (one starting off a 16-byte boundary) emulate vocabulary-parallel ranks on one GPU:
    only per-row (max, sum) and per-position target scalars are combined."""
    fo, z64, z_dev, rot, (m, y), (m0, y0), g = _forest_case("cfg0", 3000, "bf16", 4)
    C, V = fo.n_tokens, 3000
    md, yd = _dev(m, torch.int32), _dev(y, torch.int32)
    cuts = [0, 1003, 2200, 3000]
    K = len(cuts) - 1
    rmax = torch.empty(K, C, device="cuda"); rsum = torch.empty(K, C, device="cuda")
    tgt = torch.empty(K, len(m), device="cuda")
    for k in range(K):
        H.harts_logp_fwd_shard(z_dev[:, cuts[k]:cuts[k + 1]], cuts[k], md, yd, rmax[k], rsum[k], tgt[k])
    lse = torch.empty(C, device="cuda"); lam = torch.empty(len(m), device="cuda")
    H.harts_logp_combine(K, C, md, rmax, rsum, tgt, lse, lam)
    lam_ref, lse_ref = lo.mapped_logp(z64, m0, y0)
    assert np.abs(lse.cpu().numpy()[rot] - lse_ref).max() <= 2e-5
    assert np.abs(lam.cpu().numpy() - lam_ref).max() <= 2e-5
    # backward per shard writes that shard's columns of the same dz
    ptr, pos = H.harts_logp_csr(C, m)
    dz = torch.full_like(z_dev, float("nan"))
    for k in range(K):
        H.harts_logp_bwd(z_dev[:, cuts[k]:cuts[k + 1]], yd, _dev(ptr), _dev(pos), lse, _dev(g), dz[:, cuts[k]:cuts[k + 1]],
                         v_begin=cuts[k], V_total=V)
    dz_ref = lo.mapped_logp_grad(z64, m0, y0, g.astype(np.float64))
    assert _rel(dz.float().cpu().numpy().astype(np.float64)[rot], dz_ref, g) <= 5e-3


def test_bad_indices_are_reported_not_dereferenced():
    z = make_logits(4, 64, "bf16", 0)["z"].cuda()
    m = np.array([0, 9, 1], np.int32); y = np.array([3, 3, 64], np.int32)
    lse = torch.empty(4, device="cuda"); lam = torch.empty(3, device="cuda")
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    H.harts_logp_fwd(z, _dev(m), _dev(y), lse, lam, dev_status=status)
    with pytest.raises(H.HartsError):
        H.harts_la_check(status)
    assert lam.cpu().numpy()[1] == 0 and lam.cpu().numpy()[2] == 0
    with pytest.raises(H.HartsError):                        # V < 1
        H.harts_logp_fwd(z, _dev(m), _dev(y), lse, lam, V=0)
    with pytest.raises(H.HartsError):                        # dz aliases z
        ptr, pos = H.harts_logp_csr(4, np.array([0], np.int32))
        H.harts_logp_bwd(z, _dev(y[:1]), _dev(ptr), _dev(pos), lse, lam[:1], z)


def test_full_size_sampled_rows():
    """The benchmark's workload and launch configuration (about 60k compact rows x 157,184 words): rows sampled
    over the whole range, those with the most positions included, are checked one by one against the oracle."""
    from bench import LOGP_V, logp_forest
    fo, _ = logp_forest(0)
    C, V = fo.n_tokens, LOGP_V
    data = make_logits(C, V, "bf16", 50, device="cuda")
    plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64)
    m, y, _ = H.harts_logp_positions(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len,
                                     data["token_id"].cpu().numpy(), plan.row_of_token)
    g = make_logp_grad(len(m), 50, device="cuda", keep=0.6)
    z = data["z"]
    lse, lam, dz = _run(z, m, y, g.cpu().numpy(), C, V)
    ptr, pos = H.harts_logp_csr(C, m)
    count = np.diff(ptr)
    rows = np.unique(np.concatenate([np.argsort(count)[-6:], np.linspace(0, C - 1, 18).astype(np.int64)]))
    gh = g.cpu().numpy().astype(np.float64)
    lam_h = lam.cpu().numpy()
    for c in rows:
        zc = z[c].double().cpu().numpy()[None, :]
        s_ids = pos[ptr[c]:ptr[c + 1]]
        mm = np.zeros(len(s_ids), np.int64)
        lam_ref, lse_ref = lo.mapped_logp(zc, mm, y[s_ids])
        dz_ref = lo.mapped_logp_grad(zc, mm, y[s_ids], gh[s_ids])
        assert abs(float(lse[c]) - lse_ref[0]) <= 2e-5
        assert len(s_ids) == 0 or np.abs(lam_h[s_ids] - lam_ref).max() <= 2e-5
        got = dz[c].double().cpu().numpy()[None, :]
        assert _rel(got, dz_ref, gh[s_ids]) <= 5e-3, c
    # a property that holds at any size: every position's lambda is a log-probability of its own row
    assert bool((lam <= 0).all()) and bool(torch.isfinite(lam).all()) and bool(torch.isfinite(lse).all())
