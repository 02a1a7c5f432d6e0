"""GPU parity of the tree-aware causal convolution (Section 4.2) through the C ABI against the fp64 oracle.

Tolerances: y and dx are sums of at most 4 products in fp32, rounded once to the run dtype: relative Frobenius
error <= 3e-3 for bf16 (one rounding, 2^-9 per element at most) and 1e-6 for fp32.  dW is an fp32 sum over all
rows of products of dtype-rounded inputs: <= 1e-4 relative (accumulation order only)."""
import numpy as np
import pytest
import torch

import paper_2608_28158_b200 as H
from oracle import conv_oracle as co
from workloads import config_forest, make_conv_inputs, make_forest

pytestmark = pytest.mark.gpu
TOL = {"bf16": 3e-3, "fp32": 1e-6}


def _rel(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def _run(fo, D, w, dtype, seed, use_plan=True):
    C = fo.n_tokens
    inp = make_conv_inputs(C, D, w, dtype, seed)
    rot = None
    if use_plan:
        rot = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64).row_of_token
    prev, nxt, cptr, crow = H.harts_conv_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, rot)
    rows = torch.arange(C) if rot is None else torch.as_tensor(rot.astype(np.int64))
    phys = {}
    for n in ("x", "dy"):
        t = torch.empty_like(inp[n]); t[rows] = inp[n]; phys[n] = t.cuda()
    W = inp["W"].cuda()
    dev = lambda a: torch.as_tensor(np.ascontiguousarray(a)).cuda()  # noqa: E731
    prev_d, nxt_d, cptr_d = dev(prev), dev(nxt), dev(cptr)
    crow_d = dev(crow) if len(crow) else torch.zeros(1, dtype=torch.int32, device="cuda")
    y = torch.full_like(phys["x"], float("nan")); dx = torch.full_like(phys["x"], float("nan"))
    dW = torch.full_like(W, float("nan"))
    scratch = torch.empty(H.harts_conv_scratch_bytes(D, w), dtype=torch.uint8, device="cuda")
    H.harts_conv_fwd(phys["x"], W, prev_d, y)
    H.harts_conv_bwd(phys["x"], W, phys["dy"], nxt_d, cptr_d, crow_d, dx, dW, scratch)
    torch.cuda.synchronize()
    x64, dy64, W64 = inp["x"].double().numpy(), inp["dy"].double().numpy(), inp["W"].double().numpy()
    y_ref = co.conv_fwd(fo, x64, W64)
    dx_ref, dW_ref = co.conv_bwd(fo, x64, W64, dy64)
    rc = rows.cuda()
    return (_rel(y[rc].double().cpu().numpy(), y_ref), _rel(dx[rc].double().cpu().numpy(), dx_ref),
            _rel(dW.double().cpu().numpy(), dW_ref))


@pytest.mark.parametrize("name,D,w,dtype", [("cfg0", 64, 4, "fp32"), ("cfg0b", 512, 4, "bf16"), ("cfg0b", 4096, 4, "bf16"),
                                            ("cfg0", 1032, 3, "bf16"), ("cfg0b", 8, 2, "fp32"), ("cfg1", 512, 4, "bf16")])
def test_parity_on_trees(name, D, w, dtype):
    ey, ex, ew = _run(config_forest(name), D, w, dtype, 1)
    assert ey <= TOL[dtype] and ex <= TOL[dtype] and ew <= 1e-4, (ey, ex, ew)


def test_bench_size_all_rows_of_sampled_channels():
    """The benchmark's workload (cfg3's 588,899 compact rows x 4096 channels, bf16, w = 4, plan row order).  The
    convolution is depthwise, so a channel can be checked on its own: for eight channels spread over the width, every
    row of y and dx (all strip heads and tails, every fork row) and the channels' dW against the oracle."""
    fo = config_forest("cfg3")
    C, Dm, w = fo.n_tokens, 4096, 4
    inp = make_conv_inputs(C, Dm, w, "bf16", 7, device="cuda")
    rot = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64).row_of_token
    prev, nxt, cptr, crow = H.harts_conv_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, rot)
    rows = torch.as_tensor(rot.astype(np.int64)).cuda()
    x = torch.empty_like(inp["x"]); x[rows] = inp["x"]
    dy = torch.empty_like(inp["dy"]); dy[rows] = inp["dy"]
    W = inp["W"]
    dev = lambda a: torch.as_tensor(np.ascontiguousarray(a)).cuda()  # noqa: E731
    y = torch.full_like(x, float("nan")); dx = torch.full_like(x, float("nan")); dW = torch.full_like(W, float("nan"))
    scratch = torch.empty(H.harts_conv_scratch_bytes(Dm, w), dtype=torch.uint8, device="cuda")
    H.harts_conv_fwd(x, W, dev(prev), y)
    H.harts_conv_bwd(x, W, dy, dev(nxt), dev(cptr), dev(crow), dx, dW, scratch)
    torch.cuda.synchronize()
    ch = [0, 1, 7, 8, 1023, 2048, 4094, 4095]
    cht = torch.as_tensor(ch).cuda()
    x64, dy64 = (inp[n][:, cht].double().cpu().numpy() for n in ("x", "dy"))
    W64 = W[cht].double().cpu().numpy()
    y_ref = co.conv_fwd(fo, x64, W64)
    dx_ref, dW_ref = co.conv_bwd(fo, x64, W64, dy64)
    got_y = y[rows][:, cht].double().cpu().numpy()
    got_dx = dx[rows][:, cht].double().cpu().numpy()
    assert _rel(got_y, y_ref) <= TOL["bf16"] and _rel(got_dx, dx_ref) <= TOL["bf16"]
    # row by row as well: one wrong row must not hide in the norm over 589 k rows (bf16 rounding: 2^-9 per element)
    for got, ref in ((got_y, y_ref), (got_dx, dx_ref)):
        row_err = np.linalg.norm(got - ref, axis=1)
        floor = np.sqrt((ref ** 2).mean() * ref.shape[1])
        assert (row_err / np.maximum(np.linalg.norm(ref, axis=1), floor)).max() <= 2 * TOL["bf16"]
    assert _rel(dW[cht].double().cpu().numpy(), dW_ref) <= 1e-4
    assert bool(torch.isfinite(y.float()).all()) and bool(torch.isfinite(dx.float()).all())


def test_parity_without_a_row_map_and_on_bushy_trees():
    # every token forks: roots of 3 tokens with children at every offset, grandchildren too
    par = [-1, 0, 0, 0, 1, 1, 2, 4]
    off = [0, 1, 2, 3, 1, 2, 1, 1]
    ln = [3, 2, 1, 4, 1, 3, 2, 1]
    fo = make_forest([(par, off, ln), ([-1], [0], [1]), (par, off, ln)])
    for use_plan in (False, True):
        ey, ex, ew = _run(fo, 128, 4, "fp32", 2, use_plan)
        assert ey <= 1e-6 and ex <= 1e-6 and ew <= 1e-5, (ey, ex, ew)


def test_argument_errors():
    x = torch.zeros(4, 64, device="cuda"); W = torch.zeros(64, 4, device="cuda")
    prev = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    with pytest.raises(H.HartsError):
        H.harts_conv_fwd(x, W, prev, x)                                 # in place
    with pytest.raises(H.HartsError):
        H.harts_conv_fwd(x[:, :60].contiguous(), W[:60], prev, torch.zeros(4, 60, device="cuda"))   # D % 8
    with pytest.raises(H.HartsError):
        H.harts_conv_fwd(x, torch.zeros(64, 5, device="cuda"), prev, torch.zeros_like(x))            # w > 4
