"""Seeded q/k/v/g/dO tensors in canonical token order.

Distributions: q, k ~ N(0,1)/8; v ~ N(0,1); g = log(sigmoid(N(3,1))) (a log-decay,
always negative); dO ~ N(0,1).  Values are rounded to the run dtype here, so every
consumer (oracle or CUDA path) sees exactly the same numbers.  ``g`` stays fp32.

The draw uses torch's generator of the chosen device: a CPU draw and a CUDA draw
give different (equally valid) values, so a test that compares two consumers
draws once and hands both the same tensors.
"""
from __future__ import annotations

import torch

_DTYPES = {"fp32": torch.float32, "bf16": torch.bfloat16}


def make_inputs(n_tokens: int, H: int, dk: int, dv: int, dtype: str, seed: int, device="cpu"):
    """dict(q [C,H,dk], k [C,H,dk], v [C,H,dv], g [C,H] fp32, dO [C,H,dv])."""
    dt = _DTYPES[dtype]
    gen = torch.Generator(device=device)
    gen.manual_seed(1000003 * (seed + 1))

    def normal(*shape):
        return torch.randn(*shape, generator=gen, device=device, dtype=torch.float32)

    q = (normal(n_tokens, H, dk) / 8.0).to(dt)
    k = (normal(n_tokens, H, dk) / 8.0).to(dt)
    v = normal(n_tokens, H, dv).to(dt)
    g = torch.nn.functional.logsigmoid(normal(n_tokens, H) + 3.0).contiguous()
    dO = normal(n_tokens, H, dv).to(dt)
    return {"q": q, "k": k, "v": v, "g": g, "dO": dO}


def make_gk(n_tokens: int, H: int, dk: int, seed: int, device="cpu", strong_every: int = 0, strong_shift: float = 7.0):
    """Per-channel log-decay gk [C,H,dk] fp32 = log(sigmoid(N(3,1))) (the distribution of the scalar gate, drawn per
    key channel).  strong_every > 0: every strong_every-th channel gets log(sigmoid(N(3 - strong_shift, 1))) instead --
    with the default shift decays of about e^-4 per token, e^-250 over a chunk -- to exercise gates far outside the usual
    range."""
    gen = torch.Generator(device=device)
    gen.manual_seed(1000003 * (seed + 1) + 77)
    x = torch.randn(n_tokens, H, dk, generator=gen, device=device, dtype=torch.float32) + 3.0
    if strong_every > 0:
        x[:, :, ::strong_every] -= strong_shift
    return torch.nn.functional.logsigmoid(x).contiguous()


def make_logits(n_rows: int, V: int, dtype: str, seed: int, device="cpu", peak: float = 6.0):
    """Compact logit rows and token ids for the log-probability step.

    z [n_rows, V]: N(0, 2^2) background with one favoured word per row raised by ``peak`` (a language-model
    row is peaked, not flat); rounded to the run dtype.  token_id int32 [n_rows]: the vocabulary id of each
    compact token, uniform over the vocabulary except that with probability 1/2 a token is the favoured
    word of the row before it (so that target logits cover both the peak and the background).
    Rows are drawn in slabs so that the fp32 staging buffer stays small."""
    dt = _DTYPES[dtype]
    gen = torch.Generator(device=device)
    gen.manual_seed(7000003 * (seed + 1))
    fav = torch.randint(0, V, (n_rows,), generator=gen, device=device)
    uni = torch.randint(0, V, (n_rows,), generator=gen, device=device)
    coin = torch.rand(n_rows, generator=gen, device=device) < 0.5
    token_id = uni.clone()
    token_id[1:] = torch.where(coin[1:], fav[:-1], uni[1:])
    z = torch.empty(n_rows, V, dtype=dt, device=device)
    slab = max(1, (64 << 20) // max(V, 1))
    for lo in range(0, n_rows, slab):
        hi = min(n_rows, lo + slab)
        blk = torch.randn(hi - lo, V, generator=gen, device=device, dtype=torch.float32) * 2.0
        blk[torch.arange(hi - lo, device=device), fav[lo:hi]] += peak
        z[lo:hi] = blk.to(dt)
    return {"z": z, "token_id": token_id.to(torch.int32)}


def make_logp_grad(n_pos: int, seed: int, device="cpu", keep: float = 0.6):
    """dL/dlambda for every non-terminal semantic position: an advantage-like N(0,1) value divided by the
    number of positions, exactly zero where a Bernoulli(keep) action mask drops the position."""
    gen = torch.Generator(device=device)
    gen.manual_seed(9000011 * (seed + 1))
    adv = torch.randn(n_pos, generator=gen, device=device, dtype=torch.float32)
    mask = torch.rand(n_pos, generator=gen, device=device) < keep
    return torch.where(mask, adv / max(n_pos, 1), torch.zeros_like(adv))


def make_conv_inputs(n_rows: int, D: int, w: int, dtype: str, seed: int, device="cpu"):
    """Inputs of the short causal convolution: x, dy ~ N(0,1) rounded to the run dtype, W ~ N(0,1)/sqrt(w) fp32."""
    dt = _DTYPES[dtype]
    gen = torch.Generator(device=device)
    gen.manual_seed(3000017 * (seed + 1))
    x = torch.randn(n_rows, D, generator=gen, device=device, dtype=torch.float32).to(dt)
    dy = torch.randn(n_rows, D, generator=gen, device=device, dtype=torch.float32).to(dt)
    W = torch.randn(D, w, generator=gen, device=device, dtype=torch.float32) / (w ** 0.5)
    return {"x": x, "dy": dy, "W": W}


def make_attn_inputs(n_rows: int, Hq: int, Hkv: int, d: int, dtype: str, seed: int, device="cpu"):
    """q, k, v, dO ~ N(0,1) rounded to the run dtype (scores scaled by 1/sqrt(d) have unit variance)."""
    dt = _DTYPES[dtype]
    gen = torch.Generator(device=device)
    gen.manual_seed(5000011 * (seed + 1))
    mk = lambda h: torch.randn(n_rows, h, d, generator=gen, device=device, dtype=torch.float32).to(dt)  # noqa: E731
    return {"q": mk(Hq), "k": mk(Hkv), "v": mk(Hkv), "dO": mk(Hq)}
