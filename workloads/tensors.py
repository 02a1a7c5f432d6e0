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
