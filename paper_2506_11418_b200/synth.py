"""Seeded synthetic inputs shaped like long-context KV caches.

This module holds no arithmetic of the method itself: it only draws tensors.  The
CUDA path and the CPU oracle are both fed from here, so that they see the same bits.

Keys follow a per-head AR(1) process along the sequence, k_t = rho * k_{t-1} + eps_t
with eps ~ N(0, I) and a stationary start, plus an optional per-head mean offset.
Neighbouring keys are then highly similar and the similarity decays convexly with
distance, the property of real key caches that the paper's Observations 1 and 2
describe.  Values are i.i.d. N(0, 1).
"""
from __future__ import annotations

import torch

CONFIGS = {
    # name: the five workloads, by the numbers of their descriptions
    "tiny": dict(L=1, H=1, G=1, s=2048, d=128, dtype="f32", chunk=64, rho=(0.9, 0.9), mean_std=0.0, seed=0),
    "llama8b_32k": dict(L=32, H=8, G=4, s=32768, d=128, dtype="bf16", chunk=64, rho=(0.7, 0.95), mean_std=0.5, seed=0),
    "llama8b_128k": dict(L=32, H=8, G=4, s=131072, d=128, dtype="bf16", chunk=64, rho=(0.7, 0.95), mean_std=0.5, seed=0),
    "decode_b32": dict(L=1, H=8, G=4, s=32768, slots=8192, batch=32, d=128, dtype="bf16", seed=0),
    "serving_mix": dict(L=32, H=8, G=4, d=128, dtype="bf16", chunk=64, batch=64, ctx=(4096, 65536), seed=1),
}

_BLOCK = 256


def torch_dtype(name: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _gen(seed: int, device):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def head_rhos(L: int, H: int, rho_range, seed: int, device="cpu"):
    """Per-(layer, head) AR(1) coefficient, uniform on [rho_range)."""
    lo, hi = rho_range
    u = torch.rand(L * H, generator=_gen(seed * 1000003 + 11, "cpu"), dtype=torch.float64)
    return (lo + (hi - lo) * u).to(torch.float32).to(device)


def ar1_keys(L: int, H: int, s: int, d: int, rho_range=(0.9, 0.9), mean_std: float = 0.0, seed: int = 0,
             dtype: str = "f32", device="cpu"):
    """[L, H, s, d] keys: AR(1) along s per head, stationary start, plus a per-head mean ~ N(0, mean_std^2)."""
    device = torch.device(device)
    out = torch.empty((L, H, s, d), dtype=torch_dtype(dtype), device=device)
    rhos = head_rhos(L, H, rho_range, seed, device).view(L, H)
    means = torch.randn((L, H, 1, d), generator=_gen(seed * 1000003 + 13, "cpu"), dtype=torch.float32).to(device) * mean_std
    i = torch.arange(_BLOCK, device=device, dtype=torch.float32)
    prev_tf32 = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    try:
        for l in range(L):
            g = _gen(seed * 1000003 + 17 + l, device)
            rho = rhos[l].view(H, 1, 1)
            # lower-triangular Toeplitz filter T[i, j] = rho^(i-j) for one block of the recurrence
            expo = (i.view(-1, 1) - i.view(1, -1)).clamp(min=0)
            T = torch.tril(rho ** expo)                                   # [H, B, B]
            carry_w = rho ** (i.view(1, -1, 1) + 1.0)                      # [H, B, 1]
            carry = torch.randn((H, 1, d), generator=g, device=device) / torch.sqrt(1.0 - rho * rho)
            for b0 in range(0, s, _BLOCK):
                nb = min(_BLOCK, s - b0)
                eps = torch.randn((H, nb, d), generator=g, device=device)
                blk = torch.bmm(T[:, :nb, :nb], eps) + carry_w[:, :nb] * carry
                carry = blk[:, nb - 1:nb, :]
                out[l, :, b0:b0 + nb] = (blk + means[l]).to(out.dtype)
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev_tf32
    return out


def normal_values(L: int, H: int, s: int, d: int, seed: int = 0, dtype: str = "f32", device="cpu"):
    """[L, H, s, d] values, i.i.d. N(0, 1)."""
    device = torch.device(device)
    out = torch.empty((L, H, s, d), dtype=torch_dtype(dtype), device=device)
    for l in range(L):
        g = _gen(seed * 1000003 + 500009 + l, device)
        out[l] = torch.randn((H, s, d), generator=g, device=device).to(out.dtype)
    return out


def random_degrees(shape, slots: int, total: int, seed: int = 0, device="cpu"):
    """Integer degrees [*shape, slots], each >= 1, summing to `total` along the last axis:
    1 + Multinomial(total - slots, uniform)."""
    g = _gen(seed * 1000003 + 700001, "cpu")
    n = 1
    for x in shape:
        n *= x
    extra = total - slots
    idx = torch.randint(0, slots, (n, extra), generator=g)
    deg = torch.ones((n, slots), dtype=torch.int32)
    deg.scatter_add_(1, idx, torch.ones_like(idx, dtype=torch.int32))
    return deg.view(*shape, slots).to(device)


def queries(batch: int, heads: int, d: int, seed: int = 0, dtype: str = "f32", device="cpu"):
    """[batch, heads, d] queries ~ N(0, 1)."""
    g = _gen(seed * 1000003 + 900007, "cpu")
    return torch.randn((batch, heads, d), generator=g, dtype=torch.float32).to(torch_dtype(dtype)).to(device)


def context_lengths(batch: int, lo: int, hi: int, seed: int = 1):
    """Per-sequence context lengths, uniform integers on [lo, hi]."""
    g = _gen(seed * 1000003 + 31, "cpu")
    return torch.randint(lo, hi + 1, (batch,), generator=g).tolist()
