"""ckv_decode_attn_static -- the decode entry point for callers that cannot allocate device memory (no
workspace argument; its scratch is a fixed array inside the library) -- must give the same output as
ckv_decode_attn.  This file sorts last on purpose, so that a run that stops at the first failure has
already run every other test."""
import math

import pytest
import torch

from paper_2506_11418_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _batch(b, lens, H, dtype, seed):
    caches = []
    for i, n in enumerate(lens):
        cap = n + 8
        K = synth.ar1_keys(1, H, cap, 128, (0.7, 0.95), 0.5, seed=seed + i, dtype=dtype, device=DEV)
        V = synth.normal_values(1, H, cap, 128, seed=seed + i, dtype=dtype, device=DEV)
        deg = torch.ones((1, H, cap), dtype=torch.int32)
        deg[:, :, :n] = synth.random_degrees((1, H), n, 3 * n, seed=seed + i)
        deg = deg.to(DEV)
        caches.append(b.Cache(K, V, deg, torch.log(deg.float()), n))
    return caches


@pytest.mark.parametrize("dtype,tol", [("bf16", 2e-2), ("f32", 2e-4)])
def test_static_scratch_matches_workspace_entry_point(dtype, tol):
    from paper_2506_11418_b200 import binding as b
    H, G = 4, 4
    scale = 1.0 / math.sqrt(128)
    # two calls in a row with different shapes: the second finds the array as the first left it
    for call, lens in enumerate([[3000, 517, 64, 2048], [129, 4100]]):
        caches = _batch(b, lens, H, dtype, seed=200 + 10 * call)
        q = synth.queries(len(lens), H * G, 128, seed=300 + call, dtype=dtype, device=DEV)
        ref, got = torch.zeros_like(q), torch.full_like(q, 5.0)
        max_len = max(lens)
        ws = torch.empty(b.decode_workspace_bytes(len(lens), H, G, 128, max_len), dtype=torch.uint8, device=DEV)
        views = b.layer_views(caches, 0, DEV)
        b.decode_attn(views, H, G, q, ref, scale, max_len, ws)
        b.decode_attn_static(views, H, G, q, got, scale, max_len)
        torch.cuda.synchronize()
        err = (got.float() - ref.float()).abs().max().item()
        assert err <= tol, f"call {call}: static-scratch output differs from the workspace entry point by {err}"


def test_static_scratch_rejects_what_does_not_fit():
    from paper_2506_11418_b200 import binding as b
    # 4096 sequences x 8 KV heads x 8 query heads x 132 floats exceed the 1 Mi-float array even with one split;
    # the size check comes before anything touches the GPU, so dummy pointers are enough
    st = b.lib.ckv_decode_attn_static(0x1000, 4096, 8, 8, 128, b.BF16, 0x1000, 0x2000, 0.1, 1024, None)
    assert st == 3
