"""The library only enqueues work on the caller's stream (kernels and one memset; no allocation, no synchronisation), so a
whole step -- compress, append, decode over every layer -- can be captured once into a CUDA graph and replayed.  The replay
must reproduce the eager results bit for bit."""
import math

import pytest
import torch

from paper_2506_11418_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_step_replays_from_a_cuda_graph():
    from paper_2506_11418_b200 import binding as b
    L, H, G, D, s, c = 3, 8, 4, 128, 8192, 64
    K = synth.ar1_keys(L, H, s, D, (0.7, 0.95), 0.5, seed=11, dtype="bf16", device=DEV)
    V = synth.normal_values(L, H, s, D, seed=11, dtype="bf16", device=DEV)
    kn = synth.ar1_keys(L, H, c, D, (0.7, 0.95), 0.5, seed=12, dtype="bf16", device=DEV)
    vn = synth.normal_values(L, H, c, D, seed=12, dtype="bf16", device=DEV)
    q = synth.queries(L, H * G, D, seed=13, dtype="bf16", device=DEV)
    p = b.Params(chunk=c, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)
    src = b.Cache(K, V, None, None, s)
    out_len, _, cap = b.compress_plan(s, p)
    final_len = out_len + c // 2
    scale = 1.0 / math.sqrt(D)

    def fresh():
        dst = b.Cache.empty(L, H, cap + c, D, K.dtype, DEV)
        ws = torch.empty(max(b.workspace_bytes(src, p), b.workspace_bytes(dst, p)), dtype=torch.uint8, device=DEV)
        wsd = torch.empty(b.decode_workspace_bytes(1, H, G, D, cap + c), dtype=torch.uint8, device=DEV)
        out = torch.zeros_like(q)
        return dst, ws, wsd, out

    def step(dst, ws, wsd, out, views):
        b.compress_prefill(src, dst, p, ws)
        b.compress_append(dst, kn, vn, p, ws)
        for l in range(L):
            b.decode_attn(views[l], H, G, q[l:l + 1], out[l:l + 1], scale, final_len, wsd)

    def views_of(dst):
        dst.len = final_len  # a function of shapes and parameters only
        return [b.layer_views([dst], l, DEV) for l in range(L)]

    # eager
    dst_e, ws_e, wsd_e, out_e = fresh()
    step(dst_e, ws_e, wsd_e, out_e, views_of(dst_e))
    torch.cuda.synchronize()
    assert dst_e.len == final_len and b.workspace_status(ws_e) == 0

    # captured once (after a warm-up on the capture stream's buffers), replayed twice
    dst_g, ws_g, wsd_g, out_g = fresh()
    views_g = views_of(dst_g)
    step(dst_g, ws_g, wsd_g, out_g, views_g)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step(dst_g, ws_g, wsd_g, out_g, views_g)
    for _ in range(2):
        for t in (dst_g.k, dst_g.v, out_g):
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        n = final_len
        assert torch.equal(dst_g.k[:, :, :n], dst_e.k[:, :, :n]) and torch.equal(dst_g.v[:, :, :n], dst_e.v[:, :, :n])
        assert torch.equal(dst_g.deg[:, :, :n], dst_e.deg[:, :, :n])
        assert torch.equal(out_g, out_e)
    assert b.workspace_status(ws_g) == 0
