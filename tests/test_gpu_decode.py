"""Parity of ckv_decode_attn (Eq. 3) against the oracle's fp64 softmax attention with the log-degree bias."""
import math

import numpy as np
import pytest
import torch

from oracle import ckv_oracle as O
from paper_2506_11418_b200 import synth
import parity_util as PU

pytestmark = pytest.mark.gpu
DEV = "cuda"


def B():
    from paper_2506_11418_b200 import binding
    return binding


def build_batch(lens, caps, H, dtype, seed, with_deg=True, total_factor=4):
    b = B()
    caches = []
    for i, (n, cap) in enumerate(zip(lens, caps)):
        K = synth.ar1_keys(1, H, cap, 128, (0.7, 0.95), 0.5, seed=seed + i, dtype=dtype, device=DEV)
        V = synth.normal_values(1, H, cap, 128, seed=seed + i, dtype=dtype, device=DEV)
        if with_deg and n > 0:
            deg = torch.ones((1, H, cap), dtype=torch.int32)
            deg[:, :, :n] = synth.random_degrees((1, H), n, total_factor * n, seed=seed + i)
            deg = deg.to(DEV)
            logdeg = torch.log(deg.float())
        elif with_deg:
            deg = torch.ones((1, H, cap), dtype=torch.int32, device=DEV)
            logdeg = torch.zeros((1, H, cap), dtype=torch.float32, device=DEV)
        else:
            deg, logdeg = None, None
        caches.append(b.Cache(K, V, deg, logdeg, n))
    return caches


def run_decode(caches, H, G, dtype, seed, scale=None):
    b = B()
    Bz = len(caches)
    q = synth.queries(Bz, H * G, 128, seed=seed, dtype=dtype, device=DEV)
    out = torch.full_like(q, 7.0)
    max_len = max(c.len for c in caches)
    ws = torch.empty(b.decode_workspace_bytes(Bz, H, G, 128, max_len), dtype=torch.uint8, device=DEV)
    views = b.layer_views(caches, 0, DEV)
    scale = scale if scale is not None else 1.0 / math.sqrt(128)
    b.decode_attn(views, H, G, q, out, scale, max_len, ws)
    torch.cuda.synchronize()
    return q, out, scale


def check_decode(caches, H, G, dtype, seed, scale=None, tol=None, what="decode", require_sensitive=True):
    q, out, scale = run_decode(caches, H, G, dtype, seed, scale)
    results = []
    for i, c in enumerate(caches):
        got = PU.to_np64(out[i])
        if c.len == 0:
            assert np.all(got == 0)
            continue
        n = c.len
        deg = c.deg[0, :, :n].cpu().numpy().astype(np.int64) if c.deg is not None else None
        results.append(PU.check_attention(got, PU.to_np64(q[i]), PU.to_np64(c.k[0, :, :n]), PU.to_np64(c.v[0, :, :n]), deg, scale,
                                          dtype, f"sequence {i}", bar=tol))
    return PU.summarize_attention(results, what, require_sensitive)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("G", [1, 4, 8])
def test_decode_ragged_batch(dtype, G):
    lens = [1, 33, 500, 0, 4097, 128, 2600]
    caps = [8, 40, 512, 16, 4100, 128, 2700]
    caches = build_batch(lens, caps, 2, dtype, seed=50 + G)
    check_decode(caches, 2, G, dtype, seed=60 + G)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_decode_unit_degrees_is_plain_attention(dtype):
    """logdeg = NULL: Eq. 3 reduces to Eq. 1."""
    caches = build_batch([777, 2048], [800, 2048], 4, dtype, seed=70, with_deg=False)
    check_decode(caches, 4, 4, dtype, seed=71)


def test_decode_config1_after_compress():
    """Config 1 end to end: compress the tiny fp32 cache, then one decode query ~ N(0,1) over the centroids."""
    b = B()
    K = synth.ar1_keys(1, 1, 2048, 128, (0.9, 0.9), 0.0, seed=0, dtype="f32", device=DEV)
    V = synth.normal_values(1, 1, 2048, 128, seed=0, dtype="f32", device=DEV)
    p = b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)
    src = b.Cache(K, V, None, None, 2048)
    dst = b.Cache.empty(1, 1, 1024, 128, K.dtype, DEV)
    ws = torch.empty(b.workspace_bytes(src, p), dtype=torch.uint8, device=DEV)
    b.compress_prefill(src, dst, p, ws)
    torch.cuda.synchronize()
    assert dst.len == 1024
    check_decode([dst], 1, 1, "f32", seed=0)
    # the compressed output approximates attention over the original cache (Sec. 3): same order of magnitude check only
    q, out, scale = run_decode([dst], 1, 1, "f32", seed=0)
    exact = O.attn(PU.to_np64(q[0]), PU.to_np64(K[0]), PU.to_np64(V[0]), scale)
    assert np.abs(PU.to_np64(out[0]) - exact).max() < 0.5


def test_decode_large_scores_are_stable():
    """Scores far from zero: the online softmax must not overflow."""
    caches = build_batch([3000], [3000], 1, "f32", seed=80)
    check_decode(caches, 1, 2, "f32", seed=81, scale=1.0, tol=1e-3)


def test_decode_config4_shape_small_batch():
    """Config 4's shape at a reduced batch: 8 KV heads, 4 query heads each, 8192 centroids whose degrees sum to 32768."""
    caches = build_batch([8192, 8192], [8448, 8448], 8, "bf16", seed=90, total_factor=4)
    worst = check_decode(caches, 8, 4, "bf16", seed=91)
    assert worst < 2e-2


@pytest.mark.parametrize("lens,H,G", [([16416], 8, 4), ([5000], 2, 8), ([4096, 9000, 130], 1, 4), ([20000], 1, 1)])
def test_decode_small_batch_cluster_path(lens, H, G):
    """Few (sequence, head) pairs and long caches: the launch where the CTAs of a pair form a thread-block cluster and
    combine their partials through distributed shared memory (16 CTAs per pair here; the ragged batches above take
    the 8-CTA shape, large batches the two-kernel path).  The first case is the decode leg of the benchmark's step."""
    caches = build_batch(lens, [n + 7 for n in lens], H, "bf16", seed=300 + H, total_factor=4)
    worst = check_decode(caches, H, G, "bf16", seed=310 + G)
    assert worst < 2e-2


def test_decode_one_sequence_longer_than_two_gib():
    """Maximum sizes: a single head of 2^23 + 37 slots, so that the keys of one (sequence, head) pass 2^31 bytes; batch 1
    takes the cluster launch, the same cache twice in a batch of 24 the split kernel with its combine kernel."""
    import psutil
    if psutil.virtual_memory().available < 96 * 2**30:
        pytest.skip("the fp64 oracle of this case needs about 40 GiB of host memory")
    n = (1 << 23) + 37
    caches = build_batch([n], [n + 3], 1, "bf16", seed=90)
    # (over 8 million slots the rounding bound of the value sum is a fifth of what the bias moves: this case is about
    # offsets, the bias is judged on the shorter ones)
    check_decode(caches, 1, 4, "bf16", seed=91, what=f"decode, one head of {n} slots", require_sensitive=False)
    b = B()
    q = synth.queries(24, 4, 128, seed=92, dtype="bf16", device=DEV)
    q[1:] = q[:1]
    out = torch.full_like(q, 7.0)
    ws = torch.empty(b.decode_workspace_bytes(24, 1, 4, 128, n), dtype=torch.uint8, device=DEV)
    views = b.layer_views(caches * 24, 0, DEV)
    b.decode_attn(views, 1, 4, q, out, 1.0 / math.sqrt(128), n, ws)
    one = torch.full_like(q[:1], 7.0)
    b.decode_attn(b.layer_views(caches, 0, DEV), 1, 4, q[:1], one, 1.0 / math.sqrt(128), n, ws)
    torch.cuda.synchronize()
    # the split points differ between the two launches, so the sums round differently: the arithmetic bound of the
    # parity check is far above this, a wrong offset far below it
    assert bool((out.float() - one.float()).abs().max() <= 2e-3)
    assert bool((out == out[:1]).all())
