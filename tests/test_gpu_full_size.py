"""Parity at the full sizes of the five workloads, in the launch configuration the benchmark times: the whole
tensor goes through the C ABI once; what is checked is (i) properties that hold at any size, computed on the GPU
over every slab, and (ii) sampled (layer, head) slabs or (sequence, head) outputs against the CPU oracle."""
import math

import numpy as np
import pytest
import torch

from oracle import ckv_oracle as O
from paper_2506_11418_b200 import synth
import parity_util as PU
import test_gpu_compress as TC

pytestmark = pytest.mark.gpu
DEV = "cuda"


def B():
    from paper_2506_11418_b200 import binding
    return binding


def need_free(gib):
    free, _ = torch.cuda.mem_get_info()
    if free < gib * 2**30:
        pytest.skip(f"needs {gib} GiB of free device memory")


def invariants_over_everything(K, V, dst, s, rounds):
    """Sec. 3 / Eq. 5 at any size: the degrees of every (layer, head) sum to the original length, and the
    degree-weighted sum of the stored centroids equals the sum of the original rows up to storage rounding.
    Every round stores its centroids within half a bf16 ulp (2^-9 relative), and averaging never increases the
    degree-weighted L1 mass, so the first moment moves by at most rounds * 2^-9 * sum_i |x_i| per column."""
    L, H, _, D = K.shape
    n = dst.len
    assert torch.equal(dst.deg[:, :, :n].sum(dim=2, dtype=torch.int64), torch.full((L, H), s, dtype=torch.int64, device=K.device))
    assert int(dst.deg[:, :, :n].min()) >= 1
    if dst.logdeg is not None:
        torch.testing.assert_close(dst.logdeg[:, :, :n], torch.log(dst.deg[:, :, :n].float()), rtol=1e-6, atol=1e-7)
    for l in range(L):
        w = dst.deg[l, :, :n].double().unsqueeze(-1)
        for src, out in ((K, dst.k), (V, dst.v)):
            moment = (w * out[l, :, :n].double()).sum(dim=1)
            x = src[l].double()
            bound = x.abs().sum(dim=1) * (rounds * 2.0 ** -9 * 1.001) + 1e-6
            assert bool(((moment - x.sum(dim=1)).abs() <= bound).all()), f"layer {l}: first moment not conserved"
            del x


def slab_matches_full_run(K, V, p, dst, assign, l, h, dtype="bf16"):
    """Clustering is independent per (layer, head): the slab alone must reproduce its slice of the full run bit for bit,
    and the slab alone is then checked against the oracle round by round."""
    Ks, Vs = K[l:l + 1, h:h + 1].contiguous(), V[l:l + 1, h:h + 1].contiguous()
    st = TC.multi_round_check(Ks, Vs, dtype, p)
    d1, n = st["dst"], dst.len
    assert d1.len == n
    assert torch.equal(d1.k[0, 0, :n], dst.k[l, h, :n]) and torch.equal(d1.v[0, 0, :n], dst.v[l, h, :n])
    assert torch.equal(d1.deg[0, 0, :n], dst.deg[l, h, :n])
    assert torch.equal(st["assign"][0, 0], assign[l, h])
    return st


def full_prefill(workload, p, slabs):
    b = B()
    cfg = synth.CONFIGS[workload]
    L, H, s, D = cfg["L"], cfg["H"], cfg["s"], cfg["d"]
    K = synth.ar1_keys(L, H, s, D, cfg["rho"], cfg["mean_std"], seed=cfg["seed"], dtype="bf16", device=DEV)
    V = synth.normal_values(L, H, s, D, seed=cfg["seed"], dtype="bf16", device=DEV)
    dst, assign, rounds = TC.run_gpu_prefill(K, V, None, p, want_assign=True, cap_extra=0)
    invariants_over_everything(K, V, dst, s, rounds)
    stats = [slab_matches_full_run(K, V, p, dst, assign, l, h) for l, h in slabs]
    return dst, rounds, stats


def test_config2_llama8b_32k_one_round():
    """32 layers x 8 KV heads x 32768 tokens, bf16, chunk 64, retain 50 %: the launch the benchmark times."""
    need_free(12)
    b = B()
    p = b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)
    dst, rounds, _ = full_prefill("llama8b_32k", p, [(0, 0), (17, 5), (31, 7)])
    assert rounds == 1 and dst.len == 16384
    torch.cuda.empty_cache()


def test_llama8b_32k_chunk256_paper_schedule():
    """The paper's default chunk (256) and schedule on the 32k workload, to a 25 % budget: six rounds ranked per head on
    the tensor-memory kernel (full chunks) and the tile kernel (the shorter last chunk of every round)."""
    need_free(12)
    b = B()
    s = synth.CONFIGS["llama8b_32k"]["s"]
    p = b.Params(chunk=256, n_sink=16, n_recent=64, n_rounds_max=16, r_init=0.8, r_decay=0.2, r_min=0.2, budget=s // 4)
    dst, rounds, _ = full_prefill("llama8b_32k", p, [(2, 3), (29, 0)])
    assert dst.len == s // 4 and rounds >= 4
    torch.cuda.empty_cache()


def test_llama8b_32k_chunk256_every_edge_and_per_chunk_ranking():
    need_free(12)
    b = B()
    for p in (b.Params(chunk=256, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0),
              b.Params(chunk=256, n_sink=0, n_recent=0, n_rounds_max=2, r_init=0.5, r_decay=0.0, r_min=0.5, select=b.SELECT_CHUNK)):
        dst, rounds, _ = full_prefill("llama8b_32k", p, [(9, 6)])
        torch.cuda.empty_cache()


def test_config3_llama8b_128k_two_rounds_ratio_one():
    """131072 tokens to 25 %: two rounds at ratio 1."""
    need_free(60)
    b = B()
    p = b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0)
    dst, rounds, _ = full_prefill("llama8b_128k", p, [(3, 1), (30, 6)])
    assert rounds == 2 and dst.len == 32768
    torch.cuda.empty_cache()


def test_config3_llama8b_128k_paper_schedule():
    """131072 tokens to a 25 % budget with the paper's defaults (16 sinks, 64 recent, r 0.8 - 0.2 j floored at 0.2),
    edges ranked across all chunks of a head."""
    need_free(60)
    b = B()
    s = synth.CONFIGS["llama8b_128k"]["s"]
    p = b.Params(chunk=64, n_sink=16, n_recent=64, n_rounds_max=16, r_init=0.8, r_decay=0.2, r_min=0.2, budget=s // 4)
    dst, rounds, _ = full_prefill("llama8b_128k", p, [(12, 4)])
    assert dst.len == s // 4 and rounds >= 4
    torch.cuda.empty_cache()


def test_config4_decode_batch32():
    """Batch 32, 8 KV heads x 4 query heads, 8192 centroids whose degrees sum to 32768 (plus appended tokens of
    degree 1), against the same kernel on the uncompressed 32768-token cache; sampled sequences against the oracle."""
    need_free(12)
    b = B()
    cfg = synth.CONFIGS["decode_b32"]
    Bz, H, G, D = cfg["batch"], cfg["H"], cfg["G"], cfg["d"]
    scale = 1.0 / math.sqrt(D)
    for slots, extra, with_deg in ((cfg["slots"], 256, True), (cfg["slots"], 0, True), (cfg["s"], 0, False)):
        cap, n = slots + 256, slots + extra
        caches = []
        for i in range(Bz):
            k = torch.randn((1, H, cap, D), device=DEV, generator=torch.Generator(DEV).manual_seed(1000 + i)).to(torch.bfloat16)
            v = torch.randn((1, H, cap, D), device=DEV, generator=torch.Generator(DEV).manual_seed(2000 + i)).to(torch.bfloat16)
            deg = logdeg = None
            if with_deg:
                deg = torch.ones((1, H, cap), dtype=torch.int32)
                deg[:, :, :slots] = synth.random_degrees((1, H), slots, cfg["s"], seed=i)
                assert int(deg[0, 0, :slots].sum()) == cfg["s"]
                deg = deg.to(DEV)
                logdeg = torch.log(deg.float())
            caches.append(b.Cache(k, v, deg, logdeg, n))
        q = synth.queries(Bz, H * G, D, seed=3, dtype="bf16", device=DEV)
        out = torch.full_like(q, 9.0)
        ws = torch.empty(b.decode_workspace_bytes(Bz, H, G, D, n), dtype=torch.uint8, device=DEV)
        b.decode_attn(b.layer_views(caches, 0, DEV), H, G, q, out, scale, n, ws)
        torch.cuda.synchronize()
        results = []
        for i in (0, 13, 31):
            c = caches[i]
            deg = c.deg[0, :, :n].cpu().numpy().astype(np.int64) if with_deg else None
            results.append(PU.check_attention(PU.to_np64(out[i]), PU.to_np64(q[i]), PU.to_np64(c.k[0, :, :n]), PU.to_np64(c.v[0, :, :n]),
                                              deg, scale, "bf16", f"slots {slots}+{extra}, sequence {i}"))
        PU.summarize_attention(results, f"batch 32, {slots}+{extra} slots")
        del caches
        torch.cuda.empty_cache()


def test_config5_serving_mix_reduced_layers():
    """Batch 64 with context lengths uniform on [4096, 65536], 75 % reduction at prefill (two rounds at ratio 1), then
    lock-step decoding: every step appends one token per sequence and runs decode attention over the ragged batch;
    every completed chunk of 64 appended tokens is clustered 64 -> 32 -> 16.  The cache shape is the workload's except
    for the number of layers (2 instead of 32, which only repeats the same launches) and 130 steps instead of 1024
    (two chunk triggers).  Two sampled sequences are replayed by the oracle on one layer and two KV heads."""
    need_free(40)
    b = B()
    cfg = synth.CONFIGS["serving_mix"]
    Bz, H, G, D, c = cfg["batch"], cfg["H"], cfg["G"], cfg["d"], cfg["chunk"]
    L, steps = 2, 130
    ctx = synth.context_lengths(Bz, cfg["ctx"][0], cfg["ctx"][1], seed=cfg["seed"])
    assert len(ctx) == Bz and min(ctx) >= 4096 and max(ctx) <= 65536
    p = b.Params(chunk=c, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0)
    scale = 1.0 / math.sqrt(D)
    sampled = {5: None, 40: None}
    oh = [1, 6]  # KV heads replayed by the oracle
    caches = []
    ws = None
    for i, n0 in enumerate(ctx):
        K = synth.ar1_keys(L, H, n0, D, (0.7, 0.95), 0.5, seed=100 + i, dtype="bf16", device=DEV)
        V = synth.normal_values(L, H, n0, D, seed=100 + i, dtype="bf16", device=DEV)
        src = b.Cache(K, V, None, None, n0)
        out_len, rounds, cap = b.compress_plan(n0, p)
        dst = b.Cache.empty(L, H, max(cap, out_len + steps), D, K.dtype, DEV)
        need = max(b.workspace_bytes(src, p), b.workspace_bytes(dst, p))
        if ws is None or ws.numel() < need:
            ws = torch.empty(need, dtype=torch.uint8, device=DEV)
        b.compress_prefill(src, dst, p, ws)
        assert b.workspace_status(ws) == 0 and rounds == 2
        caches.append(dst)
        if i in sampled:
            po = PU.oracle_params(p)
            Ko, Vo, do, _, _ = O.compress_prefill(PU.to_np64(K[1:2, oh]), PU.to_np64(V[1:2, oh]), None, po, storage="bf16")
            sampled[i] = [Ko, Vo, do, 0]
        del K, V, src
    wsd = torch.empty(b.decode_workspace_bytes(Bz, H, G, D, max(x.len for x in caches) + steps), dtype=torch.uint8, device=DEV)
    po = PU.oracle_params(p)
    worst = 0.0
    results = []
    for step in range(steps):
        kn = synth.ar1_keys(L, H, Bz, D, (0.7, 0.95), 0.5, seed=5000 + step, dtype="bf16", device=DEV)   # token b of every (layer, head)
        vn = synth.normal_values(L, H, Bz, D, seed=5000 + step, dtype="bf16", device=DEV)
        q = synth.queries(Bz, H * G, D, seed=7000 + step, dtype="bf16", device=DEV)
        for i, cache in enumerate(caches):
            b.compress_append(cache, kn[:, :, i:i + 1].contiguous(), vn[:, :, i:i + 1].contiguous(), p, ws)
        max_len = max(x.len for x in caches)
        outs = []
        for l in range(L):
            out = torch.empty_like(q)
            b.decode_attn(b.layer_views(caches, l, DEV), H, G, q, out, scale, max_len, wsd)
            outs.append(out)
        torch.cuda.synchronize()
        for i, st in sampled.items():
            st[0], st[1], st[2], st[3] = O.compress_append(st[0], st[1], st[2], st[3], PU.to_np64(kn[1:2, oh, i:i + 1]),
                                                           PU.to_np64(vn[1:2, oh, i:i + 1]), po, storage="bf16")
            assert caches[i].len == st[0].shape[2] and caches[i].pending == st[3]
            if step % 16 == 0 or step in (63, 64, 127, 128, steps - 1):
                n = caches[i].len
                np.testing.assert_array_equal(caches[i].deg[1, oh, :n].cpu().numpy(), st[2][0])
                qs = PU.to_np64(q[i]).reshape(H, G, D)[oh].reshape(len(oh) * G, D)
                got = PU.to_np64(outs[1][i]).reshape(H, G, D)[oh].reshape(len(oh) * G, D)
                # against the oracle's own replay of the cache (storage rounding of two rounds may differ by an ulp in a
                # few rows, so the stated bar alone applies here) ...
                ref = O.app_attn(qs, st[0][0], st[1][0], st[2][0], scale)
                worst = max(worst, float(np.abs(got - ref).max()))
                # ... and, with the arithmetic bound, against the oracle's attention over the GPU's stored cache
                results.append(PU.check_attention(got, qs, PU.to_np64(caches[i].k[1, oh, :n]), PU.to_np64(caches[i].v[1, oh, :n]),
                                                  st[2][0], scale, "bf16", f"step {step}, sequence {i}"))
    assert worst <= 2e-2, f"decode attention over the serving mix: max abs error {worst:.3e}"
    PU.summarize_attention(results, "serving mix")
    for i, cache in enumerate(caches):   # every sequence: degrees account for every token ever written
        n = cache.len
        total = ctx[i] + steps
        assert torch.equal(cache.deg[:, :, :n].sum(dim=2, dtype=torch.int64),
                           torch.full((L, H), total, dtype=torch.int64, device=DEV))
    # sampled sequences: the cache itself, two ulp for the two rounds of storage rounding
    for i, st in sampled.items():
        n = caches[i].len
        for t, ref in ((caches[i].k, st[0]), (caches[i].v, st[1])):
            got = PU.to_np64(t[1, oh, :n])
            assert np.all(np.abs(got - ref[0]) <= 2 * PU.bf16_ulp(ref[0]) * 1.0001 + 1e-30)
    del caches
    torch.cuda.empty_cache()


def test_config5_serving_mix_at_its_stated_size():
    """The serving mix as stated: batch 64, context lengths uniform on [4096, 65536], 32 layers x 8 KV heads, bf16.
    Every sequence is prefill-compressed to 25 % one at a time from a scratch buffer (the uncompressed caches together
    would not fit), then 1024 lock-step steps: one appended token per sequence (ckv_compress_append_batch; every
    completed chunk of 64 appended tokens is clustered 64 -> 32 -> 16: sixteen triggers per sequence) and decode
    attention over the ragged batch on all 32 layers.  The oracle replays two sampled sequences on one layer and two
    KV heads: cache lengths and pending counts at every step; degrees, stored rows and attention outputs at sampled
    steps, among them the steps around a trigger; degree sums over everything at the end."""
    need_free(110)
    b = B()
    cfg = synth.CONFIGS["serving_mix"]
    Bz, L, H, G, D, c = cfg["batch"], cfg["L"], cfg["H"], cfg["G"], cfg["d"], cfg["chunk"]
    steps = 1024
    ctx = synth.context_lengths(Bz, cfg["ctx"][0], cfg["ctx"][1], seed=cfg["seed"])
    p = b.Params(chunk=c, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0)
    po = PU.oracle_params(p)
    scale = 1.0 / math.sqrt(D)
    ol, oh = 17, [2, 5]                        # the layer and KV heads the oracle follows
    sampled = {3: None, 41: None}              # and the sequences
    growth = (steps // c + 1) * (c // 4) + c + 8
    caches, ws = [], None
    for i, n0 in enumerate(ctx):
        K = synth.ar1_keys(L, H, n0, D, (0.7, 0.95), 0.5, seed=100 + i, dtype="bf16", device=DEV)
        V = synth.normal_values(L, H, n0, D, seed=100 + i, dtype="bf16", device=DEV)
        src = b.Cache(K, V, None, None, n0)
        out_len, rounds, cap = b.compress_plan(n0, p)
        dst = b.Cache.empty(L, H, max(cap, out_len + growth), D, K.dtype, DEV)
        need = max(b.workspace_bytes(src, p), b.workspace_bytes(dst, p))
        if ws is None or ws.numel() < need:
            ws = None
            torch.cuda.empty_cache()
            ws = torch.empty(need, dtype=torch.uint8, device=DEV)
        b.compress_prefill(src, dst, p, ws)
        assert b.workspace_status(ws) == 0 and rounds == 2 and dst.len == out_len
        assert torch.equal(dst.deg[:, :, :out_len].sum(dim=2, dtype=torch.int64), torch.full((L, H), n0, dtype=torch.int64, device=DEV))
        caches.append(dst)
        if i in sampled:
            Ko, Vo, do, _, _ = O.compress_prefill(PU.to_np64(K[ol:ol + 1, oh]), PU.to_np64(V[ol:ol + 1, oh]), None, po, storage="bf16")
            sampled[i] = [Ko, Vo, do, 0]
        del K, V, src
    torch.cuda.empty_cache()
    wsd = torch.empty(b.decode_workspace_bytes(Bz, H, G, D, max(x.cap for x in caches)), dtype=torch.uint8, device=DEV)
    results, worst, triggers = [], 0.0, 0
    out = torch.empty((Bz, H * G, D), dtype=torch.bfloat16, device=DEV)   # the other layers' outputs
    out_l = torch.empty_like(out)                                          # the followed layer's
    for step in range(steps):
        kn = synth.ar1_keys(L, H, Bz, D, (0.7, 0.95), 0.5, seed=5000 + step, dtype="bf16", device=DEV)   # token b of every (layer, head)
        vn = synth.normal_values(L, H, Bz, D, seed=5000 + step, dtype="bf16", device=DEV)
        q = synth.queries(Bz, H * G, D, seed=7000 + step, dtype="bf16", device=DEV)
        before = caches[0].len
        b.compress_append_batch(caches, kn, vn, p, ws)
        triggers += caches[0].len < before
        max_len = max(x.len for x in caches)
        views = b.layer_views_all(caches, DEV)
        check = step % 97 == 0 or step % 64 in (62, 63, 0) and step % 256 < 70 or step == steps - 1
        for l in range(L):
            b.decode_attn(views[l], H, G, q, out_l if l == ol else out, scale, max_len, wsd)
        for i, st in sampled.items():
            st[0], st[1], st[2], st[3] = O.compress_append(st[0], st[1], st[2], st[3], PU.to_np64(kn[ol:ol + 1, oh, i:i + 1]),
                                                           PU.to_np64(vn[ol:ol + 1, oh, i:i + 1]), po, storage="bf16")
            assert caches[i].len == st[0].shape[2] and caches[i].pending == st[3]
            if check:
                torch.cuda.synchronize()
                n = caches[i].len
                np.testing.assert_array_equal(caches[i].deg[ol, oh, :n].cpu().numpy(), st[2][0])
                qs = PU.to_np64(q[i]).reshape(H, G, D)[oh].reshape(len(oh) * G, D)
                got = PU.to_np64(out_l[i]).reshape(H, G, D)[oh].reshape(len(oh) * G, D)
                worst = max(worst, float(np.abs(got - O.app_attn(qs, st[0][0], st[1][0], st[2][0], scale)).max()))
                results.append(PU.check_attention(got, qs, PU.to_np64(caches[i].k[ol, oh, :n]), PU.to_np64(caches[i].v[ol, oh, :n]),
                                                  st[2][0], scale, "bf16", f"step {step}, sequence {i}"))
    assert b.workspace_status(ws) == 0
    assert triggers == steps // c                       # sixteen windows per sequence
    assert worst <= 2e-2, f"decode attention over the serving mix: max abs error {worst:.3e}"
    PU.summarize_attention(results, f"serving mix at full size, {len(results)} sampled outputs")
    for i, cache in enumerate(caches):   # every sequence: degrees account for every token ever written
        n = cache.len
        assert torch.equal(cache.deg[:, :, :n].sum(dim=2, dtype=torch.int64),
                           torch.full((L, H), ctx[i] + steps, dtype=torch.int64, device=DEV))
        torch.testing.assert_close(cache.logdeg[:, :, :n], torch.log(cache.deg[:, :, :n].float()), rtol=1e-6, atol=1e-7)
    for i, st in sampled.items():        # the cache itself: two ulp for the two rounds of storage rounding
        n = caches[i].len
        for t, ref in ((caches[i].k, st[0]), (caches[i].v, st[1])):
            got = PU.to_np64(t[ol, oh, :n])
            assert np.all(np.abs(got - ref[0]) <= 2 * PU.bf16_ulp(ref[0]) * 1.0001 + 1e-30)
    del caches
    torch.cuda.empty_cache()


def test_no_chunking_16k_four_layers():
    """chunk = 0 (plain Bipartite Soft Matching) in the launch the benchmark's no-chunk section times: the first 16384
    tokens of 4 layers x 8 KV heads, every edge merged.  Invariants over everything, two slabs against the oracle."""
    need_free(8)
    b = B()
    cfg = synth.CONFIGS["llama8b_32k"]
    L, H, s, D = 4, cfg["H"], 16384, cfg["d"]
    K = synth.ar1_keys(L, H, s, D, cfg["rho"], cfg["mean_std"], seed=cfg["seed"], dtype="bf16", device=DEV)
    V = synth.normal_values(L, H, s, D, seed=cfg["seed"], dtype="bf16", device=DEV)
    p = b.Params(chunk=0, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)
    dst, assign, rounds = TC.run_gpu_prefill(K, V, None, p, want_assign=True, cap_extra=0)
    assert rounds == 1 and dst.len == s // 2
    invariants_over_everything(K, V, dst, s, rounds)
    for l, h in ((0, 0), (3, 5)):
        slab_matches_full_run(K, V, p, dst, assign, l, h)
    torch.cuda.empty_cache()


def test_no_chunking_128k_sampled_rows():
    """chunk = 0 at 131072 tokens (the length at which the paper's un-chunked variant runs out of memory): one layer,
    8 KV heads, ratio 1.  The n^2 / 4 similarities are never stored.  Sampled A tokens are checked one by one: the
    oracle's cosine row against all 65536 B tokens of the head names the target; the GPU's choice must be that token
    or one whose cosine is within 1e-5 of the best (rounding order of an fp32 contraction)."""
    need_free(6)
    b = B()
    cfg = synth.CONFIGS["llama8b_128k"]
    L, H, s, D = 1, cfg["H"], cfg["s"], cfg["d"]
    K = synth.ar1_keys(L, H, s, D, cfg["rho"], cfg["mean_std"], seed=cfg["seed"], dtype="bf16", device=DEV)
    V = synth.normal_values(L, H, s, D, seed=cfg["seed"], dtype="bf16", device=DEV)
    p = b.Params(chunk=0, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)
    dst, assign, rounds = TC.run_gpu_prefill(K, V, None, p, want_assign=True, cap_extra=0)
    assert rounds == 1 and dst.len == s // 2
    invariants_over_everything(K, V, dst, s, rounds)
    rng = np.random.default_rng(5)
    for h in (0, 6):
        Kh = K[0, h].cpu().float().numpy().astype(np.float64)
        KB = Kh[1::2]
        asg = assign[0, h].cpu().numpy()
        rows = np.concatenate([[0, s // 2 - 1], rng.integers(0, s // 2, size=62)])
        S = O.cosine_matrix(Kh[0::2][rows], KB)
        for i, a_idx in enumerate(rows):
            got = int(asg[2 * a_idx])  # every edge is merged: B token j survives in slot j
            assert 0 <= got < s // 2
            best = int(np.argmax(S[i]))
            assert got == best or S[i, got] >= S[i, best] - 1e-5, f"head {h} A token {a_idx}: {got} vs {best}"
        # every B token's degree is one plus the number of A tokens that chose it
        counts = np.bincount(asg[0::2], minlength=s // 2) + 1
        np.testing.assert_array_equal(dst.deg[0, h, :s // 2].cpu().numpy(), counts)
    torch.cuda.empty_cache()


def window_matches_full_run(K, V, p, dst, assign, t0, t1, out0, dtype="bf16"):
    """With every edge merged (or ranked per chunk) a chunk's clusters depend on that chunk alone, so source tokens
    [t0, t1) (t0 on a boundary of every round's chunks) clustered on their own must reproduce rows out0 ... of the full
    run bit for bit; the window's own run is checked against the oracle round by round."""
    Kw, Vw = K[:, :, t0:t1].contiguous(), V[:, :, t0:t1].contiguous()
    st = TC.multi_round_check(Kw, Vw, dtype, p)
    d1 = st["dst"]
    n = d1.len
    assert torch.equal(d1.k[0, 0, :n], dst.k[0, 0, out0:out0 + n]) and torch.equal(d1.v[0, 0, :n], dst.v[0, 0, out0:out0 + n])
    assert torch.equal(d1.deg[0, 0, :n], dst.deg[0, 0, out0:out0 + n])
    assert torch.equal(st["assign"][0, 0] + out0, assign[0, 0, t0:t1])
    return n


def test_one_head_longer_than_four_gib():
    """Maximum sizes: one (layer, head) of 2^24 + 202 tokens, whose keys alone take more than 4 GiB, so that row offsets
    inside a single slab pass 2^31 and 2^32 bytes.  Windows around both marks and the ragged end are compared with the
    same windows clustered alone (and those with the oracle); the degrees of the whole slab must sum to its length."""
    need_free(40)
    b = B()
    s = (1 << 24) + 202
    K = synth.ar1_keys(1, 1, s, 128, (0.9, 0.9), 0.5, seed=5, dtype="bf16", device=DEV)
    V = synth.normal_values(1, 1, s, 128, seed=5, dtype="bf16", device=DEV)
    marks = [(0, 2048), ((1 << 23) - 1024, (1 << 23) + 1024), ((1 << 24) - 2048, s)]
    cases = [
        (b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0), lambda t: t // 2),
        (b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0), lambda t: t // 4),
        (b.Params(chunk=256, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0), lambda t: t // 2),
        (b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=1, r_init=0.5, r_decay=0.0, r_min=0.5, select=b.SELECT_CHUNK),
         lambda t: t // 64 * 48),
    ]
    for p, out_of in cases:
        dst, assign, rounds = TC.run_gpu_prefill(K, V, None, p, want_assign=True, cap_extra=0)
        n = dst.len
        assert int(dst.deg[0, 0, :n].sum(dtype=torch.int64)) == s and int(dst.deg[0, 0, :n].min()) >= 1
        end = 0
        for t0, t1 in marks:
            end = out_of(t0) + window_matches_full_run(K, V, p, dst, assign, t0, t1, out_of(t0))
        assert end == n  # the last window ends where the compressed slab ends
        del dst, assign
        torch.cuda.empty_cache()
    # ranked over the whole head: nothing local to compare with, the invariants must still hold
    p = b.Params(chunk=64, n_sink=16, n_recent=64, n_rounds_max=2, r_init=0.8, r_decay=0.2, r_min=0.2)
    dst, assign, rounds = TC.run_gpu_prefill(K, V, None, p, want_assign=True, cap_extra=0)
    n = dst.len
    assert int(dst.deg[0, 0, :n].sum(dtype=torch.int64)) == s and int(dst.deg[0, 0, :n].min()) >= 1
    assert int(assign[0, 0].min()) == 0 and int(assign[0, 0].max()) == n - 1
    del dst, assign
    torch.cuda.empty_cache()
