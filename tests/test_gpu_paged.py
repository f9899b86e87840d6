"""Paged cache: ckv_decode_attn_paged against the oracle (Eq. 3 over the gathered sequence), and the flow
read pages -> compress -> write back -> attend, with the pages a sequence no longer needs returned to the pool."""
import math

import numpy as np
import pytest
import torch

from oracle import ckv_oracle as O
from paper_2506_11418_b200 import synth
import parity_util as PU

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make_pool(n_pages, H, P, D, seed):
    g = torch.Generator(DEV).manual_seed(seed)
    kp = torch.randn((n_pages, H, P, D), device=DEV, generator=g).to(torch.bfloat16)   # junk wherever no sequence writes
    vp = torch.randn((n_pages, H, P, D), device=DEV, generator=g).to(torch.bfloat16)
    dp = torch.full((n_pages, H, P), 77, dtype=torch.int32, device=DEV)
    lp = torch.full((n_pages, H, P), 3.0, dtype=torch.float32, device=DEV)
    return kp, vp, dp, lp


def paged_decode_case(P, G, with_deg, lens, H):
    from paper_2506_11418_b200 import binding as b
    D = 128
    n_blocks = [(n + P - 1) // P for n in lens]
    pool = sum(n_blocks) + 7
    kp, vp, dp, lp = make_pool(pool, H, P, D, seed=5)
    perm = torch.randperm(pool, generator=torch.Generator().manual_seed(9)).to(torch.int32)
    tables, off = [], 0
    for i, n in enumerate(lens):
        tab = perm[off:off + max(n_blocks[i], 1)].to(DEV)
        off += n_blocks[i]
        tables.append(tab)
        if n == 0:
            continue
        K = synth.ar1_keys(1, H, n, D, (0.7, 0.95), 0.5, seed=40 + i, dtype="bf16", device=DEV)[0]
        V = synth.normal_values(1, H, n, D, seed=40 + i, dtype="bf16", device=DEV)[0]
        deg = synth.random_degrees((H,), n, 3 * n, seed=40 + i).to(DEV)
        b.pages_scatter(tab, n, K, V, deg, kp, vp, dp, lp)
    q = synth.queries(len(lens), H * G, D, seed=11, dtype="bf16", device=DEV)
    out = torch.full_like(q, 5.0)
    max_len = max(lens)
    ws = torch.empty(b.decode_workspace_bytes(len(lens), H, G, D, max_len), dtype=torch.uint8, device=DEV)
    views = b.paged_views(tables, lens, DEV)
    scale = 1.0 / math.sqrt(D)
    b.decode_attn_paged(views, kp, vp, lp if with_deg else None, H, G, q, out, scale, max_len, ws)
    torch.cuda.synchronize()
    kpn, vpn, dpn = PU.to_np64(kp), PU.to_np64(vp), dp.cpu().numpy().astype(np.int64)
    results = []
    for i, n in enumerate(lens):
        got = PU.to_np64(out[i])
        if n == 0:
            assert np.all(got == 0)
            continue
        tab = tables[i].cpu().numpy()
        # Eq. 3 over a paged cache is, by definition, Eq. 3 over the gathered sequence
        ref = O.app_attn_paged(PU.to_np64(q[i]), kpn, vpn, dpn if with_deg else None, tab, n, scale)
        r = PU.check_attention(got, PU.to_np64(q[i]), O.gather_pages(kpn, tab, n), O.gather_pages(vpn, tab, n),
                               O.gather_pages(dpn, tab, n) if with_deg else None, scale, "bf16", f"sequence {i} (len {n})")
        assert abs(np.abs(got - ref).max() - r["err"]) < 1e-12
        results.append(r)
    PU.summarize_attention(results, f"paged, page {P}, lens {lens}")


@pytest.mark.parametrize("P,G,with_deg", [(64, 4, True), (32, 1, True), (128, 8, False), (64, 4, False)])
def test_paged_decode_ragged_batch(P, G, with_deg):
    paged_decode_case(P, G, with_deg, [1, 63, 64, 65, 1000, 0, 4100, 2500, 96], 2)


@pytest.mark.parametrize("P,G,lens,H", [(64, 4, [20000], 1), (32, 8, [9000, 8200, 8500, 8300], 2), (128, 2, [1000, 64, 0], 2),
                                        (256, 4, [16416], 8)])
def test_paged_decode_small_batch(P, G, lens, H):
    """Few (sequence, head) pairs: the paged kernel in its thread-block-cluster forms (16, 10 and 8 CTAs per pair)."""
    paged_decode_case(P, G, True, lens, H)


def test_pages_compress_write_back_attend():
    """One sequence, two layers' worth of heads in one pool: gather its pages, cluster to 25 % (two rounds at ratio 1),
    scatter the result back into the first quarter of its pages, attend over the pages; the other pages go back to the pool."""
    from paper_2506_11418_b200 import binding as b
    H, G, D, P, n = 4, 4, 128, 64, 4096
    n_blocks = n // P
    pool = n_blocks + 5
    kp, vp, dp, lp = make_pool(pool, H, P, D, seed=6)
    table = torch.randperm(pool, generator=torch.Generator().manual_seed(3))[:n_blocks].to(torch.int32).to(DEV)
    K = synth.ar1_keys(1, H, n, D, (0.7, 0.95), 0.5, seed=70, dtype="bf16", device=DEV)
    V = synth.normal_values(1, H, n, D, seed=70, dtype="bf16", device=DEV)
    b.pages_scatter(table, n, K[0], V[0], None, kp, vp, dp, lp)
    # read pages
    src = b.Cache.empty(1, H, n, D, torch.bfloat16, DEV)
    b.pages_gather(table, n, kp, vp, dp, src.k[0], src.v[0], src.deg[0], src.logdeg[0])
    src.len = n
    assert torch.equal(src.k, K) and torch.equal(src.v, V) and int(src.deg.min()) == 1 == int(src.deg.max())
    # compress
    p = b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0)
    out_len, _, cap = b.compress_plan(n, p)
    dst = b.Cache.empty(1, H, cap, D, torch.bfloat16, DEV)
    ws = torch.empty(b.workspace_bytes(src, p), dtype=torch.uint8, device=DEV)
    b.compress_prefill(src, dst, p, ws)
    assert b.workspace_status(ws) == 0 and dst.len == out_len == n // 4
    # write back: the sequence keeps the first ceil(out_len / P) pages of its table, the rest are free again
    keep = (out_len + P - 1) // P
    b.pages_scatter(table[:keep], out_len, dst.k[0], dst.v[0], dst.deg[0], kp, vp, dp, lp)
    # attend over the pages
    q = synth.queries(1, H * G, D, seed=12, dtype="bf16", device=DEV)
    out = torch.empty_like(q)
    wsd = torch.empty(b.decode_workspace_bytes(1, H, G, D, out_len), dtype=torch.uint8, device=DEV)
    scale = 1.0 / math.sqrt(D)
    b.decode_attn_paged(b.paged_views([table[:keep]], [out_len], DEV), kp, vp, lp, H, G, q, out, scale, out_len, wsd)
    torch.cuda.synchronize()
    po = PU.oracle_params(p)
    Ko, Vo, do, _, _ = O.compress_prefill(PU.to_np64(K), PU.to_np64(V), None, po, storage="bf16")
    got_deg = O.gather_pages(dp.cpu().numpy().astype(np.int64), table[:keep].cpu().numpy(), out_len)
    np.testing.assert_array_equal(got_deg, do[0])
    # the attention must agree with the oracle on the GPU's own stored cache (bit-exact input) and, within the bf16 bar,
    # with the oracle end to end
    ref_own = O.app_attn_paged(PU.to_np64(q[0]), PU.to_np64(kp), PU.to_np64(vp), dp.cpu().numpy().astype(np.int64),
                               table[:keep].cpu().numpy(), out_len, scale)
    assert np.abs(PU.to_np64(out[0]) - ref_own).max() <= 2e-2
    tabn = table[:keep].cpu().numpy()
    PU.summarize_attention([PU.check_attention(PU.to_np64(out[0]), PU.to_np64(q[0]), O.gather_pages(PU.to_np64(kp), tabn, out_len),
                                               O.gather_pages(PU.to_np64(vp), tabn, out_len),
                                               O.gather_pages(dp.cpu().numpy().astype(np.int64), tabn, out_len), scale, "bf16",
                                               "pages after write-back")], "pages after write-back")
    ref = O.app_attn(PU.to_np64(q[0]), Ko[0], Vo[0], do[0], scale)
    assert np.abs(PU.to_np64(out[0]) - ref).max() <= 2e-2


def test_paged_argument_checks():
    from paper_2506_11418_b200 import binding as b
    # page size must be a power of two >= 32; fp32 pages are not supported by the paged attention kernel
    assert b.lib.ckv_decode_attn_paged(0x1000, 0x2000, 0x3000, None, 48, 1, 1, 1, 128, b.BF16, 0x4000, 0x5000, 0.1, 10, 0x6000, 1 << 20, None) == 6
    assert b.lib.ckv_decode_attn_paged(0x1000, 0x2000, 0x3000, None, 64, 1, 1, 1, 128, b.F32, 0x4000, 0x5000, 0.1, 10, 0x6000, 1 << 20, None) == 6
    assert b.lib.ckv_pages_gather(0x1000, 10, 0x2000, 0x3000, None, 16, 1, 128, b.BF16, 0x4000, 0x5000, None, None, 10, None) == 6
    assert b.lib.ckv_pages_gather(0x1000, 10, 0x2000, 0x3000, None, 64, 1, 128, b.BF16, 0x4000, 0x5000, None, None, 5, None) == 1


# ----------------------------------------------------------------------------- clustering directly on pages

def make_pools(L, n_pages, H, P, D, seed):
    pools = []
    for l in range(L):
        kp, vp, dp, lp = make_pool(n_pages, H, P, D, seed=seed + l)
        pools.append((kp, vp, dp, lp))
    return pools


def gathered(pools, table, n):
    """The sequence a block table describes, as the oracle sees it: K, V [L, H, n, D] float64, deg [L, H, n]."""
    tab = table.cpu().numpy()
    K = np.stack([O.gather_pages(PU.to_np64(kp), tab, n) for kp, _, _, _ in pools])
    V = np.stack([O.gather_pages(PU.to_np64(vp), tab, n) for _, vp, _, _ in pools])
    deg = np.stack([O.gather_pages(dp.cpu().numpy().astype(np.int64), tab, n) for _, _, dp, _ in pools])
    lg = np.stack([O.gather_pages(lp.cpu().numpy().astype(np.float64), tab, n) for _, _, _, lp in pools])
    return K, V, deg, lg


def paged_compress_case(L, H, P, s, p, seed):
    """read pages -> compress -> write back -> free blocks, without leaving the pages.  By definition the result is the
    oracle's compress_prefill of the gathered sequence, found through the table that ckv_pages_plan names; the number of
    pages the sequence keeps is ceil(out_len / P)."""
    from paper_2506_11418_b200 import binding as b
    D = 128
    own = (s + P - 1) // P
    out_len, rounds, n_scratch, in_scratch, kept = b.pages_plan(s, p, P)
    assert kept == (out_len + P - 1) // P
    pool_pages = own + n_scratch + 3
    pools = make_pools(L, pool_pages, H, P, D, seed)
    perm = torch.randperm(pool_pages, generator=torch.Generator().manual_seed(seed)).to(torch.int32)
    table, scratch = perm[:own].to(DEV), perm[own:own + n_scratch].to(DEV)
    spare = perm[own + n_scratch:]
    K = synth.ar1_keys(L, H, s, D, (0.7, 0.95), 0.5, seed=seed, dtype="bf16", device=DEV)
    V = synth.normal_values(L, H, s, D, seed=seed, dtype="bf16", device=DEV)
    for l, (kp, vp, dp, lp) in enumerate(pools):
        b.pages_scatter(table, s, K[l], V[l], None, kp, vp, dp, lp)
    untouched = [(kp[spare.long()].clone(), vp[spare.long()].clone()) for kp, vp, _, _ in pools]
    ws = torch.empty(b.paged_workspace_bytes(L, H, D, torch.bfloat16, s, p), dtype=torch.uint8, device=DEV)
    got_len, got_in_scratch = b.compress_paged(pools, table, s, False, scratch if n_scratch else None, p, ws)
    assert b.workspace_status(ws) == 0
    assert got_len == out_len and got_in_scratch == in_scratch
    result_table = (scratch if in_scratch else table)[:kept]
    Kg, Vg, dg, lg = gathered(pools, result_table, out_len)
    po = PU.oracle_params(p)
    Ko, Vo, do, _, logs = O.compress_prefill(PU.to_np64(K), PU.to_np64(V), None, po, storage="bf16")
    assert len(logs) == rounds and Ko.shape[2] == out_len
    np.testing.assert_array_equal(dg, do)
    np.testing.assert_allclose(lg, np.log(do.astype(np.float64)), rtol=1e-6, atol=1e-7)
    for got, ref in ((Kg, Ko), (Vg, Vo)):
        assert np.all(np.abs(got - ref) <= max(rounds, 1) * PU.bf16_ulp(ref) * 1.0001 + 1e-30)
        assert np.mean(got == ref) >= 0.99
    for (kp, vp, _, _), (k0, v0) in zip(pools, untouched):          # pages of neither table are left alone
        assert torch.equal(kp[spare.long()], k0) and torch.equal(vp[spare.long()], v0)
    return pools, result_table, out_len, K, V


@pytest.mark.parametrize("P,s,sink,recent,rounds,r,decay,select,budget", [
    (64, 4096, 0, 0, 1, 1.0, 0.0, 0, 0),          # page-aligned chunks, one round: the result is in the scratch pages
    (64, 4096 + 37, 16, 64, 2, 1.0, 0.0, 0, 0),   # chunks straddle pages, a shorter last chunk, two rounds: back in its own pages
    (128, 3000, 16, 64, 1, 0.8, 0.0, 0, 0),       # ranked per head: matching pass, ranking, merge pass; last chunk staged
    (256, 5000, 5, 9, 3, 0.5, 0.0, 1, 0),         # ranked per chunk, three rounds
    (64, 6000, 16, 64, 16, 0.8, 0.2, 0, 1500),    # the paper's schedule to a 25 % budget: six rounds, the last one trimmed
    (64, 100, 0, 0, 1, 1.0, 0.0, 0, 0),           # one full chunk and a last chunk
    (64, 50, 0, 0, 2, 1.0, 0.0, 0, 0),            # nothing but a last chunk
    (64, 1, 0, 0, 1, 1.0, 0.0, 0, 0),             # nothing to merge
])
def test_compress_paged_against_the_oracle(P, s, sink, recent, rounds, r, decay, select, budget):
    from paper_2506_11418_b200 import binding as b
    p = b.Params(chunk=64, n_sink=sink, n_recent=recent, n_rounds_max=rounds, r_init=r, r_decay=decay, r_min=min(r, 0.2) if decay else r,
                 select=select, budget=budget)
    paged_compress_case(2, 3, P, s, p, seed=600 + s)


def test_compress_paged_again_with_degrees_then_attend():
    """A second compression of the same sequence reads the degrees the first one left in the pages; decode attention then
    runs over the kept pages."""
    from paper_2506_11418_b200 import binding as b
    L, H, G, P, s, D = 2, 2, 4, 64, 3000, 128
    p1 = b.Params(chunk=64, n_sink=16, n_recent=64, n_rounds_max=1, r_init=0.6, r_decay=0.0, r_min=0.6, select=b.SELECT_GLOBAL)
    pools, table, n1, K, V = paged_compress_case(L, H, P, s, p1, seed=77)
    # second call: fresh scratch pages (appended to every pool)
    out_len, rounds, n_scratch, in_scratch, kept = b.pages_plan(n1, p1, P)
    base = pools[0][0].shape[0]
    pools = [(torch.cat([kp, torch.zeros((n_scratch, H, P, D), dtype=kp.dtype, device=DEV)]),
              torch.cat([vp, torch.zeros((n_scratch, H, P, D), dtype=vp.dtype, device=DEV)]),
              torch.cat([dp, torch.zeros((n_scratch, H, P), dtype=dp.dtype, device=DEV)]),
              torch.cat([lp, torch.zeros((n_scratch, H, P), dtype=lp.dtype, device=DEV)])) for kp, vp, dp, lp in pools]
    scratch = torch.arange(base, base + n_scratch, dtype=torch.int32, device=DEV)
    K1, V1, d1, _ = gathered(pools, table, n1)
    ws = torch.empty(b.paged_workspace_bytes(L, H, D, torch.bfloat16, n1, p1), dtype=torch.uint8, device=DEV)
    got_len, got_in = b.compress_paged(pools, table, n1, True, scratch, p1, ws)
    assert b.workspace_status(ws) == 0 and got_len == out_len and got_in == in_scratch
    res = (scratch if in_scratch else table)[:kept]
    Kg, Vg, dg, _ = gathered(pools, res, out_len)
    Ko, Vo, do, _, _ = O.compress_prefill(K1, V1, d1, PU.oracle_params(p1), storage="bf16")
    np.testing.assert_array_equal(dg, do)
    assert int(dg.sum(axis=2).min()) == s == int(dg.sum(axis=2).max())     # every original token is still accounted for
    for got, ref in ((Kg, Ko), (Vg, Vo)):
        assert np.all(np.abs(got - ref) <= PU.bf16_ulp(ref) * 1.0001 + 1e-30)
    q = synth.queries(1, H * G, D, seed=13, dtype="bf16", device=DEV)
    out = torch.empty_like(q)
    wsd = torch.empty(b.decode_workspace_bytes(1, H, G, D, out_len), dtype=torch.uint8, device=DEV)
    scale = 1.0 / math.sqrt(D)
    kp, vp, dp, lp = pools[1]
    b.decode_attn_paged(b.paged_views([res], [out_len], DEV), kp, vp, lp, H, G, q, out, scale, out_len, wsd)
    torch.cuda.synchronize()
    PU.summarize_attention([PU.check_attention(PU.to_np64(out[0]), PU.to_np64(q[0]), Kg[1], Vg[1], dg[1], scale, "bf16",
                                               "pages clustered twice")], "pages clustered twice")


def test_compress_paged_argument_checks():
    from paper_2506_11418_b200 import binding as b
    import ctypes as C
    pool = (b.CkvPagePool * 1)(b.CkvPagePool(0x1000, 0x2000, 0x3000, None))
    p = b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)
    call = lambda **kw: b.lib.ckv_compress_paged(pool, 1, kw.get("H", 2), 128, kw.get("dtype", b.BF16), kw.get("P", 64), 0x4000, kw.get("n", 1000), 0,
                                                 kw.get("scratch", 0x5000), kw.get("n_scratch", 100), C.byref(kw.get("p", p).c()), kw.get("ws", 0x6000),
                                                 kw.get("ws_bytes", 1 << 30), None, None, None)
    assert call(P=48) == 6 and call(P=32) == 6 and call(dtype=b.F32) == 6             # page size, dtype: unsupported here
    assert call(p=b.Params(chunk=128, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)) == 6
    assert call(n_scratch=3) == 3                                                     # too few scratch pages
    assert call(ws_bytes=64) == 4                                                     # workspace too small
    out_len, rounds, n_scratch, in_scratch, kept = b.pages_plan(1000, p, 64)
    assert (out_len, rounds, n_scratch, in_scratch, kept) == (500, 1, 8, True, 8)


# ----------------------------------------------------------------------------- append + attention in one launch

@pytest.mark.parametrize("P,G,H,lens", [(64, 4, 2, [0, 1, 63, 64, 65, 1000, 4100, 2500, 127]), (128, 8, 1, [20000]),
                                        (32, 1, 8, [9000, 31, 32]), (256, 4, 8, [16415])])
def test_decode_append_attn_paged(P, G, H, lens):
    """One decoding step of Algorithm 1 in one launch: the new token of every sequence lands in slot len of its pages
    with degree 1, and Eq. 3 runs over len + 1 tokens.  By definition: append, then the oracle's attention over the
    gathered sequence.  Several steps in a row (the lengths cross page and tile boundaries); the pages must end up
    exactly as a separate append would leave them, and pages of other sequences untouched."""
    from paper_2506_11418_b200 import binding as b
    D, steps = 128, 3
    n_blocks = [(n + steps + P - 1) // P for n in lens]
    pool = sum(n_blocks) + 5
    kp, vp, dp, lp = make_pool(pool, H, P, D, seed=21)
    perm = torch.randperm(pool, generator=torch.Generator().manual_seed(4)).to(torch.int32)
    tables, off = [], 0
    ref = []   # per sequence: K, V [H, n, D] float64, deg [H, n]
    for i, n in enumerate(lens):
        tab = perm[off:off + n_blocks[i]].to(DEV)
        off += n_blocks[i]
        tables.append(tab)
        if n > 0:
            K = synth.ar1_keys(1, H, n, D, (0.7, 0.95), 0.5, seed=80 + i, dtype="bf16", device=DEV)[0]
            V = synth.normal_values(1, H, n, D, seed=80 + i, dtype="bf16", device=DEV)[0]
            deg = synth.random_degrees((H,), n, 3 * n, seed=80 + i).to(DEV)
            b.pages_scatter(tab, n, K, V, deg, kp, vp, dp, lp)
            ref.append([PU.to_np64(K), PU.to_np64(V), deg.cpu().numpy().astype(np.int64)])
        else:
            ref.append([np.zeros((H, 0, D)), np.zeros((H, 0, D)), np.zeros((H, 0), dtype=np.int64)])
    idle = perm[off:].long()
    idle_before = (kp[idle].clone(), vp[idle].clone(), dp[idle].clone())
    scale = 1.0 / math.sqrt(D)
    cur = list(lens)
    for step in range(steps):
        kn = synth.ar1_keys(1, len(lens) * H, 1, D, (0.7, 0.95), 0.5, seed=900 + step, dtype="bf16", device=DEV).view(len(lens), H, D).contiguous()
        vn = synth.normal_values(1, len(lens) * H, 1, D, seed=900 + step, dtype="bf16", device=DEV).view(len(lens), H, D).contiguous()
        q = synth.queries(len(lens), H * G, D, seed=950 + step, dtype="bf16", device=DEV)
        out = torch.full_like(q, 5.0)
        max_len = max(cur) + 1
        ws = torch.empty(b.decode_workspace_bytes(len(lens), H, G, D, max_len), dtype=torch.uint8, device=DEV)
        b.decode_append_attn_paged(b.paged_views(tables, cur, DEV), kp, vp, dp, lp, H, G, kn, vn, q, out, scale, max_len, ws)
        torch.cuda.synchronize()
        results = []
        for i in range(len(lens)):
            ref[i][0] = np.concatenate([ref[i][0], PU.to_np64(kn[i])[:, None, :]], axis=1)
            ref[i][1] = np.concatenate([ref[i][1], PU.to_np64(vn[i])[:, None, :]], axis=1)
            ref[i][2] = np.concatenate([ref[i][2], np.ones((H, 1), dtype=np.int64)], axis=1)
            cur[i] += 1
            results.append(PU.check_attention(PU.to_np64(out[i]), PU.to_np64(q[i]), ref[i][0], ref[i][1], ref[i][2], scale, "bf16",
                                              f"step {step}, sequence {i} (len {cur[i]})"))
        PU.summarize_attention(results, f"append + attention, page {P}, step {step}")
    # the pages hold what a separate append would have written
    kpn, vpn, dpn, lpn = PU.to_np64(kp), PU.to_np64(vp), dp.cpu().numpy().astype(np.int64), lp.cpu().numpy().astype(np.float64)
    for i, n in enumerate(cur):
        tab = tables[i].cpu().numpy()
        np.testing.assert_array_equal(O.gather_pages(kpn, tab, n), ref[i][0])
        np.testing.assert_array_equal(O.gather_pages(vpn, tab, n), ref[i][1])
        np.testing.assert_array_equal(O.gather_pages(dpn, tab, n), ref[i][2])
        np.testing.assert_allclose(O.gather_pages(lpn, tab, n), np.log(ref[i][2].astype(np.float64)), rtol=1e-6, atol=1e-7)
    assert torch.equal(kp[idle], idle_before[0]) and torch.equal(vp[idle], idle_before[1]) and torch.equal(dp[idle], idle_before[2])
