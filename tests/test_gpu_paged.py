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
