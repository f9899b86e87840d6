"""Parity of the CUDA compress path (ckv_compress_prefill / ckv_compress_append through the C ABI)
against the CPU oracle, element by element on the same seeded inputs."""
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


def make_inputs(L, H, s, dtype, seed, rho=(0.7, 0.95), mean_std=0.5, deg_max=1):
    K = synth.ar1_keys(L, H, s, 128, rho, mean_std, seed=seed, dtype=dtype, device=DEV)
    V = synth.normal_values(L, H, s, 128, seed=seed, dtype=dtype, device=DEV)
    deg = None
    if deg_max > 1:
        g = torch.Generator().manual_seed(seed + 5)
        deg = torch.randint(1, deg_max + 1, (L, H, s), generator=g, dtype=torch.int32).to(DEV)
    return K, V, deg


def run_gpu_prefill(K, V, deg, p, want_assign=True, cap_extra=3):
    b = B()
    L, H, s, D = K.shape
    src = b.Cache(K, V, deg, None, s)
    out_len, rounds, cap = b.compress_plan(s, p)
    dst = b.Cache.empty(L, H, cap + cap_extra, D, K.dtype, DEV)
    ws = torch.empty(b.workspace_bytes(src, p), dtype=torch.uint8, device=DEV)
    assign = torch.full((L, H, s), -7, dtype=torch.int32, device=DEV) if want_assign else None
    r = b.compress_prefill(src, dst, p, ws, assign)
    assert b.workspace_status(ws) == 0      # synchronises; nonzero would mean a bounded wait gave up
    assert r == rounds and dst.len == out_len
    return dst, assign, rounds


def single_round_case(L, H, s, dtype, p, seed, deg_max=1, **kw):
    """One round on the GPU against one oracle round; p must describe exactly one round."""
    K, V, deg = make_inputs(L, H, s, dtype, seed, deg_max=deg_max, **kw)
    dst, assign, rounds = run_gpu_prefill(K, V, deg, p)
    assert rounds == 1
    po = PU.oracle_params(p)
    degn = deg.cpu().numpy().astype(np.int64) if deg is not None else np.ones((L, H, s), dtype=np.int64)
    stats = {}
    PU.check_round(PU.to_np64(K), PU.to_np64(V), degn, PU.gpu_cache_to_np(dst, assign), po, O.ratio_for_round(po, 0), dtype, stats)
    PU.report_near_ties(stats, f"one round, chunk {p.chunk}, {L}x{H}x{s} {dtype}")
    return stats


def one_round(b, chunk, r, select, sink=0, recent=0, budget=0):
    return b.Params(chunk=chunk, n_sink=sink, n_recent=recent, n_rounds_max=1, r_init=r, r_decay=0.0, r_min=r,
                    select=select, budget=budget)


def test_config1_tiny_fp32():
    """1 layer, 1 KV head, seq 2048, d 128, fp32, AR(1) rho 0.9, chunk 64, retain 50 %, seed 0."""
    b = B()
    stats = single_round_case(1, 1, 2048, "f32", one_round(b, 64, 1.0, b.SELECT_GLOBAL), seed=0, rho=(0.9, 0.9), mean_std=0.0)
    assert stats["edges"] == 1024


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("chunk,s,sink,recent", [(64, 1000, 16, 64), (64, 517, 0, 0), (2, 37, 1, 0), (4, 50, 0, 3), (8, 131, 5, 6),
                                                 (128, 700, 16, 64), (256, 1100, 16, 64), (256, 300, 0, 0), (6, 64, 2, 2)])
def test_round_all_edges(dtype, chunk, s, sink, recent):
    """Ratio 1: every edge merges; ragged last chunks, odd chunks, single-token chunks, degrees > 1 on input."""
    b = B()
    single_round_case(2, 3, s, dtype, one_round(b, chunk, 1.0, b.SELECT_GLOBAL, sink, recent), seed=chunk + s, deg_max=5)


@pytest.mark.parametrize("deg_max", [1, 7])
@pytest.mark.parametrize("s,sink,recent", [(64, 0, 0), (8192, 0, 0), (8229, 0, 0), (4000, 16, 64), (12345, 3, 1)])
def test_round_bf16_chunk64_ratio1(deg_max, s, sink, recent):
    """The configuration the benchmark times (bf16, chunk 64, ratio 1): many full chunks per head plus a shorter
    last one, with and without degrees on input."""
    b = B()
    single_round_case(3, 5, s, "bf16", one_round(b, 64, 1.0, b.SELECT_GLOBAL, sink, recent), seed=s + deg_max, deg_max=deg_max)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("chunk,s,r", [(64, 1000, 0.5), (8, 131, 0.34), (256, 1100, 0.8), (64, 517, 0.2), (4, 50, 0.5)])
def test_round_chunk_top_m(dtype, chunk, s, r):
    b = B()
    single_round_case(2, 2, s, dtype, one_round(b, chunk, r, b.SELECT_CHUNK, 3, 9), seed=7 * chunk + s, deg_max=3)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("chunk,s,r,budget", [(64, 3000, 0.6, 0), (8, 131, 0.34, 0), (256, 2500, 0.8, 0), (64, 5000, 0.8, 4000),
                                              (64, 1200, 0.05, 0), (2, 300, 0.5, 0)])
def test_round_global_top_m(dtype, chunk, s, r, budget):
    """Ranking across all chunks of a head; with a budget the merge count is trimmed onto it."""
    b = B()
    single_round_case(2, 2, s, dtype, one_round(b, chunk, r, b.SELECT_GLOBAL, 16, 64, budget), seed=3 * chunk + s, deg_max=3)


@pytest.mark.parametrize("dtype,c", [("f32", 64), ("bf16", 64), ("bf16", 128), ("bf16", 256), ("f32", 6), ("bf16", 0)])
def test_identical_keys_tie_to_lowest_index(dtype, c):
    """All keys of a chunk equal: every similarity ties at 1, the first B token must win, the centroid key is that key.
    Without chunks (c = 0) the whole head is one chunk and its first B token collects every A token."""
    b = B()
    L, H, s = 1, 2, 768
    cc = c if c else s
    base = synth.normal_values(L, H, s // cc, 128, seed=3, dtype=dtype, device=DEV)
    K = base.repeat_interleave(cc, dim=2).contiguous()
    V = synth.normal_values(L, H, s, 128, seed=4, dtype=dtype, device=DEV)
    p = one_round(b, c, 1.0, b.SELECT_GLOBAL)
    dst, assign, _ = run_gpu_prefill(K, V, None, p)
    a = assign.cpu().numpy()
    expect = (np.arange(s) // cc) * (cc // 2)            # every A token of chunk i lands in slot of B token 1 of chunk i
    pos = np.arange(s)
    is_a = pos % 2 == 0
    np.testing.assert_array_equal(a[0, 0][is_a], expect[is_a])
    stats = {}
    PU.check_round(PU.to_np64(K), PU.to_np64(V), np.ones((L, H, s), dtype=np.int64), PU.gpu_cache_to_np(dst, assign),
                   PU.oracle_params(p), 1.0, dtype, stats)


def test_zero_keys_and_ratio_zero():
    b = B()
    K, V, _ = make_inputs(1, 2, 200, "f32", seed=9)
    K[:, :, 40:60] = 0          # zero-norm keys: similarity 0 by definition
    p = one_round(b, 8, 1.0, b.SELECT_GLOBAL, 2, 2)
    dst, assign, _ = run_gpu_prefill(K, V, None, p)
    stats = {}
    PU.check_round(PU.to_np64(K), PU.to_np64(V), np.ones((1, 2, 200), dtype=np.int64), PU.gpu_cache_to_np(dst, assign),
                   PU.oracle_params(p), 1.0, "f32", stats)
    # ratio 0: three rounds that merge nothing return the input bit for bit
    p0 = b.Params(chunk=8, n_sink=2, n_recent=2, n_rounds_max=3, r_init=0.0, r_decay=0.0, r_min=0.0, select=b.SELECT_GLOBAL)
    dst, assign, rounds = run_gpu_prefill(K, V, None, p0)
    assert rounds == 3 and dst.len == 200
    assert torch.equal(dst.k[:, :, :200], K) and torch.equal(dst.v[:, :, :200], V)
    assert torch.equal(assign[0, 0].cpu(), torch.arange(200, dtype=torch.int32))
    assert int(dst.deg[:, :, :200].min()) == 1 and int(dst.deg[:, :, :200].max()) == 1


def test_short_sequences_are_copied():
    """Fewer than two tokens between sinks and recent tokens: nothing to cluster."""
    b = B()
    for s in (1, 5, 81):
        K, V, _ = make_inputs(1, 1, s, "bf16", seed=s)
        p = b.Params(chunk=64, n_sink=16, n_recent=64, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0, select=b.SELECT_GLOBAL)
        dst, assign, _ = run_gpu_prefill(K, V, None, p)
        assert dst.len == s and torch.equal(dst.k[:, :, :s], K) and torch.equal(dst.v[:, :, :s], V)


def multi_round_case(L, H, s, dtype, p, seed):
    K, V, _ = make_inputs(L, H, s, dtype, seed)
    return multi_round_check(K, V, dtype, p)


def multi_round_check(K, V, dtype, p):
    """End to end against the oracle's multi-round driver; if a near tie made the GPU choose differently,
    fall back to checking every round against an oracle round fed with the GPU's own previous output.
    Returns the statistics, with the GPU result under "dst" and "assign"."""
    b = B()
    L, H, s, _ = K.shape
    dst, assign, rounds = run_gpu_prefill(K, V, None, p)
    po = PU.oracle_params(p)
    Ko, Vo, do, asg, logs = O.compress_prefill(PU.to_np64(K), PU.to_np64(V), None, po, storage=dtype)
    assert len(logs) == rounds and Ko.shape[2] == dst.len
    g = PU.gpu_cache_to_np(dst, assign)
    # invariants that hold whatever the clusters are: degrees sum to the original length (Sec. 3)
    np.testing.assert_array_equal(g["deg"].sum(axis=2), np.full((L, H), s))
    stats = dict(rounds=rounds, dst=dst, assign=assign)
    if np.array_equal(g["assign"], asg):
        np.testing.assert_array_equal(g["deg"], do)
        close = True
        for l in range(L):
            for h in range(H):
                # bf16 storage between rounds can flip a rounding in an earlier round: allow one ulp per round.  Where a
                # flipped centroid later meets members that cancel it, its one ulp is many ulps of the small result:
                # such a run is not accepted here but checked round by round below.
                if dtype == "bf16":
                    diff = np.abs(g["K"][l, h] - Ko[l, h])
                    close &= bool(np.all(diff <= rounds * PU.bf16_ulp(Ko[l, h]) * 1.0001))
                    diff = np.abs(g["V"][l, h] - Vo[l, h])
                    close &= bool(np.all(diff <= rounds * PU.bf16_ulp(Vo[l, h]) * 1.0001 + 1e-30))
                else:
                    PU.compare_values(g["K"][l, h], Ko[l, h], dtype, "K")
                    PU.compare_values(g["V"][l, h], Vo[l, h], dtype, "V")
        if close:
            stats["end_to_end"] = True
            stats["edges"] = sum(len(e.a_pos) for lg in logs for e in lg.edges)
            PU.report_near_ties(stats, f"{rounds} rounds, chunk {p.chunk}, {L}x{H}x{s} {dtype}, end to end")
            return stats
    # round by round on the GPU's own intermediates
    stats["end_to_end"] = False
    cur = b.Cache(K, V, None, None, s)
    for j in range(rounds):
        r = O.ratio_for_round(po, j)
        pj = b.Params(chunk=p.chunk, n_sink=p.n_sink, n_recent=p.n_recent, n_rounds_max=1, r_init=r, r_decay=0.0, r_min=r,
                      select=p.select, budget=p.budget)
        nxt, asg_j, _ = run_gpu_prefill(cur.k[:, :, :cur.len].contiguous(), cur.v[:, :, :cur.len].contiguous(),
                                        cur.deg[:, :, :cur.len].contiguous() if cur.deg is not None else None, pj)
        degn = cur.deg[:, :, :cur.len].cpu().numpy().astype(np.int64) if cur.deg is not None else np.ones((L, H, s), dtype=np.int64)
        PU.check_round(PU.to_np64(cur.k[:, :, :cur.len]), PU.to_np64(cur.v[:, :, :cur.len]), degn,
                       PU.gpu_cache_to_np(nxt, asg_j), PU.oracle_params(pj), r, dtype, stats)
        cur = nxt
    assert cur.len == dst.len
    # the single rounds reproduce the multi-round call: degrees exactly; rows bit for bit, except that two ratio-1 rounds
    # in one pass sum a cluster on the tensor cores, whose fp32 additions may round differently from the scalar sums of a
    # single round: there one bf16 step per round
    assert torch.equal(cur.deg[:, :, :cur.len], dst.deg[:, :, :dst.len])
    for a_, b_ in ((cur.k, dst.k), (cur.v, dst.v)):
        x, y = PU.to_np64(a_[:, :, :cur.len]), PU.to_np64(b_[:, :, :dst.len])
        assert np.all(np.abs(x - y) <= rounds * PU.bf16_ulp(y) * 1.0001 + 1e-30) and np.mean(x == y) >= 0.99
    PU.report_near_ties(stats, f"{rounds} rounds, chunk {p.chunk}, {L}x{H}x{s} {dtype}, round by round")
    return stats


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_two_rounds_ratio_one(dtype):
    """75 % reduction beyond a single pass: two rounds at ratio 1 (64 -> 32 -> 16 per chunk)."""
    b = B()
    p = b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0, select=b.SELECT_GLOBAL)
    st = multi_round_case(2, 2, 4096, dtype, p, seed=21)
    assert st["rounds"] == 2


@pytest.mark.parametrize("s,sink,recent,rounds", [(4096 + 64, 0, 0, 2), (4096 + 64 + 37, 0, 0, 2), (3000, 16, 64, 2), (130, 0, 0, 2),
                                                 (127, 0, 0, 2), (256 + 5, 3, 0, 2), (8192 + 192, 16, 64, 3), (20000, 0, 7, 4)])
def test_rounds_in_one_pass_edges(s, sink, recent, rounds):
    """Two ratio-1 rounds at chunk 64 on a cache without degrees run as one pass over pairs of chunks; an odd chunk, a
    shorter last chunk, sinks and recent tokens take the two rounds one after the other, later rounds follow."""
    b = B()
    p = b.Params(chunk=64, n_sink=sink, n_recent=recent, n_rounds_max=rounds, r_init=1.0, r_decay=0.0, r_min=1.0, select=b.SELECT_CHUNK)
    st = multi_round_case(2, 3, s, "bf16", p, seed=77 + s)
    assert st["rounds"] == rounds


def test_rounds_in_one_pass_without_slot_map():
    """The same call with and without the optional slot map gives the same cache, bit for bit."""
    b = B()
    p = b.Params(chunk=64, n_sink=5, n_recent=9, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0, select=b.SELECT_GLOBAL)
    K, V, _ = make_inputs(2, 2, 5000, "bf16", seed=91)
    d1, _, _ = run_gpu_prefill(K, V, None, p, want_assign=True)
    d2, _, _ = run_gpu_prefill(K, V, None, p, want_assign=False)
    n = d1.len
    assert d2.len == n and torch.equal(d1.k[:, :, :n], d2.k[:, :, :n]) and torch.equal(d1.v[:, :, :n], d2.v[:, :, :n])
    assert torch.equal(d1.deg[:, :, :n], d2.deg[:, :, :n]) and torch.equal(d1.logdeg[:, :, :n], d2.logdeg[:, :, :n])


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("select", [0, 1])
def test_paper_schedule_to_quarter_budget(dtype, select):
    """Defaults of the paper: 16 sinks, 64 recent tokens, r_init 0.8, delta_r 0.2 (floored at 0.2), budget 25 %."""
    b = B()
    s = 6000
    p = b.Params(chunk=64, n_sink=16, n_recent=64, n_rounds_max=16, r_init=0.8, r_decay=0.2, r_min=0.2, select=select, budget=s // 4)
    st = multi_round_case(1, 2, s, dtype, p, seed=33)
    assert st["rounds"] >= 4


def test_chunk256_paper_default():
    b = B()
    s = 9000
    p = b.Params(chunk=256, n_sink=16, n_recent=64, n_rounds_max=16, r_init=0.8, r_decay=0.2, r_min=0.2, select=b.SELECT_GLOBAL, budget=s // 4)
    multi_round_case(1, 2, s, "bf16", p, seed=35)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_append_with_chunk_trigger(dtype):
    """K = [K, k], N = [N, 1]; every completed window of `chunk` appended tokens is clustered 64 -> 32 -> 16."""
    b = B()
    L, H, s0, c = 2, 2, 300, 64
    K, V, _ = make_inputs(L, H, s0, dtype, seed=41)
    p = b.Params(chunk=c, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0, select=b.SELECT_GLOBAL)
    cache = b.Cache.empty(L, H, 700, 128, K.dtype, DEV)
    cache.k[:, :, :s0], cache.v[:, :, :s0] = K, V
    cache.deg[:, :, :s0] = 1
    cache.len = s0
    ws = torch.empty(b.workspace_bytes(cache, p), dtype=torch.uint8, device=DEV)
    Ko, Vo = PU.to_np64(K), PU.to_np64(V)
    do, pend = np.ones((L, H, s0), dtype=np.int64), 0
    po = PU.oracle_params(p)
    total = s0
    for step, t_new in enumerate([1, 1, 30, 40, 64, 150, 1, 63]):
        kn, vn, _ = make_inputs(L, H, t_new, dtype, seed=100 + step)
        b.compress_append(cache, kn, vn, p, ws)
        torch.cuda.synchronize()
        Ko, Vo, do, pend = O.compress_append(Ko, Vo, do, pend, PU.to_np64(kn), PU.to_np64(vn), po, storage=dtype)
        total += t_new
        assert cache.len == Ko.shape[2] and cache.pending == pend
        g = PU.gpu_cache_to_np(cache)
        np.testing.assert_array_equal(g["deg"].sum(axis=2), np.full((L, H), total))
        np.testing.assert_array_equal(g["deg"], do)
        np.testing.assert_allclose(g["logdeg"], np.log(do.astype(np.float64)), rtol=1e-6, atol=1e-7)
        for l in range(L):
            for h in range(H):
                if dtype == "bf16":
                    assert np.all(np.abs(g["K"][l, h] - Ko[l, h]) <= 2 * PU.bf16_ulp(Ko[l, h]) * 1.0001)
                    assert np.all(np.abs(g["V"][l, h] - Vo[l, h]) <= 2 * PU.bf16_ulp(Vo[l, h]) * 1.0001 + 1e-30)
                else:
                    PU.compare_values(g["K"][l, h], Ko[l, h], dtype, "K")
                    PU.compare_values(g["V"][l, h], Vo[l, h], dtype, "V")


@pytest.mark.parametrize("dtype,Bz", [("bf16", 5), ("f32", 3), ("bf16", 70)])
def test_append_batch_in_lock_step(dtype, Bz):
    """One new token per sequence and step, all sequences written by one launch (two past 64 sequences); the sequences
    start with different lengths and different numbers of pending tokens, so their windows complete at different steps.
    Every sequence is replayed by the oracle, and a second set of caches driven one sequence at a time through
    ckv_compress_append must end up identical bit for bit."""
    b = B()
    L, H, c, steps = 2, 2, 64, 70
    p = b.Params(chunk=c, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0, select=b.SELECT_GLOBAL)
    po = PU.oracle_params(p)
    rng = np.random.default_rng(Bz)
    lens = [int(x) for x in rng.integers(1, 200, Bz)]
    pend0 = [int(min(n, x)) for n, x in zip(lens, rng.integers(0, c, Bz))]
    replay = range(Bz) if Bz <= 8 else (0, 63, 64, Bz - 1)      # sequences the oracle follows
    batch, single, oracle = [], [], {}
    for i, n in enumerate(lens):
        K, V, _ = make_inputs(L, H, n, dtype, seed=500 + i)
        for group in (batch, single):
            cache = b.Cache.empty(L, H, n + steps + 3, 128, K.dtype, DEV)
            cache.k[:, :, :n], cache.v[:, :, :n] = K, V
            cache.deg[:, :, :n] = 1
            cache.len, cache.pending = n, pend0[i]
            group.append(cache)
        if i in replay:
            oracle[i] = [PU.to_np64(K), PU.to_np64(V), np.ones((L, H, n), dtype=np.int64), pend0[i]]
    ws = torch.empty(max(b.workspace_bytes(x, p) for x in batch), dtype=torch.uint8, device=DEV)
    for step in range(steps):
        kn, vn, _ = make_inputs(L, H, Bz, dtype, seed=900 + step)
        b.compress_append_batch(batch, kn, vn, p, ws)
        for i, cache in enumerate(single):
            b.compress_append(cache, kn[:, :, i:i + 1].contiguous(), vn[:, :, i:i + 1].contiguous(), p, ws)
        for i, st in oracle.items():
            st[0], st[1], st[2], st[3] = O.compress_append(st[0], st[1], st[2], st[3], PU.to_np64(kn[:, :, i:i + 1]),
                                                           PU.to_np64(vn[:, :, i:i + 1]), po, storage=dtype)
            assert batch[i].len == st[0].shape[2] and batch[i].pending == st[3]
    assert b.workspace_status(ws) == 0
    for x, y in zip(batch, single):
        n = x.len
        assert n == y.len and x.pending == y.pending
        assert torch.equal(x.k[:, :, :n], y.k[:, :, :n]) and torch.equal(x.v[:, :, :n], y.v[:, :, :n])
        assert torch.equal(x.deg[:, :, :n], y.deg[:, :, :n]) and torch.equal(x.logdeg[:, :, :n], y.logdeg[:, :, :n])
    for i, (Ko, Vo, do, _) in oracle.items():
        g = PU.gpu_cache_to_np(batch[i])
        np.testing.assert_array_equal(g["deg"], do)
        np.testing.assert_allclose(g["logdeg"], np.log(do.astype(np.float64)), rtol=1e-6, atol=1e-7)
        for l in range(L):
            for h in range(H):
                if dtype == "bf16":
                    assert np.all(np.abs(g["K"][l, h] - Ko[l, h]) <= 2 * PU.bf16_ulp(Ko[l, h]) * 1.0001)
                    assert np.all(np.abs(g["V"][l, h] - Vo[l, h]) <= 2 * PU.bf16_ulp(Vo[l, h]) * 1.0001 + 1e-30)
                else:
                    PU.compare_values(g["K"][l, h], Ko[l, h], dtype, "K")
                    PU.compare_values(g["V"][l, h], Vo[l, h], dtype, "V")
    # a full cache is refused before anything is enqueued
    batch[0].len = batch[0].cap
    with pytest.raises(b.CkvError) as e:
        b.compress_append_batch(batch, kn, vn, p, ws)
    assert e.value.status == 3


def test_status_codes_on_device_buffers():
    b = B()
    K, V, _ = make_inputs(1, 1, 256, "bf16", seed=1)
    p = b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)
    src = b.Cache(K, V, None, None, 256)
    ws = torch.empty(b.workspace_bytes(src, p), dtype=torch.uint8, device=DEV)
    small = b.Cache.empty(1, 1, 100, 128, K.dtype, DEV)
    with pytest.raises(b.CkvError) as e:
        b.compress_prefill(src, small, p, ws)
    assert e.value.status == 3
    with pytest.raises(b.CkvError) as e:
        b.compress_prefill(src, b.Cache(K, V, src.deg if src.deg is not None else torch.zeros(1, 1, 256, dtype=torch.int32, device=DEV), None, 256), p, ws)
    assert e.value.status == 1      # dst overlaps src
    dst = b.Cache.empty(1, 1, 128, 128, K.dtype, DEV)
    with pytest.raises(b.CkvError) as e:
        b.compress_prefill(src, dst, p, ws[:16])
    assert e.value.status == 4
    pb = b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=4, r_init=0.0, r_decay=0.0, r_min=0.0, budget=100)
    with pytest.raises(b.CkvError) as e:
        b.compress_prefill(src, dst, pb, ws)
    assert e.value.status == 5


@pytest.mark.parametrize("s,sink,recent,r", [(300, 0, 0, 1.0), (1001, 16, 64, 0.5), (2500, 3, 0, 0.8), (130, 0, 1, 0.3), (4096, 0, 0, 1.0)])
def test_no_chunking_single_round(s, sink, recent, r):
    """chunk = 0: every A token against every B token of its head (plain Bipartite Soft Matching), tensor-core matching."""
    b = B()
    single_round_case(2, 2, s, "bf16", one_round(b, 0, r, b.SELECT_GLOBAL, sink, recent), seed=900 + s, deg_max=4)


def test_no_chunking_ranked_per_chunk_is_the_same_thing():
    """With one chunk per head the two ranking scopes coincide; a budget is only trimmed to in the per-head scope."""
    b = B()
    single_round_case(1, 3, 1500, "bf16", one_round(b, 0, 0.5, b.SELECT_CHUNK, 4, 8), seed=77, deg_max=3)
    p = b.Params(chunk=0, n_sink=4, n_recent=8, n_rounds_max=16, r_init=0.6, r_decay=0.2, r_min=0.2, select=b.SELECT_CHUNK, budget=500)
    st = multi_round_case(1, 2, 1500, "bf16", p, seed=78)
    assert st["rounds"] >= 3 and st["dst"].len <= 500


def test_no_chunking_paper_schedule():
    b = B()
    s = 3000
    p = b.Params(chunk=0, n_sink=16, n_recent=64, n_rounds_max=16, r_init=0.8, r_decay=0.2, r_min=0.2, select=b.SELECT_GLOBAL, budget=s // 4)
    st = multi_round_case(1, 2, s, "bf16", p, seed=37)
    assert st["rounds"] >= 4


def test_no_chunking_is_bf16_only():
    b = B()
    K, V, _ = make_inputs(1, 1, 64, "f32", seed=2)
    p = one_round(b, 0, 1.0, b.SELECT_GLOBAL)
    src = b.Cache(K, V, None, None, 64)
    dst = b.Cache.empty(1, 1, 64, 128, K.dtype, DEV)
    ws = torch.empty(max(b.workspace_bytes(src, p), 1 << 20), dtype=torch.uint8, device=DEV)
    with pytest.raises(b.CkvError) as e:
        b.compress_prefill(src, dst, p, ws)
    assert e.value.status == 6


@pytest.mark.parametrize("chunk,ranked", [(64, True), (128, True), (256, True), (64, False), (256, False)])
def test_repeated_schedules_are_bit_identical(chunk, ranked):
    """The launches of a round overlap where they are independent (the shorter last chunk and the copies of sinks and
    recent tokens run beside the round's main kernel).  A missing ordering would show as a run that differs: the same
    schedule (per-head ranking, sinks, recent tokens, shorter last chunks, six rounds) is repeated into fresh, poisoned
    buffers and every run must reproduce the first bit for bit, slot map included."""
    b = B()
    L, H, s = 3, 8, 20000 + chunk // 2 + 7
    K, V, _ = make_inputs(L, H, s, "bf16", seed=77)
    if ranked:
        p = b.Params(chunk=chunk, n_sink=16, n_recent=64, n_rounds_max=16, r_init=0.8, r_decay=0.2, r_min=0.2, budget=s // 4)
    else:  # every edge, three rounds: at chunk 64 the first two run in one pass, with an odd chunk left over
        p = b.Params(chunk=chunk, n_sink=16, n_recent=64, n_rounds_max=3, r_init=1.0, r_decay=0.0, r_min=1.0)
    src = b.Cache(K, V, None, None, s)
    out_len, rounds, cap = b.compress_plan(s, p)
    first = None
    for run in range(12):
        dst = b.Cache.empty(L, H, cap, 128, K.dtype, DEV)
        dst.k.fill_(float("nan")); dst.v.fill_(float("nan")); dst.deg.fill_(-1)
        ws = torch.empty(b.workspace_bytes(src, p), dtype=torch.uint8, device=DEV)
        ws.fill_(0xA5 if run % 2 else 0x00)
        assign = torch.full((L, H, s), -7, dtype=torch.int32, device=DEV)
        assert b.compress_prefill(src, dst, p, ws, assign) == rounds and dst.len == out_len
        assert b.workspace_status(ws) == 0
        got = (dst.k[:, :, :out_len].clone(), dst.v[:, :, :out_len].clone(), dst.deg[:, :, :out_len].clone(), assign)
        if first is None:
            first = got
            assert int(got[2].sum()) == L * H * s
        else:
            for x, y in zip(first, got):
                assert torch.equal(x.view(torch.int16) if x.dtype == torch.bfloat16 else x, y.view(torch.int16) if y.dtype == torch.bfloat16 else y)
