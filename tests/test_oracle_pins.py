"""Pins for the CPU oracle: each test checks oracle/ckv_oracle.py against something
other than itself -- brute force written with plain loops, closed forms, invariants
that follow from the paper's equations, or a textbook routine."""
import itertools
import json
import math
import os

import numpy as np
import pytest
from scipy.special import softmax

from oracle import ckv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_cache(rng, L, H, s, d, ar=0.0):
    K = rng.standard_normal((L, H, s, d))
    if ar > 0:
        for t in range(1, s):
            K[:, :, t] = ar * K[:, :, t - 1] + K[:, :, t]
    V = rng.standard_normal((L, H, s, d))
    return K, V


# ----------------------------------------------------------------------------- P1: brute force on tiny chunks

def brute_round(K, V, deg, n_sink, n_recent, c, M):
    """One round written with plain loops: full cosine matrix, exhaustive choice of
    the M edges with the largest total similarity, explicit member lists (Sec. 5.2, 5.3, Eq. 2, Eq. 5)."""
    s, d = len(K), len(K[0])
    lo, hi = n_sink, s - n_recent

    def cos(i, j):
        dot = sum(K[i][x] * K[j][x] for x in range(d))
        ni = math.sqrt(sum(K[i][x] ** 2 for x in range(d)))
        nj = math.sqrt(sum(K[j][x] ** 2 for x in range(d)))
        return dot / (ni * nj)

    edges = []  # (a, b, sim)
    start = lo
    while start < hi and hi - lo >= 2:
        end = min(start + c, hi)
        odd_1idx = [p for p in range(start, end) if (p - start + 1) % 2 == 1]   # 1-indexed odd = set A
        even_1idx = [p for p in range(start, end) if (p - start + 1) % 2 == 0]  # set B
        for a in odd_1idx:
            best, best_s = None, None
            for b in even_1idx:
                sc = cos(a, b)
                if best is None or sc > best_s:
                    best, best_s = b, sc
            if best is not None:
                edges.append((a, best, best_s))
        start = end
    best_subset, best_total = (), -1e300
    for sub in itertools.combinations(range(len(edges)), M):
        tot = sum(edges[i][2] for i in sub)
        if tot > best_total + 1e-15:
            best_subset, best_total = sub, tot
    clusters = {}
    gone = set()
    for i in best_subset:
        a, b, _ = edges[i]
        clusters.setdefault(b, [b]).append(a)
        gone.add(a)
    Ko, Vo, do = [], [], []
    for p in range(s):
        if p in gone:
            continue
        mem = clusters.get(p, [p])
        n = sum(deg[m] for m in mem)
        Ko.append([sum(deg[m] * K[m][x] for m in mem) / n for x in range(d)])
        Vo.append([sum(deg[m] * V[m][x] for m in mem) / n for x in range(d)])
        do.append(n)
    return np.array(Ko), np.array(Vo), np.array(do), len(edges)


@pytest.mark.parametrize("c", [4, 6, 8])
@pytest.mark.parametrize("r", [1.0, 0.5, 0.34])
@pytest.mark.parametrize("sink,recent,s", [(0, 0, 16), (1, 2, 19), (3, 0, 12)])
def test_p1_brute_force_rounds(c, r, sink, recent, s):
    rng = np.random.default_rng(100 * c + s)
    K, V = rand_cache(rng, 1, 1, s, 5, ar=0.7)
    deg = np.ones((1, 1, s), dtype=np.int64)
    p = O.Params(chunk=c, n_sink=sink, n_recent=recent, select=O.SELECT_GLOBAL, budget=0)
    for _ in range(3):  # three rounds: degrees > 1 enter the later ones
        Ko, Vo, do, _, log = O.csm_round(K, V, deg, p, r)
        n_edges = len(log.edges[0].a_pos)
        M = int(math.floor(r * n_edges + 1e-9))
        Kb, Vb, db, n_edges_b = brute_round(K[0, 0].tolist(), V[0, 0].tolist(), deg[0, 0].tolist(), sink, recent, c, M)
        assert n_edges == n_edges_b
        assert Ko.shape[2] == Kb.shape[0] == K.shape[2] - M
        np.testing.assert_allclose(Ko[0, 0], Kb, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(Vo[0, 0], Vb, rtol=1e-12, atol=1e-12)
        np.testing.assert_array_equal(do[0, 0], db)
        K, V, deg = Ko, Vo, do


@pytest.mark.parametrize("r,sink,recent,s", [(1.0, 0, 0, 12), (0.5, 2, 1, 15), (0.34, 0, 3, 13)])
def test_no_chunking_is_plain_bipartite_soft_matching(r, sink, recent, s):
    """chunk = 0: the whole middle region is one chunk (the "w/o chunk" ablation): brute force with a chunk larger than
    the sequence, two rounds; the similarity step then costs n^2 d / 4 multiply-adds (Table 1, BSM)."""
    rng = np.random.default_rng(200 + s)
    K, V = rand_cache(rng, 1, 1, s, 5, ar=0.7)
    deg = np.ones((1, 1, s), dtype=np.int64)
    p = O.Params(chunk=0, n_sink=sink, n_recent=recent, select=O.SELECT_GLOBAL, budget=0)
    for _ in range(2):
        Ko, Vo, do, _, log = O.csm_round(K, V, deg, p, r)
        n_edges = len(log.edges[0].a_pos)
        mid = K.shape[2] - sink - recent
        assert n_edges == (mid + 1) // 2 and log.macs == ((mid + 1) // 2) * (mid // 2) * 5
        M = int(math.floor(r * n_edges + 1e-9))
        Kb, Vb, db, _ = brute_round(K[0, 0].tolist(), V[0, 0].tolist(), deg[0, 0].tolist(), sink, recent, 10 ** 9, M)
        np.testing.assert_allclose(Ko[0, 0], Kb, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(Vo[0, 0], Vb, rtol=1e-12, atol=1e-12)
        np.testing.assert_array_equal(do[0, 0], db)
        K, V, deg = Ko, Vo, do


def test_p1_chunk_mode_is_per_chunk_top_m():
    rng = np.random.default_rng(7)
    s, c = 24, 8
    K, V = rand_cache(rng, 1, 1, s, 4, ar=0.5)
    deg = np.ones((1, 1, s), dtype=np.int64)
    p = O.Params(chunk=c, n_sink=0, n_recent=0, select=O.SELECT_CHUNK)
    Ko, Vo, do, _, _ = O.csm_round(K, V, deg, p, 0.5)
    outs = []
    for i in range(s // c):  # each chunk on its own, brute force, M = floor(0.5 * 4) = 2
        sl = slice(i * c, (i + 1) * c)
        Kb, Vb, db, _ = brute_round(K[0, 0, sl].tolist(), V[0, 0, sl].tolist(), [1] * c, 0, 0, c, 2)
        outs.append((Kb, Vb, db))
    np.testing.assert_allclose(Ko[0, 0], np.concatenate([o[0] for o in outs]), rtol=1e-12)
    np.testing.assert_allclose(Vo[0, 0], np.concatenate([o[1] for o in outs]), rtol=1e-12)
    np.testing.assert_array_equal(do[0, 0], np.concatenate([o[2] for o in outs]))


def test_hand_worked_example():
    """A four-token chunk small enough to do on paper (Eq. 2, Eq. 5); numbers in tests/golden/hand_example.json."""
    g = json.load(open(os.path.join(GOLDEN, "hand_example.json")))
    K = np.array(g["K"], dtype=np.float64)[None, None]
    V = np.array(g["V"], dtype=np.float64)[None, None]
    deg = np.array(g["deg"], dtype=np.int64)[None, None]
    p = O.Params(chunk=4, n_sink=0, n_recent=0)
    Ko, Vo, do, asg, log = O.csm_round(K, V, deg, p, 1.0)
    np.testing.assert_array_equal(log.edges[0].b_pos, g["edge_b"])
    np.testing.assert_allclose(log.edges[0].sim, g["edge_sim"], rtol=1e-6)
    np.testing.assert_allclose(Ko[0, 0], g["K_out"], rtol=1e-12)
    np.testing.assert_allclose(Vo[0, 0], g["V_out"], rtol=1e-12)
    np.testing.assert_array_equal(do[0, 0], g["deg_out"])
    np.testing.assert_array_equal(asg[0, 0], g["assign"])
    # top-1 of two edges (r = 0.5): only the better edge (token 2 -> 3, cos = 1) is merged
    Ko, Vo, do, asg, _ = O.csm_round(K, V, deg, p, 0.5)
    np.testing.assert_array_equal(do[0, 0], g["deg_out_half"])
    np.testing.assert_array_equal(asg[0, 0], g["assign_half"])


# ----------------------------------------------------------------------------- P2-P5, P12: fixed points and invariants

def test_p2_ratio_zero_is_identity():
    rng = np.random.default_rng(1)
    K, V = rand_cache(rng, 2, 2, 50, 8, ar=0.8)
    p = O.Params(chunk=8, n_sink=3, n_recent=5, r_init=0.0, r_decay=0.0, r_min=0.0, n_rounds_max=3, budget=0)
    Ko, Vo, do, asg, logs = O.compress_prefill(K, V, None, p)
    assert len(logs) == 3
    np.testing.assert_array_equal(Ko, K)
    np.testing.assert_array_equal(Vo, V)
    np.testing.assert_array_equal(do, np.ones((2, 2, 50)))
    np.testing.assert_array_equal(asg[0, 0], np.arange(50))


def test_p3_identical_keys_merge_to_exact_mean():
    rng = np.random.default_rng(2)
    s, c, d = 32, 8, 6
    K = np.repeat(rng.standard_normal((1, 1, s // c, 1, d)), c, axis=3).reshape(1, 1, s, d)  # one key per chunk
    V = rng.standard_normal((1, 1, s, d))
    deg = rng.integers(1, 5, size=(1, 1, s))
    p = O.Params(chunk=c, n_sink=0, n_recent=0)
    Ko, Vo, do, asg, _ = O.csm_round(K, V, deg, p, 1.0)
    for t in range(Ko.shape[2]):
        mem = np.nonzero(asg[0, 0] == t)[0]
        np.testing.assert_allclose(Ko[0, 0, t], K[0, 0, mem[0]], rtol=1e-15, atol=0)
        w = deg[0, 0, mem]
        np.testing.assert_allclose(Vo[0, 0, t], (w[:, None] * V[0, 0, mem]).sum(0) / w.sum(), rtol=1e-13)
        assert do[0, 0, t] == w.sum()
    # all cosines are 1, so every A token ties over all B tokens and must take the first one
    e = O.match_head(K[0, 0], 0, 0, c)
    np.testing.assert_array_equal(e.b_pos, (e.a_pos // c) * c + 1)


@pytest.mark.parametrize("select", [O.SELECT_GLOBAL, O.SELECT_CHUNK])
def test_p4_p5_degree_and_first_moment_conservation(select):
    rng = np.random.default_rng(3)
    L, H, s, d = 2, 3, 203, 8
    K, V = rand_cache(rng, L, H, s, d, ar=0.9)
    p = O.Params(chunk=16, n_sink=4, n_recent=7, r_init=0.8, r_decay=0.2, r_min=0.2, budget=s // 4, select=select,
                 n_rounds_max=40)
    Ko, Vo, do, asg, logs = O.compress_prefill(K, V, None, p)
    assert len(logs) >= 2
    if select == O.SELECT_GLOBAL:
        assert Ko.shape[2] == s // 4           # the last round is trimmed onto the budget
    else:
        assert Ko.shape[2] <= s // 4
    np.testing.assert_array_equal(do.sum(axis=2), np.full((L, H), s))
    np.testing.assert_allclose((do[..., None] * Ko).sum(axis=2), K.sum(axis=2), rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose((do[..., None] * Vo).sum(axis=2), V.sum(axis=2), rtol=1e-10, atol=1e-10)
    # assign really is the cluster map: degree = member count, centroid = member mean (all original degrees are 1)
    for t in range(0, Ko.shape[2], 7):
        mem = np.nonzero(asg[1, 2] == t)[0]
        assert do[1, 2, t] == len(mem)
        np.testing.assert_allclose(Ko[1, 2, t], K[1, 2, mem].mean(axis=0), rtol=1e-10, atol=1e-12)


def test_p4_append_keeps_degree_sum_and_triggers_per_chunk():
    rng = np.random.default_rng(4)
    L, H, s, d, c = 1, 2, 40, 4, 8
    K, V = rand_cache(rng, L, H, s, d, ar=0.8)
    deg = np.ones((L, H, s), dtype=np.int64)
    p = O.Params(chunk=c, r_init=1.0, r_decay=0.0, r_min=1.0, n_rounds_max=2, budget=0)
    kn, vn = rand_cache(rng, L, H, 21, d, ar=0.8)
    Ka, Va, da, pend = O.compress_append(K, V, deg, 0, kn, vn, p)
    # 21 new tokens = two full windows (8 -> 4 -> 2 each) + 5 pending
    assert pend == 5 and Ka.shape[2] == s + 2 + 2 + 5
    np.testing.assert_array_equal(da.sum(axis=2), np.full((L, H), s + 21))
    np.testing.assert_array_equal(Ka[:, :, :s], K)                 # the old cache is not touched
    np.testing.assert_array_equal(Ka[:, :, -5:], kn[:, :, -5:])    # pending tokens are stored verbatim
    np.testing.assert_allclose((da[..., None] * Va).sum(axis=2), V.sum(axis=2) + vn.sum(axis=2), rtol=1e-10)


@pytest.mark.parametrize("r,g", [(1.0, 3), (0.5, 4), (0.3, 2)])
def test_fixed_budget_trigger_replayed_with_brute_force_rounds(r, g):
    """Algorithm 1's decoding branch: the cache is re-clustered whenever it reaches B + g tokens.  Replay: plain
    concatenation token by token and, at each trigger, the brute-force round on the whole cache with
    M = min(floor(r * n_edges), s - B) merges."""
    rng = np.random.default_rng(11)
    s0, d, c, B, sink, recent = 14, 4, 6, 14, 2, 3
    K, V = rand_cache(rng, 1, 1, s0, d, ar=0.7)
    deg = np.ones((1, 1, s0), dtype=np.int64)
    kn, vn = rand_cache(rng, 1, 1, 11, d, ar=0.7)
    p = O.Params(chunk=c, n_sink=sink, n_recent=recent, r_init=r, r_decay=0.1, r_min=0.1, budget=B, select=O.SELECT_GLOBAL)
    Ko, Vo, do, calls = O.append_recluster(K, V, deg, kn, vn, p, g)
    Kb, Vb, db, n_calls = K[0, 0], V[0, 0], deg[0, 0], 0
    for t in range(kn.shape[2]):
        Kb = np.concatenate([Kb, kn[0, 0, t:t + 1]])
        Vb = np.concatenate([Vb, vn[0, 0, t:t + 1]])
        db = np.concatenate([db, [1]])
        if len(Kb) >= B + g:
            s = len(Kb)
            mid = s - sink - recent
            n_edges = (mid // c) * (c // 2) + ((mid % c + 1) // 2 if mid % c >= 2 else 0)
            M = min(int(math.floor(r * n_edges + 1e-9)), s - B)
            Kb, Vb, db, ne = brute_round(Kb.tolist(), Vb.tolist(), db.tolist(), sink, recent, c, M)
            assert ne == n_edges and len(Kb) == s - M
            n_calls += 1
    assert calls == n_calls >= 2
    np.testing.assert_allclose(Ko[0, 0], Kb, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(Vo[0, 0], Vb, rtol=1e-12, atol=1e-12)
    np.testing.assert_array_equal(do[0, 0], db)
    assert do.sum() == s0 + kn.shape[2]                            # every token ever written is accounted for (Sec. 3)
    np.testing.assert_array_equal(Ko[0, 0, :sink], K[0, 0, :sink])  # sinks are never merged


def test_p12_at_most_half_and_borders_untouched():
    rng = np.random.default_rng(5)
    s, n1, n2 = 101, 6, 9
    K, V = rand_cache(rng, 1, 2, s, 8, ar=0.9)
    deg = rng.integers(1, 4, size=(1, 2, s))
    p = O.Params(chunk=10, n_sink=n1, n_recent=n2)
    Ko, Vo, do, _, log = O.csm_round(K, V, deg, p, 1.0)
    m = s - n1 - n2
    assert log.s_out >= s - m // 2
    assert log.s_out == s - sum(len(range(0, min(10, m - b), 2)) if min(10, m - b) >= 2 else 0 for b in range(0, m, 10))
    np.testing.assert_array_equal(Ko[:, :, :n1], K[:, :, :n1])
    np.testing.assert_array_equal(Vo[:, :, -n2:], V[:, :, -n2:])
    np.testing.assert_array_equal(do[:, :, :n1], deg[:, :, :n1])
    np.testing.assert_array_equal(do[:, :, -n2:], deg[:, :, -n2:])


def test_odd_and_single_token_chunks():
    rng = np.random.default_rng(6)
    # middle of 9 tokens with c = 4: chunks of 4, 4 and 1 -> the lone token passes through and draws no edge
    K, V = rand_cache(rng, 1, 1, 9, 4)
    e = O.match_head(K[0, 0], 0, 0, 4)
    assert len(e.a_pos) == 4 and 8 not in e.a_pos
    # middle of 7 with c = 4: last chunk has 3 tokens: A = {4, 6}, B = {5}
    e = O.match_head(K[0, 0, :7], 0, 0, 4)
    np.testing.assert_array_equal(e.a_pos, [0, 2, 4, 6])
    np.testing.assert_array_equal(e.b_pos[2:], [5, 5])


def test_zero_norm_key_has_zero_similarity():
    K = np.array([[0.0, 0.0], [1.0, 0.0], [1.0, 1.0], [0.0, 2.0]])
    e = O.match_head(K, 0, 0, 4)
    assert e.sim[0] == 0.0 and e.b_pos[0] == 1     # all-zero row: every candidate scores 0, first one wins


def test_ranking_ties_go_to_lower_position():
    # two chunks with identical content: equal similarities; M = 1 must take the edge at the lower position
    base = np.array([[1.0, 0.2], [1.0, 0.0], [0.0, 1.0], [0.3, 1.0]])
    K = np.concatenate([base, base])[None, None]
    V = np.zeros_like(K)
    deg = np.ones((1, 1, 8), dtype=np.int64)
    e = O.match_head(K[0, 0], 0, 0, 4)
    sel, _ = O.select_edges(e, 0.25, 8, 0, O.SELECT_GLOBAL)
    assert sel.sum() == 1 and e.a_pos[sel][0] == int(e.a_pos[np.argmax(e.sim)])
    assert e.a_pos[sel][0] < 4


def test_schedule_eq4_with_floor():
    p = O.Params(r_init=0.8, r_decay=0.2, r_min=0.2)
    np.testing.assert_allclose([O.ratio_for_round(p, j) for j in range(6)], [0.8, 0.6, 0.4, 0.2, 0.2, 0.2], atol=1e-12)
    assert O.merges_from_ratio(0.6, 10) == 6 and O.merges_from_ratio(0.8, 7) == 5 and O.merges_from_ratio(0.2, 4) == 0


# ----------------------------------------------------------------------------- P6-P9: attention

def textbook_attention(q, K, V, scale):
    return softmax((q @ K.T) * scale, axis=-1) @ V


def test_p6_unit_degrees_give_softmax_attention():
    rng = np.random.default_rng(10)
    H, G, s, d = 2, 3, 37, 16
    q = rng.standard_normal((H * G, d))
    K, V = rng.standard_normal((H, s, d)), rng.standard_normal((H, s, d))
    out = O.app_attn(q, K, V, np.ones((H, s), dtype=np.int64), 1 / math.sqrt(d))
    for j in range(H * G):
        np.testing.assert_allclose(out[j], textbook_attention(q[j], K[j // G], V[j // G], 1 / math.sqrt(d)), rtol=1e-12)
    np.testing.assert_allclose(O.attn(q, K, V, 1 / math.sqrt(d)), out, rtol=1e-14)


def test_p7_zero_query_returns_mean_of_original_values():
    rng = np.random.default_rng(11)
    K, V = rand_cache(rng, 1, 2, 96, 8, ar=0.9)
    p = O.Params(chunk=16, n_sink=2, n_recent=3, r_init=0.8, r_decay=0.2, r_min=0.2, budget=30)
    Ko, Vo, do, _, _ = O.compress_prefill(K, V, None, p)
    out = O.app_attn(np.zeros((2, 8)), Ko[0], Vo[0], do[0], 0.3)
    np.testing.assert_allclose(out, V[0].mean(axis=1), rtol=1e-11, atol=1e-12)


def test_p8_replication_identity():
    rng = np.random.default_rng(12)
    H, s, d = 2, 11, 8
    q = rng.standard_normal((H * 2, d))
    K, V = rng.standard_normal((H, s, d)), rng.standard_normal((H, s, d))
    deg = rng.integers(1, 6, size=(H, s))
    out = O.app_attn(q, K, V, deg, 0.4)
    for j in range(H * 2):
        h = j // 2
        Kr, Vr = np.repeat(K[h], deg[h], axis=0), np.repeat(V[h], deg[h], axis=0)
        np.testing.assert_allclose(out[j], textbook_attention(q[j], Kr, Vr, 0.4), rtol=1e-12)


def test_p9_duplicated_keys_make_the_approximation_exact():
    rng = np.random.default_rng(13)
    s, d, c = 64, 8, 16
    K = rng.standard_normal((1, 1, s, d))
    K[:, :, 0::2] = K[:, :, 1::2]                       # every A token carries its right neighbour's key
    V = rng.standard_normal((1, 1, s, d))
    p = O.Params(chunk=c, n_sink=0, n_recent=0, r_init=1.0, r_decay=0, r_min=1.0, n_rounds_max=1)
    Ko, Vo, do, asg, _ = O.compress_prefill(K, V, None, p)
    np.testing.assert_array_equal(asg[0, 0], np.arange(s) // 2)
    np.testing.assert_allclose(Ko[0, 0], K[0, 0, 1::2], rtol=1e-15)
    q = rng.standard_normal((1, d))
    np.testing.assert_allclose(O.app_attn(q, Ko[0], Vo[0], do[0], 0.35), textbook_attention(q[0], K[0, 0], V[0, 0], 0.35)[None],
                               rtol=1e-12)


# ----------------------------------------------------------------------------- P10: Theorem A.1

def c_closed_form(n, l):
    """c_{2n,l} as printed in the proof of Theorem A.1."""
    if l % 2 == 0:
        return -l ** 3 / 12 + (2 * n - 1) / 4 * l ** 2 + (6 * n - 1) / 6 * l
    return -l ** 3 / 12 + (2 * n - 1) / 4 * l ** 2 + (12 * n - 5) / 12 * l + (2 * n - 1) / 4


@pytest.mark.parametrize("n", [1, 2, 3, 4, 5])
def test_p10_alternating_partition_is_optimal(n):
    rng = np.random.default_rng(20 + n)
    A0, B0 = O.alternating_partition(2 * n)
    np.testing.assert_array_equal(A0 + 1, np.arange(1, 2 * n, 2))   # {1, 3, ...} in the theorem's 1-indexed notation
    np.testing.assert_array_equal(B0 + 1, np.arange(2, 2 * n + 1, 2))
    for _ in range(5):
        steps = np.sort(rng.random(2 * n - 1))[::-1]                # decreasing, non-negative differences => convex decreasing f
        fvals = np.concatenate([[0.0], -np.cumsum(steps)])           # fvals[dist - 1]
        f = lambda dist: fvals[dist - 1]
        best = max(O.partition_objective(A, [x for x in range(2 * n) if x not in A], f)
                   for A in itertools.combinations(range(2 * n), n))
        assert O.partition_objective(A0, B0, f) >= best - 1e-12


@pytest.mark.parametrize("n", [2, 3, 5, 7])
def test_p10_closed_form_counts(n):
    A0, B0 = O.alternating_partition(2 * n)
    dist = [abs(int(a) - int(b)) for a in A0 for b in B0]
    for i in range(1, n + 1):
        assert dist.count(2 * i - 1) == 2 * n - 2 * i + 1             # |D_{A0,B0,2i-1}|
    for l in range(1, 2 * n - 1):
        lhs = sum((l + 1 - i) * dist.count(i) for i in range(1, l + 1))
        assert abs(lhs - c_closed_form(n, l)) < 1e-9                  # equality case of the proof's bound


# ----------------------------------------------------------------------------- P11, P13

def test_p11_table1_multiply_add_count():
    g = json.load(open(os.path.join(GOLDEN, "table1_macs.json")))
    for case in g["cases"]:
        n, c, d = case["n"], case["c"], case["d"]
        K = np.random.default_rng(0).standard_normal((n, d))
        assert O.match_head(K, 0, 0, c).macs == case["macs"] == n * c * d // 4


def test_p13_ar1_edges_join_neighbours():
    import torch
    from paper_2506_11418_b200 import synth
    K = synth.ar1_keys(1, 1, 2048, 128, (0.9, 0.9), 0.0, seed=0).double().numpy()
    e = O.match_head(K[0, 0], 0, 0, 64)
    assert np.mean(np.abs(e.a_pos - e.b_pos) == 1) > 0.9
    assert 0.8 < float(np.mean(e.sim)) < 0.97   # E[cos] at distance 1 is about rho = 0.9


def test_paged_attention_does_not_depend_on_where_the_pages_are():
    """A paged cache is the same sequence whatever pages hold it: with the blocks scattered over a larger pool in a
    random order the result equals Eq. 3 on the contiguous cache, which the pins above fix."""
    rng = np.random.default_rng(21)
    H, G, d, P, n = 2, 2, 8, 4, 19
    K, V = rng.standard_normal((H, n, d)), rng.standard_normal((H, n, d))
    deg = rng.integers(1, 5, (H, n))
    q = rng.standard_normal((H * G, d))
    n_blocks, pool = (n + P - 1) // P, 11
    table = rng.permutation(pool)[:n_blocks]
    kp, vp = rng.standard_normal((pool, H, P, d)), rng.standard_normal((pool, H, P, d))   # junk everywhere else
    dp = rng.integers(1, 9, (pool, H, P))
    for t in range(n):
        kp[table[t // P], :, t % P], vp[table[t // P], :, t % P], dp[table[t // P], :, t % P] = K[:, t], V[:, t], deg[:, t]
    np.testing.assert_array_equal(O.gather_pages(kp, table, n), K)
    np.testing.assert_allclose(O.app_attn_paged(q, kp, vp, dp, table, n, 0.3), O.app_attn(q, K, V, deg, 0.3), rtol=1e-13)
    np.testing.assert_allclose(O.app_attn_paged(q, kp, vp, None, table, n, 0.3), textbook_attention_heads(q, K, V, 0.3, G), rtol=1e-12)


def textbook_attention_heads(q, K, V, scale, G):
    return np.stack([softmax(K[j // G] @ q[j] * scale) @ V[j // G] for j in range(q.shape[0])])



# ----------------------------------------------------------------------------- storage rounding (the cache dtype)

def exact_bf16(x: float) -> float:
    """Nearest bfloat16 in exact rational arithmetic: candidates are the two multiples of the format's spacing
    around x; the nearer wins, a tie goes to the even multiple; past the largest finite value it is infinity."""
    from fractions import Fraction
    if x != x or x in (math.inf, -math.inf) or x == 0.0:
        return x
    fx = Fraction(x)
    e = math.frexp(x)[1]                      # |x| in [2^(e-1), 2^e)
    q = Fraction(2) ** max(e - 8, -133)       # 8 significant bits; subnormal spacing 2^-133
    lo = math.floor(fx / q)
    rem = fx / q - lo
    n = lo if rem < Fraction(1, 2) else lo + 1 if rem > Fraction(1, 2) else lo + (lo & 1)
    r = n * q
    if abs(r) >= Fraction(2) ** 128:
        return math.copysign(math.inf, x)
    return math.copysign(float(r), x)


def f32_from_bits(b: int) -> float:
    return float(np.array([b], dtype=np.uint32).view(np.float32)[0])


def bf16_bits(x: float) -> int:
    """Upper 16 bits of the float32 pattern of a value that is exactly a bfloat16."""
    b = int(np.array([x], dtype=np.float32).view(np.uint32)[0])
    assert b & 0xFFFF == 0, "not a bfloat16 value"
    return b >> 16


@pytest.mark.parametrize("bits,expect", [
    (0x3F808000, 0x3F80),   # 1 + 2^-8: halfway, the even neighbour is 1
    (0x3F818000, 0x3F82),   # 1 + 3 * 2^-8: halfway, the even neighbour is 1 + 2^-6
    (0x3F808001, 0x3F81),   # just above a tie
    (0x3F807FFF, 0x3F80),   # just below a tie
    (0xBF808000, 0xBF80),   # ties are symmetric in sign
    (0xBF818000, 0xBF82),
    (0x00000000, 0x0000), (0x80000000, 0x8000),   # signed zeros
    (0x7F800000, 0x7F80), (0xFF800000, 0xFF80),   # infinities
    (0x7F7F0000, 0x7F7F),   # the largest finite bfloat16
    (0x7F7F7FFF, 0x7F7F),   # below the tie with infinity
    (0x7F7F8000, 0x7F80),   # the tie itself goes to the even side: infinity
    (0x00000001, 0x0000),   # smallest fp32 subnormal: far below half of 2^-133
    (0x00008000, 0x0000),   # 2^-134 = half the subnormal spacing: tie to even (zero)
    (0x00008001, 0x0001),   # just above it
    (0x00018000, 0x0002),   # 1.5 * 2^-133: tie, even is 2 * 2^-133
    (0x007F8000, 0x0080),   # the largest subnormals round up into the smallest normal
])
def test_bf16_round_hand_written_bit_patterns(bits, expect):
    got = float(O.bf16_round(f32_from_bits(bits)))
    assert bf16_bits(got) == expect
    assert bf16_bits(exact_bf16(f32_from_bits(bits))) == expect      # the rational restatement agrees with the hand values


def test_bf16_round_keeps_nan_and_rounds_float64_once():
    assert np.isnan(O.bf16_round(np.nan)) and np.isnan(O.round_to_dtype(np.array([np.nan]), "bf16"))[0]
    # 1 + 2^-8 + 2^-40 lies above the tie; rounding through float32 first would land on the tie and go down
    assert float(O.bf16_round(1 + 2.0 ** -8 + 2.0 ** -40)) == 1 + 2.0 ** -7
    assert float(O.bf16_round(1 + 2.0 ** -8 - 2.0 ** -40)) == 1.0
    assert float(O.bf16_round(-(1 + 3 * 2.0 ** -8 + 2.0 ** -45))) == -(1 + 2.0 ** -6)


def test_bf16_round_agrees_with_rational_arithmetic_and_with_torch():
    import torch
    rng = np.random.default_rng(7)
    bits = rng.integers(0, 2 ** 32, size=1_000_000, dtype=np.uint64).astype(np.uint32)
    x32 = bits.view(np.float32)
    keep = ~np.isnan(x32)
    x32 = x32[keep]
    ours = O.bf16_round(x32.astype(np.float64)).astype(np.float32).view(np.uint32)
    theirs = torch.from_numpy(x32.copy()).to(torch.bfloat16).to(torch.float32).numpy().view(np.uint32)
    np.testing.assert_array_equal(ours, theirs)
    # float64 inputs (what the oracle actually rounds), against exact rational arithmetic
    x64 = np.concatenate([rng.standard_normal(20000) * np.exp(rng.uniform(-30, 30, 20000)),
                          (1 + rng.integers(0, 256, 2000) / 128.0 + 2.0 ** -8) * 2.0 ** rng.integers(-20, 20, 2000)])  # exact ties
    got = O.bf16_round(x64)
    want = np.array([exact_bf16(float(v)) for v in x64])
    np.testing.assert_array_equal(got, want)


def test_round_to_dtype_f32_is_round_to_nearest_even():
    import struct
    assert float(O.round_to_dtype(np.array([1 + 2.0 ** -24]), "f32")[0]) == 1.0                 # tie, even is 1
    assert float(O.round_to_dtype(np.array([1 + 3 * 2.0 ** -24]), "f32")[0]) == 1 + 2.0 ** -22  # tie, even is 1 + 2^-22
    assert float(O.round_to_dtype(np.array([1 + 2.0 ** -24 + 2.0 ** -50]), "f32")[0]) == 1 + 2.0 ** -23
    rng = np.random.default_rng(8)
    x = rng.standard_normal(5000) * np.exp(rng.uniform(-20, 20, 5000))
    want = np.array([struct.unpack("f", struct.pack("f", float(v)))[0] for v in x])
    np.testing.assert_array_equal(O.round_to_dtype(x, "f32"), want)
    with pytest.raises(ValueError):
        O.round_to_dtype(x, "fp8")


@pytest.mark.parametrize("select", [O.SELECT_GLOBAL, O.SELECT_CHUNK])
def test_multi_round_driver_rounds_to_storage_between_rounds(select):
    """Algorithm 1 reassigns K, V after every call of CentroidKV; with a bf16 cache each reassignment is a rounding.
    Replay three rounds by brute force, rounding the rows with exact rational arithmetic in between."""
    rng = np.random.default_rng(31)
    s, c, d = 24, 8, 5
    K, V = rand_cache(rng, 1, 1, s, d, ar=0.7)
    K, V = O.round_to_dtype(K, "bf16"), O.round_to_dtype(V, "bf16")
    p = O.Params(chunk=c, n_sink=1, n_recent=2, n_rounds_max=3, r_init=1.0, r_decay=0.25, r_min=0.5, budget=0, select=select)
    Ko, Vo, do, _, logs = O.compress_prefill(K, V, None, p, storage="bf16")
    assert len(logs) == 3
    Kb, Vb, db = K[0, 0].tolist(), V[0, 0].tolist(), [1] * s
    for j in range(3):
        r = max(p.r_init - j * p.r_decay, p.r_min)
        if select == O.SELECT_GLOBAL:
            n_edges = len(logs[j].edges[0].a_pos)
            M = int(math.floor(r * n_edges + 1e-9))
            Kn, Vn, dn, _ = brute_round(Kb, Vb, db, 1, 2, c, M)
        else:
            Kn, Vn, dn = brute_round_per_chunk(Kb, Vb, db, 1, 2, c, r)
        Kb = [[exact_bf16(float(x)) for x in row] for row in Kn]
        Vb = [[exact_bf16(float(x)) for x in row] for row in Vn]
        db = list(dn)
    np.testing.assert_array_equal(do[0, 0], np.array(db))
    np.testing.assert_array_equal(Ko[0, 0], np.array(Kb))
    np.testing.assert_array_equal(Vo[0, 0], np.array(Vb))
    # and every stored row is a bfloat16 value
    np.testing.assert_array_equal(Ko, O.bf16_round(Ko))


def brute_round_per_chunk(K, V, deg, n_sink, n_recent, c, r):
    """Per-chunk ranking by brute force: every chunk is a stand-alone call of brute_round with its own count."""
    s = len(K)
    lo, hi = n_sink, s - n_recent
    Ko, Vo, do = [list(x) for x in K[:lo]], [list(x) for x in V[:lo]], list(deg[:lo])
    start = lo
    while start < hi:
        end = min(start + c, hi)
        n_a = (end - start + 1) // 2 if end - start >= 2 else 0
        M = int(math.floor(r * n_a + 1e-9))
        Kc, Vc, dc, _ = brute_round(K[start:end], V[start:end], deg[start:end], 0, 0, c, M)
        Ko += Kc.tolist(); Vo += Vc.tolist(); do += dc.tolist()
        start = end
    Ko += [list(x) for x in K[hi:]]; Vo += [list(x) for x in V[hi:]]; do += list(deg[hi:])
    return np.array(Ko), np.array(Vo), np.array(do)
