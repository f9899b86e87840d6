"""Shared parity checks: CUDA path (through the C ABI) against the CPU oracle.

Tolerances
  indices    bit-exact, except where the oracle's own fp64 similarities show a near tie
             (relative gap below 1e-5 between the two best candidates of an A token, or between an
             edge and the selection threshold); those are counted, and the GPU's choice must be one
             of the near-tied candidates.
  fp32 K/V   |gpu - oracle| <= 1e-3 * |oracle| + 1e-5 (1e-3 relative is the stated bar; the 1e-5
             floor covers values near zero, where a relative bound has no meaning).
  bf16 K/V   gpu == bf16(oracle) up to one bf16 ulp (the kernel rounds an fp32 result, the oracle an
             fp64 one, so values next to a rounding boundary may land on either side), at least 99 % of
             the elements equal bf16(oracle) exactly, and 2e-2 absolute against the unrounded oracle value
             wherever bf16 can resolve it: for |x| >= 2 the format's own spacing (2^-6 and up) makes
             storage rounding plus one ulp exceed 2e-2, so there only the one-ulp rule applies.  The
             fraction within 2e-2 over all elements is returned for the record.
  degrees    exact.  log-degrees 1e-6 relative.
  attention  (Eq. 3) stated bar: 2e-2 absolute for bf16, 2e-4 for fp32.  Beside it, for bf16, a bound that follows
             from the kernel's arithmetic, per output element: the output is rounded to bf16 (half an ulp:
             2^-9 |o|) and the softmax weights enter the weighted sum of V as bf16 (2^-9 relative each, numerator
             and normaliser: 2^-8 * sum_t w_t |v_t|), plus 2e-5 for the fp32 scores and exponentials.  A test
             with cluster degrees also shows that it can see a wrong bias: the oracle with and without Eq. 3's
             log n_t term must differ by at least five times that bound somewhere in the batch.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import ckv_oracle as O

NEAR_TIE = 1e-5


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().double().numpy()


def oracle_params(p) -> O.Params:
    """Oracle parameters from a binding.Params, with the ratios rounded to float32 like the C struct."""
    r_init, r_decay, r_min = p.as_float32()
    return O.Params(chunk=p.chunk, n_sink=p.n_sink, n_recent=p.n_recent, n_rounds_max=p.n_rounds_max, r_init=r_init,
                    r_decay=r_decay, r_min=r_min, budget=p.budget, select=p.select)


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    ax = np.maximum(np.abs(x), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


def compare_values(gpu: np.ndarray, ref: np.ndarray, dtype: str, what: str):
    """gpu: values read back from the GPU (as fp64); ref: oracle fp64 values before storage rounding."""
    if dtype == "f32":
        err = np.abs(gpu - ref)
        bound = 1e-3 * np.abs(ref) + 1e-5
        assert np.all(err <= bound), f"{what}: max excess {np.max(err - bound):.3e}, max err {err.max():.3e}"
        return dict(max_abs=float(err.max()) if err.size else 0.0, frac_2e2=1.0)
    ref_b = O.bf16_round(ref)
    diff = np.abs(gpu - ref_b)
    ulp = bf16_ulp(ref_b)
    # One bf16 step, except where the members of a cluster cancel: Eq. 5 in fp32 carries an absolute error of a few
    # 2^-24 * sum n_i |x_i| / n' <= a few 2^-24 * max |x|, which exceeds the ulp of a centroid much smaller than its members.
    cancel = np.abs(gpu - ref) <= 1e-6 * (np.abs(ref).max() if ref.size else 0.0)
    bad = (diff > ulp * 1.0001) & ~cancel
    assert not bad.any(), f"{what}: more than one bf16 ulp off, max {np.max((diff / ulp)[bad]):.2f} ulp"
    within = np.abs(gpu - ref) <= 2e-2
    frac = float(np.mean(within)) if gpu.size else 1.0
    assert np.all(within | (np.abs(ref) >= 2.0)), f"{what}: an element below 2 in magnitude is more than 2e-2 off"
    assert gpu.size == 0 or np.mean(diff == 0) >= 0.99, f"{what}: only {np.mean(diff == 0):.4f} of the elements round identically"
    return dict(max_abs=float(diff.max()) if diff.size else 0.0, frac_2e2=frac, n_ulp_off=int((diff > 0).sum()))


def decisions_from_assign(assign: np.ndarray, edges: O.Edges):
    """Which of the oracle's candidate edges the GPU merged, and into which B token, read off its
    slot map: a merged A token shares its slot with exactly one B token of its chunk."""
    is_a = np.zeros(len(assign), dtype=bool)
    e_a = edges.a_pos
    is_a[e_a] = True
    owner = np.full(int(assign.max()) + 1, -1, dtype=np.int64)
    others = np.nonzero(~is_a)[0]            # B tokens, sinks, recent tokens, lone tokens: they always survive
    owner[assign[others]] = others
    target = owner[assign[e_a]]
    merged = target >= 0
    return merged, target


def check_round(Kin, Vin, degin, gpu, p_oracle: O.Params, r: float, dtype: str, stats: dict):
    """One clustering round.  Kin, Vin [L,H,s,d] fp64 (storage-rounded), degin [L,H,s] int;
    gpu = dict(K, V, deg, logdeg, assign) as numpy for the same round.  Returns oracle outputs."""
    Ko, Vo, do, asg_o, log = O.csm_round(Kin, Vin, degin, p_oracle, r, storage=None)
    L, H, s, d = Kin.shape
    assert gpu["K"].shape[2] == Ko.shape[2], f"length {gpu['K'].shape[2]} vs oracle {Ko.shape[2]}"
    stats.setdefault("near_tie_argmax", 0)
    stats.setdefault("near_tie_select", 0)
    stats.setdefault("edges", 0)
    for l in range(L):
        for h in range(H):
            e, sel = log.edges[l * H + h], log.selected[l * H + h]
            stats["edges"] += len(e.a_pos)
            ag = gpu["assign"][l, h]
            ref_K, ref_V, ref_d = Ko[l, h], Vo[l, h], do[l, h]
            if not np.array_equal(ag, asg_o[l, h]):
                ref_K, ref_V, ref_d = _excuse_and_rebuild(Kin[l, h], Vin[l, h], degin[l, h], ag, e, sel, p_oracle, stats)
            np.testing.assert_array_equal(gpu["deg"][l, h], ref_d)
            compare_values(gpu["K"][l, h], ref_K, dtype, f"K[{l},{h}]")
            compare_values(gpu["V"][l, h], ref_V, dtype, f"V[{l},{h}]")
            if gpu.get("logdeg") is not None:
                np.testing.assert_allclose(gpu["logdeg"][l, h], np.log(ref_d.astype(np.float64)), rtol=1e-6, atol=1e-7)
    return Ko, Vo, do, asg_o, log


def _excuse_and_rebuild(K, V, deg, assign_gpu, e: O.Edges, sel_o, p: O.Params, stats):
    """The GPU's slot map differs from the oracle's: every difference must sit on a near tie of the
    oracle's fp64 similarities; the expected values are then Eq. 5 applied to the GPU's clusters."""
    merged, target = decisions_from_assign(assign_gpu, e)
    assert merged.sum() == sel_o.sum(), "the GPU merged a different number of edges"
    if p.select == O.SELECT_CHUNK:
        for ci in np.unique(e.chunk_id):
            m = e.chunk_id == ci
            assert merged[m].sum() == sel_o[m].sum(), "per-chunk merge count differs"
    sim64 = e.sim64            # the oracle's float64 similarities (its decisions use them rounded to float32)
    for i in np.nonzero(merged != sel_o)[0]:
        # selection flip: the edge must be within the near-tie band of the threshold (the lowest similarity the oracle merged)
        thr = np.min(sim64[sel_o]) if sel_o.any() else np.inf
        scope = (e.chunk_id == e.chunk_id[i]) if p.select == O.SELECT_CHUNK else np.ones(len(sel_o), dtype=bool)
        thr = np.min(sim64[sel_o & scope]) if (sel_o & scope).any() else thr
        assert abs(sim64[i] - thr) <= NEAR_TIE * max(abs(thr), 1e-30), f"edge {i}: selection differs without a near tie"
        stats["near_tie_select"] += 1
    for i in np.nonzero(merged & sel_o & (target != e.b_pos))[0]:
        a, b_g = int(e.a_pos[i]), int(target[i])
        cg = O.cosine_matrix(K[a:a + 1], K[b_g:b_g + 1])[0, 0]
        co = O.cosine_matrix(K[a:a + 1], K[int(e.b_pos[i]):int(e.b_pos[i]) + 1])[0, 0]
        assert e.argmax_gap[i] < NEAR_TIE and abs(cg - co) <= NEAR_TIE * max(abs(co), 1e-30), \
            f"A token {a}: GPU matched {b_g}, oracle {int(e.b_pos[i])}, gap {e.argmax_gap[i]:.3e}"
        stats["near_tie_argmax"] += 1
    # Eq. 5 on the GPU's clusters
    n_out = int(assign_gpu.max()) + 1
    w = deg.astype(np.float64)
    dsum = np.zeros(n_out)
    np.add.at(dsum, assign_gpu, w)
    Ks = np.zeros((n_out, K.shape[1]))
    Vs = np.zeros((n_out, K.shape[1]))
    np.add.at(Ks, assign_gpu, w[:, None] * K)
    np.add.at(Vs, assign_gpu, w[:, None] * V)
    single = np.bincount(assign_gpu, minlength=n_out) == 1
    Kref, Vref = Ks / dsum[:, None], Vs / dsum[:, None]
    first = np.full(n_out, -1)
    first[assign_gpu[::-1]] = np.arange(len(assign_gpu))[::-1]
    Kref[single], Vref[single] = K[first[single]], V[first[single]]   # untouched rows are bit-exact copies
    return Kref, Vref, dsum.astype(np.int64)


# Excused index differences are a subset of the oracle's own near ties, and those are rare on the AR(1) workloads:
# 3.2e-4 of the edges of the 32k workload have a top-two gap below 1e-5 relative (3.8e-5 below 1e-6, the size of the
# kernels' fp32 error).  More excused cases than this bound means the kernel is off in more than rounding.
NEAR_TIE_MAX_FRACTION = 5e-4


def report_near_ties(stats: dict, what: str):
    """One line for the record (the cases the index criterion excuses are logged), and a bound on how many there are."""
    edges, na, ns = stats.get("edges", 0), stats.get("near_tie_argmax", 0), stats.get("near_tie_select", 0)
    print(f"[near ties] {what}: {edges} edges, {na} argmax and {ns} selection decisions differ from the oracle inside the 1e-5 band")
    assert na + ns <= 3 + NEAR_TIE_MAX_FRACTION * edges, f"{what}: {na + ns} excused index differences among {edges} edges"
    return na + ns


def gpu_cache_to_np(cache, assign=None):
    n = cache.len
    out = dict(K=to_np64(cache.k[:, :, :n]), V=to_np64(cache.v[:, :, :n]), deg=cache.deg[:, :, :n].cpu().numpy().astype(np.int64),
               logdeg=cache.logdeg[:, :, :n].cpu().numpy().astype(np.float64) if cache.logdeg is not None else None)
    if assign is not None:
        out["assign"] = assign.cpu().numpy().astype(np.int64)
    return out


ATTN_BAR = {"f32": 2e-4, "bf16": 2e-2}


def check_attention(got, q, K, V, deg, scale, dtype, what, bar=None):
    """Eq. 3 for one sequence: got [H*G, d] from the GPU against the oracle on the same stored cache (K, V [H, n, d]
    float64, deg [H, n] or None).  Returns the achieved error, the arithmetic bound and the bias sensitivity."""
    ref = O.app_attn(q, K, V, deg, scale)
    err = np.abs(got - ref)
    bar = bar if bar is not None else ATTN_BAR[dtype]
    assert err.max() <= bar, f"{what}: max abs error {err.max():.3e} above the stated bar {bar:g}"
    res = dict(err=float(err.max()), bound=float("nan"), sens=float("nan"), n=int(K.shape[1]))
    if dtype == "bf16":
        spread = O.app_attn(q, K, np.abs(V), deg, scale)          # sum_t w_t |v_t|
        bound = 2.0 ** -9 * np.abs(ref) + 2.0 ** -8 * spread + 2e-5
        assert np.all(err <= bound), f"{what}: error {np.max(err / bound):.2f} x the arithmetic bound (max err {err.max():.3e})"
        res["bound"] = float(bound.max())
    if deg is not None and np.any(deg != 1):
        res["sens"] = float(np.abs(ref - O.app_attn(q, K, V, None, scale)).max())
    return res


def summarize_attention(results, what, require_sensitive=True):
    """One line per test for the record; with degrees in play the batch must be able to expose a wrong bias."""
    if not results:   # a batch of empty sequences
        return 0.0
    err = max(r["err"] for r in results)
    bounds = [r["bound"] for r in results if r["bound"] == r["bound"]]
    sens = [r["sens"] for r in results if r["sens"] == r["sens"]]
    line = f"[attention] {what}: max abs err {err:.3e}"
    if bounds:
        line += f", arithmetic bound {max(bounds):.3e}"
    if sens:
        line += f", dropping log n_t moves the output by {max(sens):.3e}"
    print(line)
    # (judged per sequence; a handful of tokens cannot: with one token the output is that token's value whatever the bias)
    judged = [r for r in results if r["sens"] == r["sens"] and r["bound"] == r["bound"] and r["n"] >= 256]
    if require_sensitive and judged:
        assert any(r["sens"] >= 5 * r["bound"] for r in judged), f"{what}: the inputs cannot expose a wrong bias: {judged}"
    return err
