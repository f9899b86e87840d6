"""CPU oracle for CentroidKV's hot path: Chunked Soft Matching, degree-weighted
centroid merge, the multi-round / append drivers and approximate attention.

THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, NumPy fp64 restatement of
the paper's algorithm, written so that it can be checked against the paper by eye.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import it.
It shares no code with the CUDA path and never imports it.

Every function names the passage of the paper it follows.  Where the paper is
silent or ambiguous the reading taken is stated next to the code.

Arithmetic: callers pass inputs already rounded to the storage dtype (fp32 or
bf16, see `round_to_dtype`); everything here is fp64, except that a similarity is
rounded to fp32 before it decides an argmax or a ranking, because the kernel takes
those decisions in fp32 and both sides must decide in the same precision.

Pins (tests/test_oracle_pins.py): brute-force matching on chunks of 4-8 tokens (also at
every trigger of the fixed-budget decoding branch),
ratio 0 is the identity, identical keys merge to their exact mean, degree and
first-moment conservation, N = 1 reduces approximate attention to softmax
attention, the q = 0 closed form, the replication identity, the duplicated-key
construction, Theorem A.1 by enumeration, Table 1's multiply-add count, the
at-most-half bound and untouched sinks / recent tokens.
Storage rounding (`bf16_round`, `round_to_dtype`, the `storage=` argument of the drivers): hand-written bit
patterns, agreement with an exact rational-arithmetic rounding and with torch's conversion on a million random
bit patterns, a multi-round brute-force replay that rounds between rounds.
Parity unpinned: nothing in this file; the *quality* of the clusters on real
model caches (the paper's accuracy tables) is outside what it computes.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

SELECT_GLOBAL = 0  # rank the edges of all chunks of one (layer, head) together (Sec. 5.2 last paragraph, Sec. 5.3)
SELECT_CHUNK = 1   # rank inside each chunk


@dataclass
class Params:
    """Algorithm 1's `Require` line plus Eq. 4's schedule."""
    chunk: int = 256          # c; 0 = no chunking (one chunk spans the whole middle region)
    n_sink: int = 16          # n1
    n_recent: int = 64        # n2
    n_rounds_max: int = 8
    r_init: float = 0.8       # Eq. 4
    r_decay: float = 0.2      # Eq. 4's delta_r
    r_min: float = 0.2        # floor on Eq. 4 (the printed schedule reaches 0 before a 25 % budget is met)
    budget: int = 0           # B of Algorithm 1 (counts sinks and recent tokens); 0 = run exactly n_rounds_max rounds
    select: int = SELECT_GLOBAL


# --------------------------------------------------------------------------- dtype rounding

def bf16_round(x):
    """The nearest bfloat16 (8 significant bits, fp32's exponent range, subnormals kept), ties to the even
    significand, overflow to infinity; computed from the float64 value in one rounding and returned as float64."""
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)                                  # |x| = m * 2^e with 0.5 <= m < 1
    quantum = np.ldexp(1.0, np.maximum(e - 8, -133))    # spacing of bfloat16 around x; 2^-133 in the subnormal range
    with np.errstate(invalid="ignore", over="ignore"):
        r = np.rint(x / quantum) * quantum              # np.rint rounds halves to the even integer
        r = np.where(np.abs(r) >= 2.0 ** 128, np.copysign(np.inf, x), r)
    return np.where(np.isfinite(x), r, x)


def round_to_dtype(x, dtype: str):
    """Round an array to the storage dtype ('f32' or 'bf16'); result is float64."""
    if dtype == "f32":
        return np.asarray(x, dtype=np.float32).astype(np.float64)
    if dtype == "bf16":
        return bf16_round(x)
    raise ValueError(dtype)


# --------------------------------------------------------------------------- Sec. 5.2: chunks and the alternating partition

def chunk_bounds(s: int, n_sink: int, n_recent: int, c: int):
    """Sec. 5.2 first paragraph: keep the first n1 (sink) and last n2 (recent)
    tokens, split what lies between into chunks of c tokens.  A shorter last
    chunk is kept and treated like the others (the paper is silent on it)."""
    lo = min(n_sink, s)
    hi = max(lo, s - n_recent)
    if hi - lo < 2:
        return lo, hi, []
    if c == 0:  # no chunking: plain Bipartite Soft Matching over the whole middle region (Sec. 5.2, the "w/o chunk" ablation of Table 8)
        c = hi - lo
    return lo, hi, [(b, min(b + c, hi)) for b in range(lo, hi, c)]


def alternating_partition(c_len: int):
    """Sec. 5.2 last paragraph and Theorem A.1: A = {1, 3, ...}, B = {2, 4, ...}
    in 1-indexed positions of the chunk, i.e. even / odd 0-based offsets.
    A is the set whose tokens draw edges (and are merged away), B receives them."""
    return np.arange(0, c_len, 2), np.arange(1, c_len, 2)


def partition_objective(A, B, f):
    """Objective of Theorem A.1: sum over x in A, y in B of f(|x - y|)."""
    return sum(f(abs(int(x) - int(y))) for x in A for y in B)


# --------------------------------------------------------------------------- Eq. 2 and the matching step

def cosine_matrix(KA, KB):
    """Eq. 2: cos(k_i, k_j) = <k_i, k_j> / (|k_i| |k_j|).  Zero-norm keys get
    similarity 0 (Eq. 2 is undefined there)."""
    dots = KA @ KB.T
    den = np.linalg.norm(KA, axis=1)[:, None] * np.linalg.norm(KB, axis=1)[None, :]
    return np.where(den > 0, dots / np.where(den > 0, den, 1.0), 0.0)


@dataclass
class Edges:
    """One edge per A token that has at least one B candidate (Sec. 5.2, BSM paragraph)."""
    a_pos: np.ndarray            # absolute position of the A token
    b_pos: np.ndarray            # absolute position of its most similar B token
    sim: np.ndarray              # float32 similarity of the edge (decision precision)
    chunk_id: np.ndarray         # chunk the edge belongs to
    argmax_gap: np.ndarray       # relative fp64 gap between best and second-best candidate (inf if one candidate)
    macs: int = 0                # multiply-adds spent on the similarity matrices (Table 1)
    sim64: np.ndarray = None     # the same similarity before it was rounded to float32 (for the record: near ties)


def match_head(K, n_sink, n_recent, c) -> Edges:
    """Sec. 5.2: inside every chunk, each A token draws an edge to its most similar
    B token of the same chunk (row argmax of the A x B cosine matrix).  Ties go to
    the lowest B position.  Keys are the current cache rows (centroids in later
    rounds), not weighted by degree."""
    s, d = K.shape
    _, _, chunks = chunk_bounds(s, n_sink, n_recent, c)
    a_pos, b_pos, sim, cid, gap, sim64 = [], [], [], [], [], []
    macs = 0
    for ci, (beg, end) in enumerate(chunks):
        A, B = alternating_partition(end - beg)
        if len(B) == 0:
            continue  # a one-token chunk: its A token has no candidate and passes through
        S = cosine_matrix(K[beg + A], K[beg + B])
        macs += len(A) * len(B) * d
        S32 = S.astype(np.float32)
        best = np.argmax(S32, axis=1)           # first maximum = lowest B position
        a_pos.extend(beg + A)
        b_pos.extend(beg + B[best])
        sim.extend(S32[np.arange(len(A)), best])
        sim64.extend(S[np.arange(len(A)), best])
        cid.extend([ci] * len(A))
        if len(B) > 1:
            top = np.sort(S, axis=1)[:, ::-1]
            gap.extend((top[:, 0] - top[:, 1]) / np.maximum(np.abs(top[:, 0]), 1e-30))
        else:
            gap.extend([np.inf] * len(A))
    return Edges(np.array(a_pos, dtype=np.int64), np.array(b_pos, dtype=np.int64),
                 np.array(sim, dtype=np.float32), np.array(cid, dtype=np.int64),
                 np.array(gap, dtype=np.float64), macs, np.array(sim64, dtype=np.float64))


# --------------------------------------------------------------------------- Sec. 5.3: which edges are merged

def ratio_for_round(p: Params, j: int) -> float:
    """Eq. 4: r = r_init - j * delta_r, floored at r_min."""
    return max(p.r_init - j * p.r_decay, p.r_min)


def merges_from_ratio(r: float, n_edges: int) -> int:
    """Number of edges kept for merging: floor(r * n_edges) (the paper does not say how it rounds)."""
    return int(np.floor(r * n_edges + 1e-9))


def rank_edges(sim, a_pos):
    """Sec. 5.3: rank candidate matches by similarity, best first; equal
    similarities are ordered by position (the paper does not break ties)."""
    return np.lexsort((a_pos, -sim.astype(np.float64)))


def select_edges(e: Edges, r: float, s: int, budget: int, select: int):
    """Sec. 5.3: only the top fraction r of the ranked edges is merged.
    GLOBAL ranks all edges of the head together and, when a budget is given, never
    merges more than s - B edges, so that the cache lands on the budget.
    CHUNK ranks inside each chunk and keeps floor(r * edges of that chunk)."""
    n = len(e.a_pos)
    selected = np.zeros(n, dtype=bool)
    sel_gap = np.inf
    if select == SELECT_GLOBAL:
        M = merges_from_ratio(r, n)
        if budget > 0:
            M = min(M, max(s - budget, 0))
        order = rank_edges(e.sim, e.a_pos)
        selected[order[:M]] = True
        if 0 < M < n:
            hi_, lo_ = float(e.sim[order[M - 1]]), float(e.sim[order[M]])
            sel_gap = (hi_ - lo_) / max(abs(hi_), 1e-30)
    else:
        for ci in np.unique(e.chunk_id):
            idx = np.nonzero(e.chunk_id == ci)[0]
            M = merges_from_ratio(r, len(idx))
            order = idx[rank_edges(e.sim[idx], e.a_pos[idx])]
            selected[order[:M]] = True
            if 0 < M < len(idx):
                hi_, lo_ = float(e.sim[order[M - 1]]), float(e.sim[order[M]])
                sel_gap = min(sel_gap, (hi_ - lo_) / max(abs(hi_), 1e-30))
    return selected, sel_gap


# --------------------------------------------------------------------------- Eq. 5: degree-weighted merge

def merge_head(K, V, deg, a_pos, b_pos, selected):
    """Eq. 5 and the sentence after it: a cluster is a B token plus every selected A
    token whose edge points at it; its key and value are the degree-weighted means
    of its members and its degree is the sum of their degrees.  Tokens outside any
    cluster pass through unchanged.  Survivors keep their relative order and a
    centroid sits at its B token's place (the paper does not state the order).
    Returns (K', V', deg', assign) with assign[p] = output slot of input token p."""
    s, _ = K.shape
    removed = np.zeros(s, dtype=bool)
    removed[a_pos[selected]] = True
    members = {}
    for a, b in zip(a_pos[selected], b_pos[selected]):
        members.setdefault(int(b), []).append(int(a))
    keep = ~removed
    slot = np.cumsum(keep) - 1
    Kout, Vout, dout = K[keep].astype(np.float64), V[keep].astype(np.float64), deg[keep].astype(np.int64)
    assign = np.empty(s, dtype=np.int64)
    assign[keep] = slot[keep]
    for b, mem in members.items():
        idx = [b] + mem
        w = deg[idx].astype(np.float64)
        n_new = int(deg[idx].sum())
        Kout[slot[b]] = (w[:, None] * K[idx]).sum(axis=0) / n_new
        Vout[slot[b]] = (w[:, None] * V[idx]).sum(axis=0) / n_new
        dout[slot[b]] = n_new
    for a, b in zip(a_pos[selected], b_pos[selected]):
        assign[a] = slot[b]
    return Kout, Vout, dout, assign


# --------------------------------------------------------------------------- one round, the prefill driver, append

@dataclass
class RoundLog:
    r: float
    s_in: int
    s_out: int
    macs: int
    min_argmax_gap: float
    min_select_gap: float
    edges: list = field(default_factory=list)      # per (layer, head): Edges
    selected: list = field(default_factory=list)   # per (layer, head): bool mask over edges


def csm_round(K, V, deg, p: Params, r: float, storage: str | None = None):
    """One call of CentroidKV(K, V, N, s, n1, n2, r, c) in Algorithm 1, for every
    (layer, head) independently (Sec. 3 works per head).  K, V: [L, H, s, d]; deg: [L, H, s].
    When `storage` is given the merged rows are rounded to that dtype, as a cache
    that stores bf16 or fp32 does between rounds."""
    L, H, s, d = K.shape
    outs, log = [], RoundLog(r, s, s, 0, np.inf, np.inf)
    for l in range(L):
        for h in range(H):
            e = match_head(K[l, h], p.n_sink, p.n_recent, p.chunk)
            sel, sgap = select_edges(e, r, s, p.budget, p.select)
            Ko, Vo, do, asg = merge_head(K[l, h], V[l, h], deg[l, h], e.a_pos, e.b_pos, sel)
            outs.append((Ko, Vo, do, asg))
            log.macs += e.macs
            if len(e.argmax_gap):
                log.min_argmax_gap = min(log.min_argmax_gap, float(e.argmax_gap.min()))
            log.min_select_gap = min(log.min_select_gap, sgap)
            log.edges.append(e)
            log.selected.append(sel)
    s_out = outs[0][0].shape[0]
    assert all(o[0].shape[0] == s_out for o in outs)  # the merge count depends on shapes only
    Kn = np.stack([o[0] for o in outs]).reshape(L, H, s_out, d)
    Vn = np.stack([o[1] for o in outs]).reshape(L, H, s_out, d)
    dn = np.stack([o[2] for o in outs]).reshape(L, H, s_out)
    an = np.stack([o[3] for o in outs]).reshape(L, H, s)
    if storage is not None:
        Kn, Vn = round_to_dtype(Kn, storage), round_to_dtype(Vn, storage)
    log.s_out = s_out
    return Kn, Vn, dn, an, log


def compress_prefill(K, V, deg, p: Params, storage: str | None = None):
    """Algorithm 1, pre-filling branch: N = [1]*n, then `while s > B: CentroidKV(...)`
    with Eq. 4's ratio for round j.  With budget 0 exactly n_rounds_max rounds run.
    Returns (K, V, deg, assign, logs); assign maps each original token to its final slot."""
    L, H, s, _ = K.shape
    if deg is None:
        deg = np.ones((L, H, s), dtype=np.int64)
    assign = np.broadcast_to(np.arange(s), (L, H, s)).copy()
    logs, j = [], 0
    while j < p.n_rounds_max and (p.budget == 0 or K.shape[2] > p.budget):
        r = ratio_for_round(p, j)
        K, V, deg, asg, log = csm_round(K, V, deg, p, r, storage)
        if log.s_out == log.s_in and p.budget > 0:
            raise RuntimeError("no progress: the schedule merges nothing but the budget is not met")
        assign = np.take_along_axis(asg, assign, axis=2)
        logs.append(log)
        j += 1
    return K, V, deg, assign, logs


def compress_append(K, V, deg, pending, k_new, v_new, p: Params, storage: str | None = None):
    """Algorithm 1, decoding branch, first line: K = [K, k], V = [V, v], N = [N, 1].
    Re-clustering uses the chunk-local trigger: whenever `chunk` generated tokens
    have accumulated at the tail, that window alone is clustered as a stand-alone
    sequence (no sinks, no recent tokens) with Eq. 4's schedule, until it is no longer
    than `budget` (budget 0: exactly n_rounds_max rounds).
    Returns (K, V, deg, pending)."""
    L, H, _, d = K.shape
    wp = Params(chunk=p.chunk, n_sink=0, n_recent=0, n_rounds_max=p.n_rounds_max, r_init=p.r_init,
                r_decay=p.r_decay, r_min=p.r_min, budget=p.budget, select=p.select)
    for t in range(k_new.shape[2]):
        K = np.concatenate([K, k_new[:, :, t:t + 1]], axis=2)
        V = np.concatenate([V, v_new[:, :, t:t + 1]], axis=2)
        deg = np.concatenate([deg, np.ones((L, H, 1), dtype=deg.dtype)], axis=2)
        pending += 1
        if pending == p.chunk:
            w0 = K.shape[2] - pending
            Kw, Vw, dw, _, _ = compress_prefill(K[:, :, w0:], V[:, :, w0:], deg[:, :, w0:], wp, storage)
            K = np.concatenate([K[:, :, :w0], Kw], axis=2)
            V = np.concatenate([V[:, :, :w0], Vw], axis=2)
            deg = np.concatenate([deg[:, :, :w0], dw], axis=2)
            pending = 0
    return K, V, deg, pending


def append_recluster(K, V, deg, k_new, v_new, p: Params, interval: int, storage: str | None = None):
    """Algorithm 1, decoding branch, as printed: for every generated token K = [K, k], V = [V, v],
    N = [N, 1], s = s + 1, and `if s >= B + g` one call of CentroidKV over the whole cache (sinks
    and recent tokens kept, the degrees carried along) with the compression ratio of round 0.
    With edges ranked per head the call merges min(floor(r * n_edges), s - B) edges, so the cache
    returns to the budget B whenever the ratio allows it (the paper is silent on how a single call
    lands on B; this is the reading taken for the pre-filling loop as well).
    Returns (K, V, deg, number of re-clusterings)."""
    L, H, _, d = K.shape
    if p.budget <= 0:
        raise ValueError("the fixed-budget trigger needs a budget B")
    calls = 0
    for t in range(k_new.shape[2]):
        K = np.concatenate([K, k_new[:, :, t:t + 1]], axis=2)
        V = np.concatenate([V, v_new[:, :, t:t + 1]], axis=2)
        deg = np.concatenate([deg, np.ones((L, H, 1), dtype=deg.dtype)], axis=2)
        if K.shape[2] >= p.budget + interval:
            K, V, deg, _, log = csm_round(K, V, deg, p, ratio_for_round(p, 0), storage)
            if log.s_out == log.s_in:
                raise RuntimeError("no progress: the round merges nothing although the cache exceeds its budget")
            calls += 1
    return K, V, deg, calls


# --------------------------------------------------------------------------- Eq. 1 and Eq. 3: attention

def app_attn(q, K, V, deg, scale):
    """Eq. 3 / Algorithm 1 decoding branch: softmax(q K^T * scale + log N) V for one
    sequence and one layer.  q: [H*G, d]; K, V: [H, s, d]; deg: [H, s] or None
    (None = all ones, which is Eq. 1).  Query head j reads KV head j // G."""
    HG, d = q.shape
    H = K.shape[0]
    G = HG // H
    out = np.empty((HG, d), dtype=np.float64)
    for j in range(HG):
        h = j // G
        z = (K[h] @ q[j]) * scale
        if deg is not None:
            z = z + np.log(deg[h].astype(np.float64))
        w = np.exp(z - z.max())
        out[j] = (w[:, None] * V[h]).sum(axis=0) / w.sum()
    return out


def attn(q, K, V, scale):
    """Eq. 1: exact softmax attention (Eq. 3 with every degree equal to one)."""
    return app_attn(q, K, V, None, scale)


# --------------------------------------------------------------------------- paged cache (block layout of serving engines)

def gather_pages(pages, block_table, length: int):
    """A paged cache stores logical token t of a sequence in page block_table[t // P] at offset t % P.
    pages: [n_pages, H, P, ...]; returns the sequence's first `length` tokens as [H, length, ...]."""
    P = pages.shape[2]
    t = np.arange(length)
    page = np.asarray(block_table)[t // P]
    return np.moveaxis(pages[page, :, t % P], 0, 1)


def app_attn_paged(q, k_pages, v_pages, deg_pages, block_table, length: int, scale):
    """Eq. 3 over a paged cache: by definition the attention over the gathered sequence."""
    deg = gather_pages(deg_pages, block_table, length) if deg_pages is not None else None
    return app_attn(q, gather_pages(k_pages, block_table, length), gather_pages(v_pages, block_table, length), deg, scale)

