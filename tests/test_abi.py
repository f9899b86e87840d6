"""The C-ABI library loads without a GPU, exports every symbol include/ckv.h declares, and its
host-side logic (round schedule, argument checks) agrees with the oracle.  No kernel is launched here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import ckv_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def b():
    from paper_2506_11418_b200 import binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ckv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ckv_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(b):
    names = declared_symbols()
    assert set(b.EXPORTS) <= set(names) and len(names) >= 7
    for n in names:
        assert hasattr(b.lib, n), f"libckv.so does not export {n}"


def test_status_strings(b):
    assert b.lib.ckv_status_string(0) == b"ok"
    assert len({b.lib.ckv_status_string(i) for i in range(8)}) == 8


def oracle_lengths(s, p: O.Params):
    """Lengths after each round of Algorithm 1's loop, from the oracle's own counting functions."""
    out = []
    j = 0
    while j < p.n_rounds_max and (p.budget == 0 or s > p.budget):
        r = O.ratio_for_round(p, j)
        _, _, chunks = O.chunk_bounds(s, p.n_sink, p.n_recent, p.chunk)
        edges = [len(O.alternating_partition(e - b_)[0]) if e - b_ >= 2 else 0 for b_, e in chunks]
        if p.select == O.SELECT_GLOBAL:
            M = O.merges_from_ratio(r, sum(edges))
            if p.budget > 0:
                M = min(M, s - p.budget)
        else:
            M = sum(O.merges_from_ratio(r, n) for n in edges)
        s -= M
        out.append(s)
        j += 1
    return out


@pytest.mark.parametrize("select", [0, 1])
@pytest.mark.parametrize("s,chunk,sink,recent,budget,rounds,r", [
    (32768, 64, 0, 0, 0, 1, (1.0, 0.0, 1.0)), (131072, 64, 0, 0, 0, 2, (1.0, 0.0, 1.0)),
    (131072, 64, 16, 64, 32768, 16, (0.8, 0.2, 0.2)), (6000, 256, 16, 64, 1500, 16, (0.8, 0.2, 0.2)),
    (517, 8, 3, 5, 0, 3, (0.34, 0.1, 0.05)), (81, 64, 16, 64, 0, 2, (1.0, 0.0, 1.0)), (1001, 6, 0, 1, 300, 30, (0.9, 0.3, 0.4))])
def test_plan_matches_oracle_lengths(b, select, s, chunk, sink, recent, budget, rounds, r):
    p = b.Params(chunk=chunk, n_sink=sink, n_recent=recent, n_rounds_max=rounds, r_init=r[0], r_decay=r[1], r_min=r[2],
                 select=select, budget=budget)
    r32 = p.as_float32()
    po = O.Params(chunk=chunk, n_sink=sink, n_recent=recent, n_rounds_max=rounds, r_init=r32[0], r_decay=r32[1], r_min=r32[2],
                  budget=budget, select=select)
    lens = oracle_lengths(s, po)
    out_len, n_rounds, cap = b.compress_plan(s, p)
    assert n_rounds == len(lens)
    assert out_len == (lens[-1] if lens else s)
    assert cap >= out_len and cap <= s


def test_plan_reports_no_progress_and_bad_arguments(b):
    with pytest.raises(b.CkvError) as e:
        b.compress_plan(1000, b.Params(chunk=64, n_sink=0, n_recent=0, r_init=0.0, r_decay=0.0, r_min=0.0, budget=10))
    assert e.value.status == 5
    for bad in (b.Params(chunk=63), b.Params(chunk=-2), b.Params(chunk=64, n_sink=-1), b.Params(chunk=64, r_init=1.5),
                b.Params(chunk=64, select=7)):
        with pytest.raises(b.CkvError) as e:
            b.compress_plan(1000, bad)
        assert e.value.status == 1
    with pytest.raises(b.CkvError) as e:
        b.compress_plan(1000, b.Params(chunk=512))
    assert e.value.status == 6


def test_round_cap_can_end_the_loop_above_the_budget(b):
    """Algorithm 1's loop also ends when n_rounds_max is used up: the status is ok and the length says what happened."""
    s = 131072
    kw = dict(chunk=64, n_sink=16, n_recent=64, r_init=0.8, r_decay=0.2, r_min=0.2, budget=s // 4)
    out_full, rounds_full, _ = b.compress_plan(s, b.Params(n_rounds_max=16, **kw))
    assert out_full == s // 4 and rounds_full == 6          # Eq. 4's defaults need six rounds for a 25 % budget
    out_cut, rounds_cut, _ = b.compress_plan(s, b.Params(n_rounds_max=3, **kw))
    assert rounds_cut == 3 and out_cut > s // 4
    lens = oracle_lengths(s, O.Params(n_rounds_max=3, **{k: (np.float32(v).item() if isinstance(v, float) else v) for k, v in kw.items()}))
    assert out_cut == lens[-1]


def test_plan_without_chunks_matches_the_oracle_lengths(b):
    """chunk = 0 (no chunking): one chunk spans the middle region; lengths after every round as the oracle counts them."""
    for s, kw in ((1000, dict(n_sink=0, n_recent=0, r_init=1.0, r_decay=0.0, r_min=1.0, n_rounds_max=2)),
                  (777, dict(n_sink=16, n_recent=64, r_init=0.8, r_decay=0.2, r_min=0.2, n_rounds_max=16, budget=200))):
        out_len, rounds, _ = b.compress_plan(s, b.Params(chunk=0, **kw))
        po = O.Params(chunk=0, **kw)
        lens = oracle_lengths(s, po)
        assert rounds == len(lens) and out_len == lens[-1]


def test_argument_checks_happen_before_any_launch(b):
    """Null or misaligned pointers are rejected on the host: these calls never reach the GPU."""
    p = b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0).c()
    src = b.CkvCache(None, None, None, None, 1, 1, 128, b.BF16, 256, 256, 0)
    dst = b.CkvCache(None, None, None, None, 1, 1, 128, b.BF16, 128, 0, 0)
    assert b.lib.ckv_compress_prefill(C.byref(src), C.byref(dst), C.byref(p), None, None, 0, None, None) == 1
    src = b.CkvCache(0x1008, 0x2000, None, None, 1, 1, 128, b.BF16, 256, 256, 0)
    dst = b.CkvCache(0x100000, 0x200000, 0x300000, None, 1, 1, 128, b.BF16, 128, 0, 0)
    assert b.lib.ckv_compress_prefill(C.byref(src), C.byref(dst), C.byref(p), None, None, 0, None, None) == 2
    src.D = 96
    dst.D = 96
    assert b.lib.ckv_compress_prefill(C.byref(src), C.byref(dst), C.byref(p), None, None, 0, None, None) == 6
    assert b.lib.ckv_decode_attn(None, 1, 1, 1, 128, b.BF16, None, None, 0.1, 10, None, 0, None) == 1
    assert b.lib.ckv_decode_attn(0x1000, 1, 1, 9, 128, b.BF16, 0x1000, 0x2000, 0.1, 10, None, 0, None) == 6
    assert b.lib.ckv_decode_attn(0x1000, 1, 1, 4, 128, b.BF16, 0x1000, 0x2000, 0.1, 10, None, 0, None) == 4
    assert b.lib.ckv_workspace_bytes(C.byref(src), C.byref(p)) == 0
    assert b.lib.ckv_decode_workspace_bytes(32, 8, 4, 128, 8448) >= 32 * 32 * 3 * 132 * 4


def test_append_recluster_argument_checks_need_no_gpu(b):
    """Everything ckv_compress_append_recluster can refuse is refused on the host before a launch (dummy pointers)."""
    L, H, D, cap = 1, 2, 128, 400

    def cache(base, length, cap=cap):
        return b.CkvCache(base, base + 0x1000000, base + 0x2000000, None, L, H, D, b.BF16, cap, length, 0)

    def call(p, live, spare, interval, t_new=4, ws_bytes=1 << 30):
        calls = C.c_int64(-1)
        return b.lib.ckv_compress_append_recluster(C.byref(live), C.byref(spare), 0x9000000, 0xA000000, t_new, C.byref(p.c()), interval,
                                                   0xB000000, ws_bytes, None, C.byref(calls))

    ok = b.Params(chunk=64, n_sink=4, n_recent=8, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0, budget=300)
    assert call(b.Params(chunk=64, budget=0), cache(0x10000000, 300), cache(0x20000000, 0), 16) == 1      # no budget
    assert call(ok, cache(0x10000000, 300), cache(0x20000000, 0), 0) == 1                                    # no interval
    assert call(ok, cache(0x10000000, 300), cache(0x20000000, 0, cap=310), 16) == 3                          # spare too small
    assert call(ok, cache(0x10000000, 300), cache(0x10000000, 0), 16) == 1                                   # same buffer
    nothing = b.Params(chunk=64, n_sink=4, n_recent=8, n_rounds_max=1, r_init=0.0, r_decay=0.0, r_min=0.0, budget=300)
    live = cache(0x10000000, 315)
    assert call(nothing, live, cache(0x20000000, 0), 16) == 5 and live.len == 315                            # merges nothing
    assert call(ok, cache(0x10000000, 315), cache(0x20000000, 0), 16, ws_bytes=64) == 4                       # workspace too small
