"""Parity of ckv_compress_append_recluster (Algorithm 1's decoding branch as printed: append, and one clustering round
over the whole cache whenever it reaches budget + interval tokens) against the oracle's replay of the same steps."""
import numpy as np
import pytest
import torch

from oracle import ckv_oracle as O
from paper_2506_11418_b200 import synth
import parity_util as PU

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("dtype,chunk,select", [("bf16", 64, 0), ("f32", 64, 0), ("bf16", 256, 0), ("bf16", 64, 1), ("bf16", 8, 0), ("bf16", 0, 0)])
def test_fixed_budget_trigger(dtype, chunk, select):
    from paper_2506_11418_b200 import binding as b
    L, H, D, s0, g = 2, 2, 128, 700, 48
    B = s0
    K = synth.ar1_keys(L, H, s0, D, (0.7, 0.95), 0.5, seed=61, dtype=dtype, device=DEV)
    V = synth.normal_values(L, H, s0, D, seed=61, dtype=dtype, device=DEV)
    p = b.Params(chunk=chunk, n_sink=16, n_recent=64, n_rounds_max=1, r_init=0.8, r_decay=0.2, r_min=0.2, select=select, budget=B)
    cap = B + g + 8
    live = b.Cache.empty(L, H, cap, D, K.dtype, DEV)
    spare = b.Cache.empty(L, H, cap, D, K.dtype, DEV)
    live.k[:, :, :s0], live.v[:, :, :s0] = K, V
    live.deg[:, :, :s0] = 1
    live.len = s0
    shape = b.Cache.empty(L, H, cap, D, K.dtype, DEV)
    shape.len = B + g
    ws = torch.empty(b.workspace_bytes(shape, p), dtype=torch.uint8, device=DEV)
    Ko, Vo, do = PU.to_np64(K), PU.to_np64(V), np.ones((L, H, s0), dtype=np.int64)
    po = PU.oracle_params(p)
    total, calls_total = s0, 0
    for step, t_new in enumerate([1, 40, 7, 1, 100, 47, 1, 200]):
        kn = synth.ar1_keys(L, H, t_new, D, (0.7, 0.95), 0.5, seed=300 + step, dtype=dtype, device=DEV)
        vn = synth.normal_values(L, H, t_new, D, seed=300 + step, dtype=dtype, device=DEV)
        calls = b.compress_append_recluster(live, spare, kn, vn, p, g, ws)
        assert b.workspace_status(ws) == 0
        Ko, Vo, do, calls_o = O.append_recluster(Ko, Vo, do, PU.to_np64(kn), PU.to_np64(vn), po, g, storage=dtype)
        total += t_new
        calls_total += calls
        assert calls == calls_o and live.len == Ko.shape[2] and live.len < B + g
        gpu = PU.gpu_cache_to_np(live)
        np.testing.assert_array_equal(gpu["deg"].sum(axis=2), np.full((L, H), total))
        np.testing.assert_array_equal(gpu["deg"], do)
        np.testing.assert_allclose(gpu["logdeg"], np.log(do.astype(np.float64)), rtol=1e-6, atol=1e-7)
        for l in range(L):
            for h in range(H):
                if dtype == "bf16":   # one ulp per storage rounding the row has been through
                    n_r = max(calls_total, 1)
                    assert np.all(np.abs(gpu["K"][l, h] - Ko[l, h]) <= n_r * PU.bf16_ulp(Ko[l, h]) * 1.0001)
                    assert np.all(np.abs(gpu["V"][l, h] - Vo[l, h]) <= n_r * PU.bf16_ulp(Vo[l, h]) * 1.0001 + 1e-30)
                else:
                    PU.compare_values(gpu["K"][l, h], Ko[l, h], dtype, "K")
                    PU.compare_values(gpu["V"][l, h], Vo[l, h], dtype, "V")
    assert calls_total >= (4 if select == 0 else 2)   # ranking per chunk does not trim onto the budget: fewer, larger rounds
    # sinks are never merged: still the first rows of the original cache
    assert torch.equal(live.k[:, :, :16], K[:, :, :16])
