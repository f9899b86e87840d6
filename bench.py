"""Benchmark of the CentroidKV hot path on B200.

A step is one pass of the whole path over the Llama-3-8B-shaped prefill workload
(32 layers, 8 KV heads, head_dim 128, 32768 tokens, bf16, chunk 64, retain 50 %):
  1. ckv_compress_prefill  -- Chunked Soft Matching + centroid merge of the whole cache
  2. ckv_compress_append   -- one chunk of 64 generated tokens, which triggers the window clustering
  3. ckv_decode_attn x 32  -- one decode step over the compressed cache, all layers (32 query heads)
`value` is the number of prefill tokens compressed per second of whole-step time, summed over ranks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Under torchrun every rank runs the same per-GPU workload (weak scaling, no collective on the data
path); time is the maximum over ranks.  `--impl reference` times the CPU oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = "llama8b_32k"
METRIC = "compressed KV tokens/s"
UNIT = "tokens/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


# --------------------------------------------------------------------------- algorithmic bytes

def compress_bytes(L, H, s, D, es, keep):
    """Per token-vector: K and V read, the kept fraction of K and V written, degrees in (4 B) and
    degree + log-degree out (8 B per kept slot)."""
    per_vec = 2 * D * es + keep * 2 * D * es + 4 + keep * 8
    return L * H * s * per_vec


def decode_bytes(rows, D, es):
    """Per cached token-vector: K and V rows plus the fp32 log-degree."""
    return rows * (2 * D * es + 4)


# --------------------------------------------------------------------------- DRAM traffic from the ncu capture

# dram__bytes_read.sum + dram__bytes_write.sum of round_fast_kernel per token-vector, from the capture summarised in
# profiles/round_fast_kernel_llama8b_4layers.md (1 048 576 token-vectors per launch; traffic grows in proportion to
# the token-vectors processed, so it is scaled to the launch timed here).  Valid only for the kernel source it
# was taken from: the digest below is of ckv_compress_fast.cu at that time.
NCU_TRAFFIC = {"bytes_per_token_vector": (536905472 + 238534912) / 1048576,
               "source": "paper_2506_11418_b200/csrc/ckv_compress_fast.cu",
               "sha256": "cac8149dd5cca459a65579e8f4920999a6aab09152ec97f72602ed07318a0b1a"}


def ncu_traffic(token_vectors: int):
    import hashlib
    try:
        with open(os.path.join(ROOT, NCU_TRAFFIC["source"]), "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None
    if digest != NCU_TRAFFIC["sha256"]:
        return None  # the kernel has changed since the counters were taken
    return NCU_TRAFFIC["bytes_per_token_vector"] * token_vectors


# --------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML from a thread while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.005):
        import threading
        self.samples, self.reasons, self.smax, self.err = [], set(), None, None
        self._stop = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.smax = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # noqa: BLE001
            self.nv, self.err = None, f"nvml unavailable: {e}"
            return
        self.period = period_s
        self.thread = threading.Thread(target=self._run, daemon=True)
        self.thread.start()

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception as e:  # noqa: BLE001
                self.err = str(e)
                return
            self._stop.wait(self.period)

    def stop(self):
        if self.nv is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [self.err]}
        self._stop.set()
        self.thread.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.smax,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- CPU oracle leg

def oracle_inputs(n_heads: int, seed: int = 0):
    """`n_heads` (layer, head) slabs of the workload as fp64 arrays holding bf16-rounded values."""
    from paper_2506_11418_b200 import synth

    cfg = synth.CONFIGS[WORKLOAD]
    s, D, c, G = cfg["s"], cfg["d"], cfg["chunk"], cfg["G"]
    f64 = lambda t: t.float().double().numpy()
    return dict(
        K=f64(synth.ar1_keys(1, n_heads, s, D, cfg["rho"], cfg["mean_std"], seed=seed, dtype="bf16")),
        V=f64(synth.normal_values(1, n_heads, s, D, seed=seed, dtype="bf16")),
        kn=f64(synth.ar1_keys(1, n_heads, c, D, cfg["rho"], cfg["mean_std"], seed=seed + 1, dtype="bf16")),
        vn=f64(synth.normal_values(1, n_heads, c, D, seed=seed + 1, dtype="bf16")),
        q=f64(synth.queries(1, n_heads * G, D, seed=seed + 2, dtype="bf16"))[0],
        n_heads=n_heads, tokens=s * n_heads / (cfg["L"] * cfg["H"]), chunk=c, D=D,
        desc=f"{n_heads} of {cfg['L'] * cfg['H']} (layer, head) slabs of {WORKLOAD}: compress + append 64 + 1 decode step")


def oracle_pass(x) -> float:
    """The oracle, as it stands, over one sample: compress, append one chunk, one decode step.  Seconds."""
    from threadpoolctl import threadpool_limits

    from oracle import ckv_oracle as O

    p = O.Params(chunk=x["chunk"], n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)
    with threadpool_limits(limits=1):
        t0 = time.perf_counter()
        Ko, Vo, do, _, _ = O.compress_prefill(x["K"], x["V"], None, p, storage="bf16")
        Ko, Vo, do, _ = O.compress_append(Ko, Vo, do, 0, x["kn"], x["vn"], p, storage="bf16")
        O.app_attn(x["q"], Ko[0], Vo[0], do[0], 1.0 / math.sqrt(x["D"]))
        return time.perf_counter() - t0


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return  # under a multi-rank launch rank 0 alone times the oracle
    x = oracle_inputs(2)
    for _ in range(min(args.warmup, 1)):
        oracle_pass(x)
    times = [oracle_pass(x) for _ in range(args.steps)]
    total = sum(times)
    value = x["tokens"] * len(times) / total
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": x["desc"]},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": x["desc"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------- GPU leg

def run_gpu(args):
    import torch

    from paper_2506_11418_b200 import binding as b, parallel, synth

    rank, local, world = parallel.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    parallel.init("nccl", dev)

    cfg = synth.CONFIGS[WORKLOAD]
    L, H, G, s, D, c = cfg["L"], cfg["H"], cfg["G"], cfg["s"], cfg["d"], cfg["chunk"]
    if args.layers > 0:
        L = args.layers
    es = 2
    seed = parallel.rank_seed(cfg["seed"], rank)
    K = synth.ar1_keys(L, H, s, D, cfg["rho"], cfg["mean_std"], seed=seed, dtype="bf16", device=dev)
    V = synth.normal_values(L, H, s, D, seed=seed, dtype="bf16", device=dev)
    kn = synth.ar1_keys(L, H, c, D, cfg["rho"], cfg["mean_std"], seed=seed + 1, dtype="bf16", device=dev)
    vn = synth.normal_values(L, H, c, D, seed=seed + 1, dtype="bf16", device=dev)
    q = synth.queries(L, H * G, D, seed=seed + 2, dtype="bf16", device=dev)  # one [1, H*G, D] query per layer
    out = torch.empty_like(q)

    p = b.Params(chunk=c, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0, select=b.SELECT_GLOBAL)
    src = b.Cache(K, V, None, None, s)
    out_len, rounds, cap = b.compress_plan(s, p)
    dst = b.Cache.empty(L, H, cap + c, D, K.dtype, dev)
    ws = torch.empty(max(b.workspace_bytes(src, p), b.workspace_bytes(dst, p)), dtype=torch.uint8, device=dev)
    wsd = torch.empty(b.decode_workspace_bytes(1, H, G, D, cap + c), dtype=torch.uint8, device=dev)
    scale = 1.0 / math.sqrt(D)
    final_len = out_len + c // 2
    # the lengths a step produces are a function of shapes only, so the decode views can be built once
    dst.len = final_len
    views = [b.layer_views([dst], l, dev) for l in range(L)]
    # prefill round, append (copy, window round, copy), and one cluster launch per layer for batch-1 decode (the split
    # and combine kernels of larger batches are one kernel here)
    launches_per_step = 1 + 3 + L

    ev = lambda: torch.cuda.Event(enable_timing=True)
    comp_ev, dec_ev = [], []

    def step(record: bool):
        e0, e1, e2, e3 = (ev(), ev(), ev(), ev()) if record else (None,) * 4
        if record:
            e0.record()
        b.compress_prefill(src, dst, p, ws)
        if record:
            e1.record()
        b.compress_append(dst, kn, vn, p, ws)
        if record:
            e2.record()
        for l in range(L):
            b.decode_attn(views[l], H, G, q[l:l + 1], out[l:l + 1], scale, final_len, wsd)
        if record:
            e3.record()
            comp_ev.append((e0, e1))
            dec_ev.append((e2, e3))
        assert dst.len == final_len

    def barrier():
        parallel.barrier(dev)

    for _ in range(max(args.warmup, 3)):
        step(False)
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    t_start, t_end = ev(), ev()
    t_start.record()
    for _ in range(args.steps):
        step(True)
    t_end.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    elapsed_ms = parallel.max_over_ranks(t_start.elapsed_time(t_end), dev)
    ms_per_step = elapsed_ms / args.steps
    value = world * s * args.steps / (elapsed_ms * 1e-3)

    comp_ms = statistics.mean(a.elapsed_time(z) for a, z in comp_ev)
    dec_ms = statistics.mean(a.elapsed_time(z) for a, z in dec_ev)
    peaks, peak_kind = measured_peaks()
    cbytes = compress_bytes(L, H, s, D, es, out_len / s)
    achieved = cbytes / (comp_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "compress round kernel (one launch per ckv_compress_prefill)", "achieved": achieved,
                "peak": peaks["hbm_gbs"], "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                "traffic": ncu_traffic(L * H * s), "bytes_per_launch": cbytes, "ms_per_launch": comp_ms,
                "frac_of_nominal_8tbs": achieved / 8000.0}
    dbytes = decode_bytes(H * final_len, D, es)
    dec_achieved = dbytes * L / (dec_ms * 1e-3) / 1e9
    extra = {"compress_ms": comp_ms, "compress_tokens_per_s": s / (comp_ms * 1e-3), "decode_ms_all_layers": dec_ms,
             "decode_gbs_batch1": dec_achieved}

    if rank == 0:
        # the same step captured once into a CUDA graph and replayed: what the GPU needs when the host issues nothing
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step(False)
        graph.replay()
        torch.cuda.synchronize()
        g0, g1 = ev(), ev()
        g0.record()
        for _ in range(args.steps):
            graph.replay()
        g1.record()
        torch.cuda.synchronize()
        extra["step_from_cuda_graph_ms"] = g0.elapsed_time(g1) / args.steps
        del graph
    if rank == 0 and not args.skip_decode_cfg4:
        extra["decode_cfg4"] = bench_decode_cfg4(b, synth, dev, peaks["hbm_gbs"])
        extra["decode_cfg4_paged"] = bench_decode_paged(b, synth, dev, peaks["hbm_gbs"])
    if rank == 0 and not args.skip_serving and args.layers == 0:
        extra["serving_mix"] = bench_serving_mix(b, synth, dev, peaks["hbm_gbs"])
    if rank == 0 and not args.skip_variants:
        extra["compress_variants"] = bench_compress_variants(b, synth, dev, K, V, peaks["hbm_gbs"], args.layers == 0)
        extra["recluster"] = bench_recluster(b, synth, dev, K, V)
        extra["no_chunk"] = bench_no_chunk(b, synth, dev, K, V, peaks, args.layers == 0)

    # end to end: inputs start in pinned host memory, the compressed cache and the decode output end there
    e2e = None
    if not args.skip_e2e:
        e2e = bench_e2e(b, torch, dev, K, V, kn, vn, q, p, dst, ws, wsd, views, final_len, out, s, world, max(2, min(args.steps, 5)))
        if world > 1:
            e2e["ms_per_step"] = parallel.max_over_ranks(e2e["ms_per_step"], dev)
            e2e["value"] = world * s / (e2e["ms_per_step"] * 1e-3)

    cpu = None
    if rank == 0 and world == 1 and not args.skip_cpu:
        x = oracle_inputs(16)
        dt = oracle_pass(x)
        cpu = {"value": x["tokens"] / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": x["desc"], "seconds": dt}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
                "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
                "data": "synthetic",
                "config": {"workload": WORKLOAD if args.layers == 0 else f"{WORKLOAD} cut to {L} layers (not the benchmark workload)", "layers": L, "kv_heads": H, "q_heads": H * G, "head_dim": D, "seq": s,
                           "chunk": c, "retain": out_len / s, "step": "compress_prefill + append 64 + decode all layers",
                           "l2": "inputs (4 GiB) exceed L2"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps, "roofline": roofline,
                "cpu_baseline": cpu, "detail": extra}
        print(json.dumps(line))
    parallel.finish()


def bench_e2e(b, torch, dev, K, V, kn, vn, q, p, dst, ws, wsd, views, final_len, out, s, world, iters, group=4):
    """The same step through the C ABI with every input starting in pinned host memory and every result ending there.
    The layers go through in groups: while one group is clustered and attended on the compute stream, the next group's
    K, V, new tokens and queries arrive on a copy stream and the previous group's compressed cache, degrees and
    attention output leave on a third one (PCIe is full duplex), so a step costs about the larger of the two transfers."""
    L, H, _, D = K.shape
    G = q.shape[1] // H
    scale = 1.0 / math.sqrt(D)
    pin = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
    hK, hV, hkn, hvn, hq = pin(K), pin(V), pin(kn), pin(vn), pin(q)
    hKo = torch.empty((L, H, final_len, D), dtype=K.dtype, pin_memory=True)
    hVo = torch.empty((L, H, final_len, D), dtype=K.dtype, pin_memory=True)
    hdeg = torch.empty((L, H, final_len), dtype=torch.int32, pin_memory=True)
    hout = torch.empty(out.shape, dtype=out.dtype, pin_memory=True)
    h2d = sum(t.numel() * t.element_size() for t in (hK, hV, hkn, hvn, hq))
    d2h = sum(t.numel() * t.element_size() for t in (hKo, hVo, hdeg, hout))
    s_in, s_cmp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    groups = [(i, min(i + group, L)) for i in range(0, L, group)]
    srcs = [b.Cache(K[i:j], V[i:j], None, None, s) for i, j in groups]
    dsts = [b.Cache(dst.k[i:j], dst.v[i:j], dst.deg[i:j], dst.logdeg[i:j], 0) for i, j in groups]
    done_cmp = [None] * len(groups)   # events of the previous step: a buffer is not refilled while it is still read
    done_out = [None] * len(groups)
    cur = torch.cuda.current_stream(dev)

    def e2e_step():
        start = torch.cuda.Event()
        start.record(cur)
        for st in (s_in, s_cmp, s_out):
            st.wait_event(start)
        for gi, (i, j) in enumerate(groups):
            with torch.cuda.stream(s_in):
                if done_cmp[gi] is not None:
                    s_in.wait_event(done_cmp[gi])
                K[i:j].copy_(hK[i:j], non_blocking=True)
                V[i:j].copy_(hV[i:j], non_blocking=True)
                kn[i:j].copy_(hkn[i:j], non_blocking=True)
                vn[i:j].copy_(hvn[i:j], non_blocking=True)
                q[i:j].copy_(hq[i:j], non_blocking=True)
                ev_in = torch.cuda.Event()
                ev_in.record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(ev_in)
                if done_out[gi] is not None:
                    s_cmp.wait_event(done_out[gi])
                dsts[gi].len, dsts[gi].pending = 0, 0
                b.compress_prefill(srcs[gi], dsts[gi], p, ws)
                b.compress_append(dsts[gi], kn[i:j], vn[i:j], p, ws)
                assert dsts[gi].len == final_len
                for l in range(i, j):
                    b.decode_attn(views[l], H, G, q[l:l + 1], out[l:l + 1], scale, final_len, wsd)
                done_cmp[gi] = torch.cuda.Event()
                done_cmp[gi].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(done_cmp[gi])
                hKo[i:j].copy_(dst.k[i:j, :, :final_len], non_blocking=True)
                hVo[i:j].copy_(dst.v[i:j, :, :final_len], non_blocking=True)
                hdeg[i:j].copy_(dst.deg[i:j, :, :final_len], non_blocking=True)
                hout[i:j].copy_(out[i:j], non_blocking=True)
                done_out[gi] = torch.cuda.Event()
                done_out[gi].record(s_out)
        cur.wait_event(done_out[-1])
        cur.wait_event(done_cmp[-1])

    e2e_step()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(iters):
        e2e_step()
    t1.record()
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / iters
    # the results really are on the host: the last group's attention output and degrees
    assert torch.equal(hout[-1], out[-1].cpu()) and int(hdeg[-1].sum()) == (s + kn.shape[2]) * H
    return {"value": world * s / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": ms, "steps": iters, "layers_per_group": group}


def bench_compress_variants(b, synth, dev, K, V, peak_gbs, with_128k):
    """ckv_compress_prefill alone on the same keys and values with other chunk sizes, ratios and ranking scopes (outside
    the timed region).  `gbs` counts what the method has to move if every round read its input once and wrote its
    output once; a round that ranks across chunks reads K twice, which is not credited."""
    import torch
    L, H, s, D = K.shape
    P = b.Params
    paper = dict(n_sink=16, n_recent=64, n_rounds_max=16, r_init=0.8, r_decay=0.2, r_min=0.2)
    variants = [
        ("chunk64 ratio1 sinks16 recent64", P(chunk=64, n_sink=16, n_recent=64, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)),
        ("chunk64 ratio0.5 ranked per chunk", P(chunk=64, n_sink=0, n_recent=0, n_rounds_max=1, r_init=0.5, r_decay=0.0, r_min=0.5, select=b.SELECT_CHUNK)),
        ("chunk64 ratio0.8 ranked per head", P(chunk=64, n_sink=16, n_recent=64, n_rounds_max=1, r_init=0.8, r_decay=0.0, r_min=0.8)),
        ("chunk128 ratio1", P(chunk=128, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)),
        ("chunk256 ratio1", P(chunk=256, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)),
        ("chunk64 paper schedule to 25%", P(chunk=64, budget=s // 4, **paper)),
        ("chunk256 paper schedule to 25%", P(chunk=256, budget=s // 4, **paper)),
        ("chunk128 ratio0.8 ranked per head", P(chunk=128, n_sink=16, n_recent=64, n_rounds_max=1, r_init=0.8, r_decay=0.0, r_min=0.8)),
        ("chunk256 ratio0.8 ranked per head", P(chunk=256, n_sink=16, n_recent=64, n_rounds_max=1, r_init=0.8, r_decay=0.0, r_min=0.8)),
        ("chunk128 paper schedule to 25%", P(chunk=128, budget=s // 4, **paper)),
    ]
    res = {}

    def time_one(name, Kx, Vx, p, iters):
        n = Kx.shape[2]
        src = b.Cache(Kx, Vx, None, None, n)
        out_len, rounds, cap = b.compress_plan(n, p)
        dst = b.Cache.empty(L, H, cap, D, Kx.dtype, dev)
        ws = torch.empty(b.workspace_bytes(src, p), dtype=torch.uint8, device=dev)
        for _ in range(2):
            b.compress_prefill(src, dst, p, ws)
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(iters):
            b.compress_prefill(src, dst, p, ws)
        t1.record()
        torch.cuda.synchronize()
        ms = t0.elapsed_time(t1) / iters
        # every round reads its input once and writes its output once
        lens, cur = [n], n
        for j in range(rounds):
            pj = P(chunk=p.chunk, n_sink=p.n_sink, n_recent=p.n_recent, n_rounds_max=j + 1, r_init=p.r_init, r_decay=p.r_decay,
                   r_min=p.r_min, select=p.select, budget=p.budget)
            cur = b.compress_plan(n, pj)[0]
            lens.append(cur)
        nbytes = sum(L * H * (lens[j] * (2 * D * 2 + 4) + lens[j + 1] * (2 * D * 2 + 8)) for j in range(rounds))
        res[name] = {"seq": n, "out_len": out_len, "rounds": rounds, "ms": ms, "tokens_per_s": n / (ms * 1e-3),
                     "gbs": nbytes / (ms * 1e-3) / 1e9, "frac_of_peak": nbytes / (ms * 1e-3) / 1e9 / peak_gbs,
                     "status": b.workspace_status(ws)}
        del dst, ws

    for name, p in variants:
        time_one(name, K, V, p, 5)
    if with_128k:
        cfg = synth.CONFIGS["llama8b_128k"]
        K3 = synth.ar1_keys(L, H, cfg["s"], D, cfg["rho"], cfg["mean_std"], seed=cfg["seed"], dtype="bf16", device=dev)
        V3 = synth.normal_values(L, H, cfg["s"], D, seed=cfg["seed"], dtype="bf16", device=dev)
        time_one("llama8b_128k chunk64 two rounds ratio1 (to 25%)", K3, V3,
                 P(chunk=64, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0), 3)
        time_one("llama8b_128k chunk64 paper schedule to 25%", K3, V3, P(chunk=64, budget=cfg["s"] // 4, **paper), 3)
        del K3, V3
    torch.cuda.empty_cache()
    return res


def bench_serving_mix(b, synth, dev, peak_gbs, steps=128):
    """Workload serving_mix: batch 64, context lengths uniform on [4096, 65536], 32 layers x 8 KV heads, caches already
    compressed to 25 % (their content does not matter for timing: random values, degrees 4).  Lock-step decoding: every
    step appends one token to every sequence (ckv_compress_append, which clusters each completed chunk of 64 appended
    tokens 64 -> 32 -> 16) and runs ckv_decode_attn for all 32 layers over the ragged batch.  The uncompressed comparison
    keeps the full contexts of the same batch on 8 layers (32 would not fit) and is scaled to 32."""
    import torch
    cfg = synth.CONFIGS["serving_mix"]
    Bz, L, H, G, D, c = cfg["batch"], cfg["L"], cfg["H"], cfg["G"], cfg["d"], cfg["chunk"]
    ctx = synth.context_lengths(Bz, cfg["ctx"][0], cfg["ctx"][1], seed=cfg["seed"])
    p = b.Params(chunk=c, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0)
    scale = 1.0 / math.sqrt(D)

    def run(layers, lens, compressed, n_steps):
        g = torch.Generator(dev).manual_seed(23)
        caches = []
        for n in lens:
            cap = n + n_steps + c
            k = torch.empty((layers, H, cap, D), dtype=torch.bfloat16, device=dev).normal_(generator=g)
            v = torch.empty((layers, H, cap, D), dtype=torch.bfloat16, device=dev).normal_(generator=g)
            deg = torch.full((layers, H, cap), 4 if compressed else 1, dtype=torch.int32, device=dev)
            caches.append(b.Cache(k, v, deg, torch.log(deg.float()) if compressed else None, n))
        ws = torch.empty(b.workspace_bytes(caches[0], p), dtype=torch.uint8, device=dev)
        wsd = torch.empty(b.decode_workspace_bytes(Bz, H, G, D, max(lens) + n_steps), dtype=torch.uint8, device=dev)
        kn = torch.empty((layers, H, Bz, D), dtype=torch.bfloat16, device=dev).normal_(generator=g)
        vn = torch.empty((layers, H, Bz, D), dtype=torch.bfloat16, device=dev).normal_(generator=g)
        new = [(kn[:, :, i:i + 1].contiguous(), vn[:, :, i:i + 1].contiguous()) for i in range(Bz)]
        q = synth.queries(Bz, H * G, D, seed=3, dtype="bf16", device=dev)
        out = torch.empty_like(q)
        att_ev = []

        def one_step(record):
            for i, cache in enumerate(caches):
                if compressed:
                    b.compress_append(cache, new[i][0], new[i][1], p, ws)
                else:   # the uncompressed cache only grows: same copy, no trigger
                    cache.k[:, :, cache.len] = new[i][0][:, :, 0]
                    cache.v[:, :, cache.len] = new[i][1][:, :, 0]
                    cache.len += 1
            max_len = max(x.len for x in caches)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for l in range(layers):
                b.decode_attn(b.layer_views(caches, l, dev), H, G, q, out, scale, max_len, wsd)
            e1.record()
            if record:
                att_ev.append((e0, e1))

        for _ in range(3):
            one_step(False)
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(n_steps - 3):
            one_step(True)
        t1.record()
        torch.cuda.synchronize()
        ms_step = t0.elapsed_time(t1) / (n_steps - 3)
        ms_att = statistics.mean(x.elapsed_time(y) for x, y in att_ev)
        rows = sum(x.len for x in caches) * H
        del caches
        torch.cuda.empty_cache()
        return ms_step, ms_att, rows

    comp_lens = [n // 4 for n in ctx]
    ms_step, ms_att, rows = run(L, comp_lens, True, steps)
    nbytes = decode_bytes(rows, D, 2) * L
    res = {"batch": Bz, "layers": L, "steps": steps - 3, "context_tokens_total": sum(ctx), "cached_slots_total": rows // H,
           "ms_per_step": ms_step, "ms_attention_per_step": ms_att, "decode_tok_s": Bz / (ms_step * 1e-3),
           "attention_gbs": nbytes / (ms_att * 1e-3) / 1e9, "attention_frac_of_peak": nbytes / (ms_att * 1e-3) / 1e9 / peak_gbs}
    Lu = 8
    ms_step_u, ms_att_u, _ = run(Lu, ctx, False, 16)
    res["uncompressed"] = {"layers_run": Lu, "ms_attention_per_step_32_layers": ms_att_u * L / Lu,
                           "decode_tok_s_attention_only": Bz / (ms_att_u * L / Lu * 1e-3)}
    res["attention_speedup"] = res["uncompressed"]["ms_attention_per_step_32_layers"] / ms_att
    return res


def bench_no_chunk(b, synth, dev, K, V, peaks, with_128k):
    """chunk = 0 (plain Bipartite Soft Matching, the paper's "w/o chunk" ablation): every A token against every B token
    of its head, n^2 d / 4 multiply-adds per head -- the one compute-bound variant.  One round at ratio 1 over (i) the
    first 16384 tokens of 4 layers x 8 KV heads and (ii) one layer of the 131072-token workload, the length at which
    the paper's variant runs out of memory (the similarities are never stored here).  The tensor-core rate divides the
    flops of the similarity contraction by the time of the whole round (norms, matching, ranking, merge)."""
    import torch

    def time_one(Ks, Vs, iters):
        L, H, n, D = Ks.shape
        p = b.Params(chunk=0, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)
        src = b.Cache(Ks, Vs, None, None, n)
        out_len, _, cap = b.compress_plan(n, p)
        dst = b.Cache.empty(L, H, cap, D, Ks.dtype, dev)
        ws = torch.empty(b.workspace_bytes(src, p), dtype=torch.uint8, device=dev)
        b.compress_prefill(src, dst, p, ws)
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(iters):
            b.compress_prefill(src, dst, p, ws)
        t1.record()
        torch.cuda.synchronize()
        ms = t0.elapsed_time(t1) / iters
        tf = 2.0 * L * H * (n / 2) * (n / 2) * D / (ms * 1e-3) / 1e12
        return {"layers": L, "seq": n, "out_len": out_len, "ms": ms, "similarity_tflops": tf, "bound": "tensor",
                "frac_of_bf16_peak": tf / peaks["bf16_tflops"], "workspace_mib": ws.numel() / 2**20,
                "status": b.workspace_status(ws)}

    L, n = min(4, K.shape[0]), 16384
    res = {"16k_4_layers": time_one(K[:L, :, :n].contiguous(), V[:L, :, :n].contiguous(), 3)}
    if with_128k:
        cfg = synth.CONFIGS["llama8b_128k"]
        H, D = K.shape[1], K.shape[3]
        K3 = synth.ar1_keys(1, H, cfg["s"], D, cfg["rho"], cfg["mean_std"], seed=cfg["seed"], dtype="bf16", device=dev)
        V3 = synth.normal_values(1, H, cfg["s"], D, seed=cfg["seed"], dtype="bf16", device=dev)
        res["128k_1_layer"] = time_one(K3, V3, 2)
        del K3, V3
    torch.cuda.empty_cache()
    return res


def bench_recluster(b, synth, dev, K, V):
    """Fixed-budget decoding branch (ckv_compress_append_recluster): a cache of B = 8192 slots per head with degrees
    above one, g = 256 appended tokens, then the re-clustering round over the whole cache back to B (paper defaults:
    16 sinks, 64 recent tokens, ratio 0.8, ranked per head)."""
    import torch
    L, H, _, D = K.shape
    B, g = 8192, 256
    p = b.Params(chunk=64, n_sink=16, n_recent=64, n_rounds_max=1, r_init=0.8, r_decay=0.2, r_min=0.2, budget=B)
    live, spare = (b.Cache.empty(L, H, B + g, D, K.dtype, dev) for _ in range(2))
    for c in (live, spare):
        c.k.copy_(K[:, :, :B + g])
        c.v.copy_(V[:, :, :B + g])
        c.deg.fill_(4)
        c.logdeg.fill_(math.log(4.0))
    live.len = B
    shape = b.Cache.empty(1, 1, 1, D, K.dtype, dev)
    shape.k = live.k
    shape.v = live.v
    shape.len = B + g
    ws = torch.empty(b.workspace_bytes(shape, p), dtype=torch.uint8, device=dev)
    kn, vn = K[:, :, B:B + g].contiguous(), V[:, :, B:B + g].contiguous()
    times = []
    for it in range(7):
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        calls = b.compress_append_recluster(live, spare, kn, vn, p, g, ws)
        t1.record()
        torch.cuda.synchronize()
        assert calls == 1 and live.len == B
        if it >= 2:
            times.append(t0.elapsed_time(t1))
    ms = statistics.mean(times)
    return {"budget": B, "interval": g, "ms_per_trigger_all_layers": ms, "us_per_decode_step_amortised": 1e3 * ms / g,
            "status": b.workspace_status(ws)}


def bench_decode_paged(b, synth, dev, peak_gbs):
    """The decode_b32 shape (batch 32, 8192 centroids) in a paged cache: 64-token pages scattered over one pool."""
    import torch
    cfg = synth.CONFIGS["decode_b32"]
    Bz, H, G, D, slots, P = cfg["batch"], cfg["H"], cfg["G"], cfg["d"], cfg["slots"], 64
    per_seq = slots // P
    pool = Bz * per_seq
    g = torch.Generator(dev).manual_seed(17)
    kp = torch.randn((pool, H, P, D), device=dev, generator=g).to(torch.bfloat16)
    vp = torch.randn((pool, H, P, D), device=dev, generator=g).to(torch.bfloat16)
    lp = torch.rand((pool, H, P), device=dev, generator=g) * 2.0
    perm = torch.randperm(pool, generator=torch.Generator().manual_seed(5)).to(torch.int32).to(dev)
    tables = [perm[i * per_seq:(i + 1) * per_seq].contiguous() for i in range(Bz)]
    views = b.paged_views(tables, [slots] * Bz, dev)
    q = synth.queries(Bz, H * G, D, seed=3, dtype="bf16", device=dev)
    out = torch.empty_like(q)
    ws = torch.empty(b.decode_workspace_bytes(Bz, H, G, D, slots), dtype=torch.uint8, device=dev)
    scale = 1.0 / math.sqrt(D)
    for _ in range(5):
        b.decode_attn_paged(views, kp, vp, lp, H, G, q, out, scale, slots, ws)
    torch.cuda.synchronize()
    iters = 50
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(iters):
        b.decode_attn_paged(views, kp, vp, lp, H, G, q, out, scale, slots, ws)
    t1.record()
    torch.cuda.synchronize()
    us = 1e3 * t0.elapsed_time(t1) / iters
    nbytes = decode_bytes(Bz * H * slots, D, 2)
    return {"slots": slots, "page_tokens": P, "us_per_layer_step": us, "gbs": nbytes / (us * 1e-6) / 1e9,
            "frac_of_peak": nbytes / (us * 1e-6) / 1e9 / peak_gbs}


def bench_decode_cfg4(b, synth, dev, peak_gbs):
    """Decode attention on the batch-32 shape: 8192 centroids (+256 appended) vs the uncompressed 32768-token cache."""
    import torch
    cfg = synth.CONFIGS["decode_b32"]
    Bz, H, G, D = cfg["batch"], cfg["H"], cfg["G"], cfg["d"]
    res = {}
    for name, slots, with_deg in (("compressed", cfg["slots"], True), ("uncompressed", cfg["s"], False)):
        cap = slots + 256
        caches = []
        for i in range(Bz):
            k = torch.randn((1, H, cap, D), device=dev, dtype=torch.float32).to(torch.bfloat16)
            v = torch.randn((1, H, cap, D), device=dev, dtype=torch.float32).to(torch.bfloat16)
            deg = logdeg = None
            if with_deg:
                deg = torch.ones((1, H, cap), dtype=torch.int32)
                deg[:, :, :slots] = synth.random_degrees((1, H), slots, cfg["s"], seed=i)
                deg = deg.to(dev)
                logdeg = torch.log(deg.float())
            caches.append(b.Cache(k, v, deg, logdeg, slots))
        q = synth.queries(Bz, H * G, D, seed=3, dtype="bf16", device=dev)
        out = torch.empty_like(q)
        ws = torch.empty(b.decode_workspace_bytes(Bz, H, G, D, cap), dtype=torch.uint8, device=dev)
        views = b.layer_views(caches, 0, dev)
        scale = 1.0 / math.sqrt(D)
        for _ in range(5):
            b.decode_attn(views, H, G, q, out, scale, slots, ws)
        torch.cuda.synchronize()
        iters = 50
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(iters):
            b.decode_attn(views, H, G, q, out, scale, slots, ws)
        t1.record()
        torch.cuda.synchronize()
        us = 1e3 * t0.elapsed_time(t1) / iters
        nbytes = decode_bytes(Bz * H * slots, D, 2) if with_deg else Bz * H * slots * 2 * D * 2
        res[name] = {"slots": slots, "us_per_layer_step": us, "gbs": nbytes / (us * 1e-6) / 1e9,
                     "frac_of_peak": nbytes / (us * 1e-6) / 1e9 / peak_gbs, "decode_tok_s_per_layer": Bz / (us * 1e-6)}
        del caches
    res["speedup"] = res["uncompressed"]["us_per_layer_step"] / res["compressed"]["us_per_layer_step"]
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default: 200; 3 for --impl reference, whose step is seconds of CPU work)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ckv", choices=["ckv", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="use only this many layers of the workload (profiling a small case)")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-decode-cfg4", action="store_true")
    ap.add_argument("--skip-variants", action="store_true")
    ap.add_argument("--skip-serving", action="store_true")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 3 if args.impl == "reference" else 200
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
