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

def compress_bytes(L, H, s, D, es, keep, with_deg=False):
    """One round, per token-vector: K and V read, the kept fraction of K and V written, degree + log-degree out (8 B per
    kept slot); the 4-byte degree read only when the source carries degrees (a cache straight from prefill does not)."""
    per_vec = 2 * D * es + keep * 2 * D * es + (4 if with_deg else 0) + keep * 8
    return L * H * s * per_vec


def schedule_bytes(L, H, s, out_len, D, es):
    """A whole schedule, whatever its number of rounds: what the method itself has to move is one read of the source
    and one write of the final cache (intermediate caches are an implementation's own traffic)."""
    return L * H * (s * 2 * D * es + out_len * (2 * D * es + 8))


def decode_bytes(rows, D, es):
    """Per cached token-vector: K and V rows plus the fp32 log-degree."""
    return rows * (2 * D * es + 4)


# --------------------------------------------------------------------------- DRAM traffic from the ncu capture

# dram__bytes_read.sum + dram__bytes_write.sum of round_fast_kernel per token-vector, from an ncu capture of a 4-layer
# cut of the workload (1 048 576 token-vectors per launch; traffic grows in proportion to the token-vectors processed,
# so it is scaled to the launch timed here).  Valid only for the kernel source it was taken from: the digest below is
# of ckv_compress_fast.cu at that time.
NCU_TRAFFIC = {"bytes_per_token_vector": (536910592 + 237573888) / 1048576,
               "source": "paper_2506_11418_b200/csrc/ckv_compress_fast.cu",
               "sha256": "cad95b42f458b35e7a4ced799296551e0fddd786303ec7a3eaa6e7557c3fab4f"}


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


def timed_burst(torch, dev, fn, iters, warm=3, rest_s=0.3):
    """Mean milliseconds of fn() over `iters` calls, after a rest and `warm` untimed calls, with the SM clock seen
    meanwhile.  The rest lets the board's power average fall back so that every row is a kernel timed alone: after a
    few hundred milliseconds of back-to-back launches the SM clock of these parts sinks from 1965 to 1.7-1.9 GHz, and
    every kernel that is not purely bandwidth-bound slows down with it (a row would then depend on the rows before it)."""
    torch.cuda.synchronize()
    time.sleep(rest_s)
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    sampler = ClockSampler(dev.index or 0, 0.002)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(iters):
        fn()
    t1.record()
    torch.cuda.synchronize()
    clk = sampler.stop()
    return t0.elapsed_time(t1) / iters, {"sm_mhz": clk.get("sm_mhz"), "reasons": clk.get("reasons")}


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


_WORKER_INPUT = None


def _oracle_worker_init():
    """Each worker process draws one (layer, head) slab of the workload and keeps it."""
    global _WORKER_INPUT
    import torch
    torch.set_num_threads(1)
    _WORKER_INPUT = oracle_inputs(1, seed=os.getpid() % 9973)


def _oracle_worker_pass(_):
    return oracle_pass(_WORKER_INPUT)


def _oracle_parity_pass(job):
    """One (layer, head) slab of the timed compression against the oracle: how many entries of the slot map differ, and
    how many of those sit where the oracle's two best candidates are closer than 1e-5 relative (near ties)."""
    import numpy as np
    from threadpoolctl import threadpool_limits

    from oracle import ckv_oracle as O

    K, V, assign_gpu, deg_gpu, chunk = job
    s = K.shape[0]
    p = O.Params(chunk=chunk, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)
    with threadpool_limits(limits=1):
        _, _, do, asg, log = O.csm_round(K[None, None].astype(np.float64), V[None, None].astype(np.float64),
                                         np.ones((1, 1, s), dtype=np.int64), p, 1.0, storage=None)
    e = log.edges[0]
    gap_at = np.full(s, np.inf)
    gap_at[e.a_pos] = e.argmax_gap
    differ = np.nonzero(asg[0, 0] != assign_gpu)[0]
    return {"edges": int(len(e.a_pos)), "differ": int(len(differ)), "near": int(np.sum(gap_at[differ] < 1e-5)),
            "deg_equal": bool(np.array_equal(do[0, 0], deg_gpu)) if len(differ) == 0 else None}


class OraclePool:
    """The oracle on the host's cores: one single-threaded NumPy process per core, each working through (layer, head)
    slabs (the method is independent per slab; the oracle itself is not changed or tuned for this).  Must be created
    before this process touches CUDA (the workers are forked)."""

    MAX_PROCS = 64

    def __init__(self):
        import multiprocessing as mp
        self.cores_available = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
        self.cores = max(1, min(self.cores_available, self.MAX_PROCS))
        self.pool = mp.get_context("fork").Pool(self.cores, initializer=_oracle_worker_init)
        cfg = __import__("paper_2506_11418_b200.synth", fromlist=["CONFIGS"]).CONFIGS[WORKLOAD]
        self.tokens_per_slab = cfg["s"] / (cfg["L"] * cfg["H"])
        self.slabs_total = cfg["L"] * cfg["H"]

    def run(self, n_slabs: int) -> float:
        """Wall seconds for n_slabs passes spread over the workers."""
        t0 = time.perf_counter()
        self.pool.map(_oracle_worker_pass, range(n_slabs), chunksize=1)
        return time.perf_counter() - t0

    def describe(self, n_slabs: int) -> str:
        return (f"{n_slabs} of {self.slabs_total} (layer, head) slabs of {WORKLOAD}: compress + append 64 + 1 decode step each, "
                f"{self.cores} single-threaded worker processes (host offers {self.cores_available} cores)")

    def close(self):
        self.pool.close()
        self.pool.join()


def cpu_baseline(pool: OraclePool, target_s: float = 12.0):
    """About target_s seconds of oracle work on every core: one slab per core first (which also sizes the sample)."""
    t1 = pool.run(pool.cores)
    rounds = max(1, min(30, int(round(target_s / max(t1, 1e-3)))))
    n = rounds * pool.cores
    dt = pool.run(n)
    return {"value": n * pool.tokens_per_slab / dt, "unit": UNIT, "cores": pool.cores, "cores_available": pool.cores_available,
            "kind": "oracle", "sample": pool.describe(n), "seconds": dt}


def workload_config(L=None):
    from paper_2506_11418_b200 import synth
    cfg = synth.CONFIGS[WORKLOAD]
    L = L or cfg["L"]
    return {"workload": WORKLOAD if L == cfg["L"] else f"{WORKLOAD} cut to {L} layers (not the benchmark workload)", "layers": L,
            "kv_heads": cfg["H"], "q_heads": cfg["H"] * cfg["G"], "head_dim": cfg["d"], "seq": cfg["s"], "chunk": cfg["chunk"],
            "retain": 0.5, "step": "compress_prefill + append 64 + decode all layers", "l2": "inputs (4 GiB) exceed L2",
            "clock_samples_cover": "warm-up (at least 0.3 s of it) and the timed region"}


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return  # under a multi-rank launch rank 0 alone times the oracle
    pool = OraclePool()
    n = pool.cores  # a step: one slab of the workload on every core
    for _ in range(min(args.warmup, 2)):
        pool.run(n)
    times = [pool.run(n) for _ in range(args.steps)]
    pool.close()
    total = sum(times)
    value = n * pool.tokens_per_slab * len(times) / total
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": pool.cores, "cores_available": pool.cores_available,
                             "kind": "oracle", "sample": "per step: " + pool.describe(n)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------- GPU leg

def run_gpu(args):
    import torch

    from paper_2506_11418_b200 import binding as b, parallel, synth

    rank, local, world = parallel.env_world()
    # the CPU baseline first: its worker processes are forked, which has to happen before this process touches CUDA
    cpu = None
    pool = None
    if rank == 0 and world == 1 and not args.skip_cpu:
        pool = OraclePool()
        cpu = cpu_baseline(pool)  # (the workers stay for the parity sample below; they never touch CUDA)
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
    if pool is not None:
        # two slabs of the timed compression, clustered on their own with the slot map, against the oracle on the host
        jobs = []
        for l, h in ((0, 0), (L // 2, 5 % H)):
            one = b.Cache(K[l:l + 1, h:h + 1].contiguous(), V[l:l + 1, h:h + 1].contiguous(), None, None, s)
            d1 = b.Cache.empty(1, 1, cap, D, K.dtype, dev)
            asg = torch.full((1, 1, s), -1, dtype=torch.int32, device=dev)
            b.compress_prefill(one, d1, p, ws, asg)
            jobs.append((one.k[0, 0].float().cpu().numpy(), one.v[0, 0].float().cpu().numpy(), asg[0, 0].cpu().numpy().astype("int64"),
                         d1.deg[0, 0, :out_len].cpu().numpy().astype("int64"), c))
        res = pool.pool.map(_oracle_parity_pass, jobs, chunksize=1)
        pool.close()
        cpu["parity_sample"] = {
            "what": "the timed compression on 2 (layer, head) slabs against the oracle (fp64): entries of the slot map that differ",
            "slabs": len(res), "edges": sum(r["edges"] for r in res), "slot_map_entries_that_differ": sum(r["differ"] for r in res),
            "of_which_near_ties_below_1e-5": sum(r["near"] for r in res),
            "degrees_equal_where_the_maps_agree": all(r["deg_equal"] for r in res if r["deg_equal"] is not None)}
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

    # the clock sampler runs from before the warm-up to after the timed region; the warm-up is stretched to at least
    # 0.3 s so that the record has samples under load however short the timed region is
    sampler = ClockSampler(local) if rank == 0 else None
    t_warm = time.perf_counter()
    for _ in range(max(args.warmup, 3)):
        step(False)
    torch.cuda.synchronize()
    untimed = max(args.warmup, 3)
    while time.perf_counter() - t_warm < 0.3:
        step(False)
        torch.cuda.synchronize()
        untimed += 1
    barrier()
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
    peak = peaks["hbm_gbs"]
    cbytes = compress_bytes(L, H, s, D, es, out_len / s, with_deg=False)   # the timed call passes no source degrees
    achieved = cbytes / (comp_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "round_fast_kernel (the one launch of ckv_compress_prefill at chunk 64, ratio 1)",
                "achieved": achieved, "peak": peak, "peak_kind": peak_kind + " copy bandwidth (MEASURED_PEAKS.json)" if peak_kind == "measured" else peak_kind,
                "unit": "GB/s", "frac": achieved / peak,
                "traffic": ncu_traffic(L * H * s), "bytes_per_launch": cbytes, "ms_per_launch": comp_ms,
                "frac_of_nominal_8tbs": achieved / 8000.0}
    dbytes = decode_bytes(H * final_len, D, es)
    dec_achieved = dbytes * L / (dec_ms * 1e-3) / 1e9
    extra = {"compress_ms": comp_ms, "compress_tokens_per_s": s / (comp_ms * 1e-3), "decode_ms_all_layers": dec_ms,
             "decode_gbs_batch1": dec_achieved, "untimed_steps_before_the_timed_region": untimed}
    targets = {}

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
    if rank == 0 and not args.skip_variants:
        extra["compress_variants"] = bench_compress_variants(b, synth, dev, K, V, peak, args.layers == 0)
        extra["recluster"] = bench_recluster(b, synth, dev, K, V)
        extra["no_chunk"] = bench_no_chunk(b, synth, dev, K, V, peaks, args.layers == 0)
        extra["paged_compress"] = bench_paged_compress(b, synth, dev, K, V, peak)
        targets["paged_compress_ratio1"] = {k: extra["paged_compress"]["chunk64 ratio1"][k] for k in ("ms", "frac_of_peak", "pages_freed")}
        targets["paged_compress_ratio1"]["sm_mhz"] = extra["paged_compress"]["chunk64 ratio1"]["clocks"]["sm_mhz"]
        cv = extra["compress_variants"]
        def pick(name):
            if name not in cv:
                return None
            row = {k: cv[name][k] for k in ("ms", "frac_of_peak", "gbs", "moved_gb", "frac_on_moved_bytes")}
            row["frac_of_nominal_8tbs"] = row["gbs"] / 8000.0
            row["sm_mhz"] = cv[name]["clocks"]["sm_mhz"]
            return row
        targets["chunk128_ratio1"] = pick("chunk128 ratio1")
        targets["chunk256_ratio1"] = pick("chunk256 ratio1")
        targets["chunk256_ratio0.8_ranked_per_head"] = pick("chunk256 ratio0.8 ranked per head")
        targets["chunk256_paper_schedule_to_25pct"] = pick("chunk256 paper schedule to 25%")
        targets["cfg3_128k_two_rounds_to_25pct"] = pick("llama8b_128k chunk64 two rounds ratio1 (to 25%)")
        targets["cfg3_128k_paper_schedule_to_25pct"] = pick("llama8b_128k chunk64 paper schedule to 25%")

    # end to end: inputs start in pinned host memory, the compressed cache and the decode output end there
    e2e = None
    if not args.skip_e2e:
        e2e = bench_e2e(b, torch, dev, K, V, kn, vn, q, p, dst, ws, wsd, views, final_len, out, s, world, max(2, min(args.steps, 5)))
        if world > 1:
            e2e["ms_per_step"] = parallel.max_over_ranks(e2e["ms_per_step"], dev)
            e2e["value"] = world * s / (e2e["ms_per_step"] * 1e-3)
    del K, V, src, dst, ws
    torch.cuda.empty_cache()
    if rank == 0 and not args.skip_decode_cfg4:
        extra["decode_cfg4"] = bench_decode_cfg4(b, synth, dev, peak)
        extra["decode_cfg4_paged"] = bench_decode_paged(b, synth, dev, peak)
        d4 = extra["decode_cfg4"]
        targets["cfg4_decode_batch32"] = {"compressed_us_per_layer_step": d4["compressed"]["us_per_layer_step"],
                                          "compressed_frac_of_peak": d4["compressed"]["frac_of_peak"],
                                          "compressed_frac_of_nominal_8tbs": d4["compressed"]["gbs"] / 8000.0,
                                          "uncompressed_us_per_layer_step": d4["uncompressed"]["us_per_layer_step"],
                                          "speedup_vs_uncompressed": d4["speedup"], "steps": d4["compressed"]["steps"],
                                          "paged_frac_of_peak": extra["decode_cfg4_paged"]["frac_of_peak"],
                                          "sm_mhz": d4["compressed"]["clocks"]["sm_mhz"]}
    if rank == 0 and not args.skip_serving and args.layers == 0:
        extra["serving_mix"] = bench_serving_mix(b, synth, dev, peak, steps=args.serving_steps)
        sm = extra["serving_mix"]
        targets["cfg5_serving_mix"] = {k: sm[k] for k in ("steps", "ms_per_step", "ms_attention_per_step", "attention_frac_of_peak",
                                                           "decode_tok_s", "attention_speedup", "prefill_compress_ms_total")}
    roofline["targets"] = targets   # the other workloads' numbers, each against the same measured peak

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
                "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
                "data": "synthetic", "config": workload_config(L),
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
                "cpu_baseline": cpu, "detail": extra, "roofline": roofline}
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
    the timed region).  `gbs` and `frac_of_peak` charge every schedule, whatever its number of rounds, what the method
    itself has to move: one read of the source and one write of the final cache.  `moved_gb` is what this
    implementation moves by construction (every round that is not fused with the next reads its input and writes its
    output; a round that ranks across chunks reads K once more), and `frac_on_moved_bytes` the rate on those."""
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
        ms, clk = timed_burst(torch, dev, lambda: b.compress_prefill(src, dst, p, ws), iters)
        lens, cur = [n], n
        for j in range(rounds):
            pj = P(chunk=p.chunk, n_sink=p.n_sink, n_recent=p.n_recent, n_rounds_max=j + 1, r_init=p.r_init, r_decay=p.r_decay,
                   r_min=p.r_min, select=p.select, budget=p.budget)
            cur = b.compress_plan(n, pj)[0]
            lens.append(cur)
        nbytes = schedule_bytes(L, H, n, out_len, D, 2)
        # what the launches move: per round input + output; two leading ratio-1 rounds at chunk 64 run as one pass; a
        # round ranked per head (neither 0 nor all of its edges merge) reads the keys twice
        moved, j = 0, 0
        while j < rounds:
            full = lambda a_, b_: a_ - b_ == (a_ - p.n_sink - p.n_recent) // p.chunk * (p.chunk // 2) + ((a_ - p.n_sink - p.n_recent) % p.chunk + 1) // 2
            fused = (p.chunk == 64 and j == 0 and rounds >= 2 and full(lens[0], lens[1]) and full(lens[1], lens[2]))
            if fused:
                moved += L * H * (lens[0] * 2 * D * 2 + lens[2] * (2 * D * 2 + 8))
                j += 2
                continue
            ranked = p.select == b.SELECT_GLOBAL and not full(lens[j], lens[j + 1]) and lens[j] != lens[j + 1]
            moved += L * H * (lens[j] * (2 * D * 2 + (4 if j else 0)) + lens[j + 1] * (2 * D * 2 + 8) + (lens[j] * D * 2 if ranked else 0))
            j += 1
        res[name] = {"seq": n, "out_len": out_len, "rounds": rounds, "ms": ms, "tokens_per_s": n / (ms * 1e-3),
                     "gbs": nbytes / (ms * 1e-3) / 1e9, "frac_of_peak": nbytes / (ms * 1e-3) / 1e9 / peak_gbs,
                     "moved_gb": moved / 1e9, "frac_on_moved_bytes": moved / (ms * 1e-3) / 1e9 / peak_gbs,
                     "clocks": clk, "status": b.workspace_status(ws)}
        del dst, ws

    for name, p in variants:
        time_one(name, K, V, p, 10)
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


def bench_serving_mix(b, synth, dev, peak_gbs, steps=1024):
    """Workload serving_mix at its stated size: batch 64, context lengths uniform on [4096, 65536], 32 layers x 8 KV
    heads, bf16.  Every sequence is prefill-compressed to 25 % (two rounds at ratio 1) one at a time from a scratch
    buffer that holds its uncompressed cache (the 64 uncompressed caches together would not fit) into its own slab.
    Then `steps` lock-step decoding steps: ckv_compress_append_batch writes one new token per sequence (every completed
    chunk of 64 appended tokens is clustered 64 -> 32 -> 16) and ckv_decode_attn runs for all 32 layers over the ragged
    batch with a fresh query.  The uncompressed comparison keeps the full contexts of the same batch on 8 layers (32
    would not fit) and is scaled to 32."""
    import torch
    cfg = synth.CONFIGS["serving_mix"]
    Bz, L, H, G, D, c = cfg["batch"], cfg["L"], cfg["H"], cfg["G"], cfg["d"], cfg["chunk"]
    ctx = synth.context_lengths(Bz, cfg["ctx"][0], cfg["ctx"][1], seed=cfg["seed"])
    p = b.Params(chunk=c, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0)
    scale = 1.0 / math.sqrt(D)
    n_q = 8   # distinct query tensors cycled through the steps
    qs = [synth.queries(Bz, H * G, D, seed=100 + i, dtype="bf16", device=dev) for i in range(n_q)]
    out = torch.empty_like(qs[0])
    g = torch.Generator(dev).manual_seed(23)

    def decode_loop(caches, layers, n_steps, compressed, ws):
        kn = torch.empty((layers, H, Bz, D), dtype=torch.bfloat16, device=dev).normal_(generator=g)
        vn = torch.empty((layers, H, Bz, D), dtype=torch.bfloat16, device=dev).normal_(generator=g)
        wsd = torch.empty(b.decode_workspace_bytes(Bz, H, G, D, max(x.cap for x in caches)), dtype=torch.uint8, device=dev)
        att_ev = []

        def one_step(i, record):
            if compressed:
                b.compress_append_batch(caches, kn, vn, p, ws)
            else:   # the uncompressed cache only grows
                for j, cache in enumerate(caches):
                    cache.k[:, :, cache.len] = kn[:, :, j]
                    cache.v[:, :, cache.len] = vn[:, :, j]
                    cache.len += 1
            max_len = max(x.len for x in caches)
            views = b.layer_views_all(caches, dev)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for l in range(layers):
                b.decode_attn(views[l], H, G, qs[i % n_q], out, scale, max_len, wsd)
            e1.record()
            if record:
                att_ev.append((e0, e1, sum(x.len for x in caches)))

        for i in range(3):
            one_step(i, False)
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for i in range(3, n_steps):
            one_step(i, True)
        t1.record()
        torch.cuda.synchronize()
        ms_step = t0.elapsed_time(t1) / (n_steps - 3)
        ms_att = statistics.mean(x.elapsed_time(y) for x, y, _ in att_ev)
        rows = statistics.mean(n for _, _, n in att_ev) * H
        return ms_step, ms_att, rows

    # ---- compressed: prefill-compress every sequence from the scratch buffer, then decode
    top = max(ctx)
    Ks = synth.ar1_keys(L, H, top, D, (0.7, 0.95), 0.5, seed=cfg["seed"], dtype="bf16", device=dev)   # every sequence reads a prefix
    Vs = synth.normal_values(L, H, top, D, seed=cfg["seed"], dtype="bf16", device=dev)
    growth = (steps // c + 1) * (c // 4) + c + 8
    caches, ws = [], None
    pre_ms, status = 0.0, 0
    for n in ctx:
        src = b.Cache(Ks, Vs, None, None, n)
        out_len, _, cap = b.compress_plan(n, p)
        dst = b.Cache.empty(L, H, max(cap, out_len + growth), D, torch.bfloat16, dev)
        need = max(b.workspace_bytes(src, p), b.workspace_bytes(dst, p))
        if ws is None or ws.numel() < need:
            ws = None
            ws = torch.empty(need, dtype=torch.uint8, device=dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        b.compress_prefill(src, dst, p, ws)
        e1.record()
        status |= b.workspace_status(ws)
        pre_ms += e0.elapsed_time(e1)
        caches.append(dst)
    del Ks, Vs
    torch.cuda.empty_cache()
    slots0 = sum(x.len for x in caches)
    ms_step, ms_att, rows = decode_loop(caches, L, steps, True, ws)
    status |= b.workspace_status(ws)
    nbytes = decode_bytes(rows, D, 2) * L
    res = {"batch": Bz, "layers": L, "steps": steps - 3, "context_tokens_total": sum(ctx), "cached_slots_after_prefill": slots0,
           "cached_slots_at_the_end": sum(x.len for x in caches), "prefill_compress_ms_total": pre_ms,
           "prefill_compress_tokens_per_s": sum(ctx) / (pre_ms * 1e-3),
           "ms_per_step": ms_step, "ms_attention_per_step": ms_att, "decode_tok_s": Bz / (ms_step * 1e-3),
           "attention_gbs": nbytes / (ms_att * 1e-3) / 1e9, "attention_frac_of_peak": nbytes / (ms_att * 1e-3) / 1e9 / peak_gbs,
           "status": status}
    del caches, ws
    torch.cuda.empty_cache()

    # ---- uncompressed comparison on 8 layers
    Lu, su = 8, 16
    caches = []
    for n in ctx:
        k = torch.empty((Lu, H, n + su + 1, D), dtype=torch.bfloat16, device=dev).normal_(generator=g)
        v = torch.empty((Lu, H, n + su + 1, D), dtype=torch.bfloat16, device=dev).normal_(generator=g)
        caches.append(b.Cache(k, v, None, None, n))
    _, ms_att_u, _ = decode_loop(caches, Lu, su, False, None)
    del caches
    torch.cuda.empty_cache()
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
        ms, clk = timed_burst(torch, dev, lambda: b.compress_prefill(src, dst, p, ws), iters, warm=1)
        tf = 2.0 * L * H * (n / 2) * (n / 2) * D / (ms * 1e-3) / 1e12
        return {"layers": L, "seq": n, "out_len": out_len, "ms": ms, "similarity_tflops": tf, "bound": "tensor",
                "frac_of_bf16_peak": tf / peaks["bf16_tflops"], "workspace_mib": ws.numel() / 2**20,
                "clocks": clk, "status": b.workspace_status(ws)}

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
    res = {"slots": slots, "page_tokens": P, "us_per_layer_step": us, "gbs": nbytes / (us * 1e-6) / 1e9,
           "frac_of_peak": nbytes / (us * 1e-6) / 1e9 / peak_gbs}
    # the same step with the new token appended inside the launch (slot `slots - 1` is rewritten every time)
    dp = torch.ones((pool, H, P), dtype=torch.int32, device=dev)
    views1 = b.paged_views(tables, [slots - 1] * Bz, dev)
    kn = torch.randn((Bz, H, D), device=dev, generator=g).to(torch.bfloat16)
    vn = torch.randn((Bz, H, D), device=dev, generator=g).to(torch.bfloat16)
    for _ in range(5):
        b.decode_append_attn_paged(views1, kp, vp, dp, lp, H, G, kn, vn, q, out, scale, slots, ws)
    torch.cuda.synchronize()
    t0.record()
    for _ in range(iters):
        b.decode_append_attn_paged(views1, kp, vp, dp, lp, H, G, kn, vn, q, out, scale, slots, ws)
    t1.record()
    torch.cuda.synchronize()
    us2 = 1e3 * t0.elapsed_time(t1) / iters
    res["append_and_attend_us_per_layer_step"] = us2
    res["append_and_attend_frac_of_peak"] = nbytes / (us2 * 1e-6) / 1e9 / peak_gbs
    return res


def bench_paged_compress(b, synth, dev, K, V, peak_gbs, page_tokens=64):
    """ckv_compress_paged on the benchmark workload held in 64-token pages scattered over per-layer pools: one round at
    ratio 1 (the timed step's compression, without leaving the pages) and the paper's schedule to 25 %, against the
    gather -> ckv_compress_prefill -> scatter route."""
    import torch
    L, H, s, D = K.shape
    P = page_tokens
    own = s // P
    res = {}
    paper = dict(n_sink=16, n_recent=64, n_rounds_max=16, r_init=0.8, r_decay=0.2, r_min=0.2)
    for name, p in (("chunk64 ratio1", b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)),
                    ("chunk64 paper schedule to 25%", b.Params(chunk=64, budget=s // 4, **paper))):
        out_len, rounds, n_scratch, in_scratch, kept = b.pages_plan(s, p, P)
        n_pages = own + n_scratch
        perm = torch.randperm(n_pages, generator=torch.Generator().manual_seed(5)).to(torch.int32).to(dev)
        table, scratch = perm[:own].contiguous(), perm[own:].contiguous()
        pools = []
        for l in range(L):
            kp = torch.empty((n_pages, H, P, D), dtype=torch.bfloat16, device=dev)
            vp = torch.empty_like(kp)
            dp = torch.ones((n_pages, H, P), dtype=torch.int32, device=dev)
            lp = torch.zeros((n_pages, H, P), dtype=torch.float32, device=dev)
            b.pages_scatter(table, s, K[l], V[l], None, kp, vp, dp, lp)
            pools.append((kp, vp, dp, lp))
        ws = torch.empty(b.paged_workspace_bytes(L, H, D, torch.bfloat16, s, p), dtype=torch.uint8, device=dev)
        # the call overwrites its source pages, which does not change what a repeated call costs
        ms, clk = timed_burst(torch, dev, lambda: b.compress_paged(pools, table, s, False, scratch, p, ws), 5, warm=2)
        nbytes = schedule_bytes(L, H, s, out_len, D, 2)
        res[name] = {"page_tokens": P, "seq": s, "out_len": out_len, "rounds": rounds, "ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9,
                     "frac_of_peak": nbytes / (ms * 1e-3) / 1e9 / peak_gbs, "pages_kept": kept, "pages_freed": own - kept,
                     "clocks": clk, "status": b.workspace_status(ws)}
        del pools, ws
        torch.cuda.empty_cache()
    return res


def bench_decode_cfg4(b, synth, dev, peak_gbs, steps=256):
    """Workload decode_b32 as stated: batch 32, 8 KV heads x 4 query heads, 8192 centroids whose degrees sum to 32768;
    256 decode steps, each with a fresh query ~ N(0, 1) and one appended degree-1 token per sequence (8192 -> 8448
    slots), one layer.  Compared with the same kernel on the uncompressed 32768-token cache (which grows the same way).
    The time is that of ckv_decode_attn alone (events around each call); the appends run between the calls."""
    import torch
    cfg = synth.CONFIGS["decode_b32"]
    Bz, H, G, D = cfg["batch"], cfg["H"], cfg["G"], cfg["d"]
    scale = 1.0 / math.sqrt(D)
    qs = synth.queries(steps * Bz, H * G, D, seed=3, dtype="bf16", device=dev).view(steps, Bz, H * G, D)
    gk = torch.Generator(dev).manual_seed(41)
    kn = torch.empty((steps, 1, H, Bz, D), dtype=torch.bfloat16, device=dev).normal_(generator=gk)
    vn = torch.empty((steps, 1, H, Bz, D), dtype=torch.bfloat16, device=dev).normal_(generator=gk)
    no_trigger = b.Params(chunk=64, n_sink=0, n_recent=0, n_rounds_max=0, r_init=1.0, r_decay=0.0, r_min=1.0)  # appended tokens stay as they are
    res = {}
    for name, slots, with_deg in (("compressed", cfg["slots"], True), ("uncompressed", cfg["s"], False)):
        cap = slots + steps
        caches = []
        for i in range(Bz):
            k = torch.randn((1, H, cap, D), device=dev, dtype=torch.float32).to(torch.bfloat16)
            v = torch.randn((1, H, cap, D), device=dev, dtype=torch.float32).to(torch.bfloat16)
            deg = torch.ones((1, H, cap), dtype=torch.int32)
            if with_deg:
                deg[:, :, :slots] = synth.random_degrees((1, H), slots, cfg["s"], seed=i)
            deg = deg.to(dev)
            caches.append(b.Cache(k, v, deg, torch.log(deg.float()) if with_deg else None, slots))
        out = torch.empty_like(qs[0])
        ws = torch.empty(b.decode_workspace_bytes(Bz, H, G, D, cap), dtype=torch.uint8, device=dev)
        wsa = torch.empty(b.workspace_bytes(caches[0], no_trigger), dtype=torch.uint8, device=dev)
        torch.cuda.synchronize()
        time.sleep(0.3)      # each arm timed alone (see timed_burst)
        for i in range(5):   # warm-up on the initial length
            b.decode_attn(b.layer_views(caches, 0, dev), H, G, qs[i], out, scale, slots, ws)
        # the view arrays of all steps are laid out on the device beforehand (only the lengths differ), so that the loop
        # is two calls per step and the GPU never waits for the host
        views_all = b.layer_views(caches, 0, dev).unsqueeze(0).repeat(steps, 1, 1)
        views_all[:, :, 3] += torch.arange(1, steps + 1, device=dev, dtype=torch.int64).view(steps, 1)
        torch.cuda.synchronize()
        sampler = ClockSampler(dev.index or 0, 0.002)
        evs, rows = [], 0
        for i in range(steps):
            b.compress_append_batch(caches, kn[i], vn[i], no_trigger, wsa)
            n = caches[0].len
            views = views_all[i]
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            b.decode_attn(views, H, G, qs[i], out, scale, n, ws)
            e1.record()
            evs.append((e0, e1))
            rows += Bz * H * n
        torch.cuda.synchronize()
        clk = sampler.stop()
        assert caches[0].len == slots + steps
        us = 1e3 * statistics.mean(x.elapsed_time(y) for x, y in evs)
        nbytes = (decode_bytes(rows, D, 2) if with_deg else rows * 2 * D * 2) / steps
        res[name] = {"slots": f"{slots} -> {slots + steps}", "steps": steps, "us_per_layer_step": us, "gbs": nbytes / (us * 1e-6) / 1e9,
                     "frac_of_peak": nbytes / (us * 1e-6) / 1e9 / peak_gbs, "decode_tok_s_per_layer": Bz / (us * 1e-6),
                     "clocks": {"sm_mhz": clk.get("sm_mhz"), "reasons": clk.get("reasons")}}
        del caches
        torch.cuda.empty_cache()
    res["speedup"] = res["uncompressed"]["us_per_layer_step"] / res["compressed"]["us_per_layer_step"]
    return res


def run_profile_case(name, layers=0):
    """A small stand-alone case for a profiler capture (a few launches of one kernel on a 4-layer cut of a workload,
    inputs larger than L2, a few GB on the device at most; --layers 32 for a one-pass launch list of the whole
    workload).  Prints nothing that is a benchmark number."""
    import torch

    from paper_2506_11418_b200 import binding as b, synth
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    cases = {
        # two ratio-1 rounds in one pass: 4 layers x 8 heads x 131072 tokens (2 GiB in)
        "two_rounds_128k": ("llama8b_128k", dict(chunk=64, n_sink=0, n_recent=0, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0)),
        # one ratio-1 round at chunk 64 / 128 / 256: 4 layers x 8 heads x 32768 tokens (512 MiB in)
        "one_round_32k_chunk64": ("llama8b_32k", dict(chunk=64, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)),
        "one_round_32k_chunk128": ("llama8b_32k", dict(chunk=128, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)),
        "one_round_32k_chunk256": ("llama8b_32k", dict(chunk=256, n_sink=0, n_recent=0, n_rounds_max=1, r_init=1.0, r_decay=0.0, r_min=1.0)),
        "ranked_round_32k_chunk256": ("llama8b_32k", dict(chunk=256, n_sink=16, n_recent=64, n_rounds_max=1, r_init=0.8, r_decay=0.0, r_min=0.8)),
        # the paper's schedule (ratios 0.8, 0.6, 0.4, 0.2, ... ranked per head, 16 sinks, 64 recent) to a 25 % budget
        "paper_schedule_32k_chunk64": ("llama8b_32k", dict(chunk=64, n_sink=16, n_recent=64, n_rounds_max=16, r_init=0.8, r_decay=0.2, r_min=0.2, budget=8192)),
        "paper_schedule_32k_chunk256": ("llama8b_32k", dict(chunk=256, n_sink=16, n_recent=64, n_rounds_max=16, r_init=0.8, r_decay=0.2, r_min=0.2, budget=8192)),
    }
    if name not in cases:
        raise SystemExit(f"unknown profile case {name!r}; known: {sorted(cases)}")
    workload, kw = cases[name]
    cfg = synth.CONFIGS[workload]
    L, H, s, D = layers or 4, cfg["H"], cfg["s"], cfg["d"]
    K = synth.ar1_keys(L, H, s, D, cfg["rho"], cfg["mean_std"], seed=cfg["seed"], dtype="bf16", device=dev)
    V = synth.normal_values(L, H, s, D, seed=cfg["seed"], dtype="bf16", device=dev)
    p = b.Params(**kw)
    src = b.Cache(K, V, None, None, s)
    out_len, rounds, cap = b.compress_plan(s, p)
    dst = b.Cache.empty(L, H, cap, D, K.dtype, dev)
    ws = torch.empty(b.workspace_bytes(src, p), dtype=torch.uint8, device=dev)
    for _ in range(3):
        b.compress_prefill(src, dst, p, ws)
    print(json.dumps({"profile_case": name, "layers": L, "seq": s, "out_len": out_len, "rounds": rounds, "status": b.workspace_status(ws)}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default: 50; 3 for --impl reference, whose step is seconds of CPU work)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ckv", choices=["ckv", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="use only this many layers of the workload (profiling a small case)")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-decode-cfg4", action="store_true")
    ap.add_argument("--skip-variants", action="store_true")
    ap.add_argument("--skip-serving", action="store_true")
    ap.add_argument("--serving-steps", type=int, default=1024, help="lock-step decode steps of the serving-mix workload (its stated size: 1024)")
    ap.add_argument("--profile-case", default=None, help="run one small named case three times and exit (for ncu captures)")
    args = ap.parse_args()
    if args.profile_case:
        run_profile_case(args.profile_case, args.layers)
        return
    if args.steps is None:
        args.steps = 3 if args.impl == "reference" else 50
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
