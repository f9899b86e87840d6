"""The N > 1 path on CPU: two gloo ranks.  The path shards without any collective -- every (layer, head)
slab is independent -- so the ranks own disjoint slabs; what is exchanged is the barrier and the
maximum of the per-rank times.  The slabs are clustered here by the oracle (no GPU in this test):
the point is the host-side sharding, seeding and reduction logic that bench.py uses at N > 1."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import torch.distributed as dist

    from oracle import ckv_oracle as O
    from paper_2506_11418_b200 import parallel, synth

    r, w = parallel.init("gloo")
    assert (r, w) == (rank, world) and dist.is_initialized()
    L, H, s, d, c = 2, 3, 256, 128, 64
    K = synth.ar1_keys(L, H, s, d, (0.7, 0.95), 0.5, seed=5, dtype="bf16").float().double().numpy().reshape(L * H, s, d)
    V = synth.normal_values(L, H, s, d, seed=5, dtype="bf16").float().double().numpy().reshape(L * H, s, d)
    lo, hi = parallel.partition(L * H, rank, world)
    p = O.Params(chunk=c, n_sink=4, n_recent=8, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0)
    Ko, Vo, do, _, _ = O.compress_prefill(K[None, lo:hi], V[None, lo:hi], None, p, storage="bf16")
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), K=Ko[0], V=Vo[0], deg=do[0], lo=lo, hi=hi)
    parallel.barrier()
    # the job's time is the slowest rank's; throughput adds up
    t = parallel.max_over_ranks(10.0 + rank)
    n = parallel.sum_over_ranks(hi - lo)
    assert t == 10.0 + (world - 1) and n == L * H
    assert parallel.rank_seed(3, rank) != parallel.rank_seed(3, (rank + 1) % world)
    parallel.finish()


def test_two_ranks_own_disjoint_slabs_and_agree_with_one_rank(tmp_path):
    from oracle import ckv_oracle as O
    from paper_2506_11418_b200 import synth

    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    L, H, s, d, c = 2, 3, 256, 128, 64
    K = synth.ar1_keys(L, H, s, d, (0.7, 0.95), 0.5, seed=5, dtype="bf16").float().double().numpy()
    V = synth.normal_values(L, H, s, d, seed=5, dtype="bf16").float().double().numpy()
    p = O.Params(chunk=c, n_sink=4, n_recent=8, n_rounds_max=2, r_init=1.0, r_decay=0.0, r_min=1.0)
    Ko, Vo, do, _, _ = O.compress_prefill(K, V, None, p, storage="bf16")
    Ko, Vo, do = Ko.reshape(L * H, -1, d), Vo.reshape(L * H, -1, d), do.reshape(L * H, -1)
    covered = []
    for r in range(world):
        z = np.load(os.path.join(tmp_path, f"rank{r}.npz"))
        lo, hi = int(z["lo"]), int(z["hi"])
        covered += list(range(lo, hi))
        np.testing.assert_array_equal(z["K"], Ko[lo:hi])
        np.testing.assert_array_equal(z["V"], Vo[lo:hi])
        np.testing.assert_array_equal(z["deg"], do[lo:hi])
    assert covered == list(range(L * H))


@pytest.mark.parametrize("n,world", [(256, 1), (256, 8), (7, 2), (3, 4), (0, 2), (64, 3)])
def test_partition_is_a_balanced_cover(n, world):
    from paper_2506_11418_b200 import parallel
    parts = [parallel.partition(n, r, world) for r in range(world)]
    assert parts[0][0] == 0 and parts[-1][1] == n
    assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
    sizes = [e - b for b, e in parts]
    assert max(sizes) - min(sizes) <= 1


def test_single_process_needs_no_group():
    from paper_2506_11418_b200 import parallel
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert parallel.env_world() == (0, 0, 1)
    assert parallel.max_over_ranks(3.5) == 3.5 and parallel.sum_over_ranks(2) == 2.0
    parallel.barrier()


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    """bench.py --impl reference under a multi-rank launch: the other ranks leave without work or output."""
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")

    class A:
        steps, warmup, gpus = 1, 0, 2
    bench.run_reference(A)
    assert capsys.readouterr().out == ""
