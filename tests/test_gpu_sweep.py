"""Seeded sweep over the parameter space of one clustering round and of short schedules: chunk sizes on every kernel
(warp-per-chunk 64, tile 128, tensor-memory 256, general even sizes, no chunking), both ranking scopes, sinks and recent
tokens, ragged lengths, degrees above one, both dtypes -- each case element by element against the oracle."""
import random

import pytest

import test_gpu_compress as TC

pytestmark = pytest.mark.gpu


def cases(n, seed):
    rng = random.Random(seed)
    out = []
    for i in range(n):
        chunk = rng.choice([0, 2, 6, 16, 62, 64, 64, 128, 128, 256, 256, 200])
        dtype = "bf16" if chunk == 0 else rng.choice(["bf16", "bf16", "f32"])
        s = rng.choice([rng.randint(3, 700), rng.randint(700, 2600), 64 * rng.randint(1, 30), 256 * rng.randint(1, 9) + rng.randint(0, 70)])
        sink, recent = rng.choice([(0, 0), (0, 0), (16, 64), (rng.randint(0, 9), rng.randint(0, 40))])
        r = rng.choice([1.0, 1.0, 0.8, 0.5, 0.3, 0.07])
        select = rng.randint(0, 1)
        deg_max = rng.choice([1, 1, 3, 300, 70000])
        out.append(pytest.param(chunk, dtype, s, sink, recent, r, select, deg_max, 1000 + i, id=f"{i}-c{chunk}-{dtype}-s{s}-r{r}-sel{select}-deg{deg_max}"))
    return out


@pytest.mark.parametrize("chunk,dtype,s,sink,recent,r,select,deg_max,seed", cases(40, 2024))
def test_single_round_sweep(chunk, dtype, s, sink, recent, r, select, deg_max, seed):
    b = TC.B()
    TC.single_round_case(1, 2, s, dtype, TC.one_round(b, chunk, r, select, sink, recent), seed=seed, deg_max=deg_max)


def schedules(n, seed):
    rng = random.Random(seed)
    out = []
    for i in range(n):
        chunk = rng.choice([0, 8, 64, 64, 128, 256])
        s = rng.randint(600, 3000)
        select = rng.randint(0, 1)
        r_init, decay = rng.choice([(0.8, 0.2), (1.0, 0.0), (0.6, 0.1), (0.9, 0.3)])
        budget = rng.choice([0, s // 4, s // 3, s // 2])
        rounds = 2 if budget == 0 else 16
        out.append(pytest.param(chunk, s, select, r_init, decay, budget, rounds, 3000 + i,
                                id=f"{i}-c{chunk}-s{s}-sel{select}-r{r_init}-d{decay}-B{budget}"))
    return out


@pytest.mark.parametrize("chunk,s,select,r_init,decay,budget,rounds,seed", schedules(12, 7))
def test_schedule_sweep(chunk, s, select, r_init, decay, budget, rounds, seed):
    b = TC.B()
    p = b.Params(chunk=chunk, n_sink=16, n_recent=64, n_rounds_max=rounds, r_init=r_init, r_decay=decay,
                 r_min=max(decay, 0.2), select=select, budget=budget)
    TC.multi_round_case(1, 2, s, "bf16", p, seed=seed)


def decode_cases(n, seed):
    rng = random.Random(seed)
    out = []
    for i in range(n):
        H = rng.choice([1, 2, 4, 8])
        G = rng.choice([1, 2, 4, 7, 8])
        Bz = rng.choice([1, 1, 2, 3, 5, 12, 40])
        top = rng.choice([40, 300, 3000, 9000, 20000]) if Bz * H <= 16 else rng.choice([40, 300, 2000])
        lens = [rng.choice([0, 1, rng.randint(1, top), top]) for _ in range(Bz)]
        dtype = rng.choice(["bf16", "bf16", "bf16", "f32"])
        out.append(pytest.param(lens, H, G, dtype, rng.random() < 0.8, 5000 + i, id=f"{i}-B{Bz}-H{H}-G{G}-{dtype}-top{top}"))
    return out


@pytest.mark.parametrize("lens,H,G,dtype,with_deg,seed", decode_cases(24, 11))
def test_decode_sweep(lens, H, G, dtype, with_deg, seed):
    """Batch sizes and lengths on both sides of every launch choice of the decode path (thread-block clusters of 16, 10
    and 8 CTAs, split kernel + combine), empty and one-token sequences included."""
    import test_gpu_decode as TD
    caches = TD.build_batch(lens, [n + 5 for n in lens], H, dtype, seed=seed, with_deg=with_deg)
    TD.check_decode(caches, H, G, dtype, seed=seed + 1)
