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
