"""Evolutionary selection (Sec. 4.2, Algorithm 1): the library's host-side operators against the
oracle, flag for flag.  No GPU: these entry points do no device work."""
import numpy as np
import pytest

from oracle import evolution as ev
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import inputs


def _problem(n_layers, seed, max_groups=24, score_hi=16000):
    u = inputs.uniform(seed, 0, n_layers)
    groups = [int(2 + v * (max_groups - 2)) for v in u]
    score = [int(v * score_hi) for v in inputs.uniform(seed, 1, sum(groups))]
    return groups, score


@pytest.mark.parametrize("n_layers,seed", [(1, 1), (2, 2), (5, 3), (12, 4)])
@pytest.mark.parametrize("with_locked", [False, True])
def test_seeds_match(n_layers, seed, with_locked):
    groups, score = _problem(n_layers, seed)
    tgt = [g // 2 for g in groups]
    locked = None
    if with_locked:
        locked = [1 if v < 0.15 else 0 for v in inputs.uniform(seed, 2, sum(groups))]
    want = ev.init_population(groups, score, tgt, 9, seed=seed + 100, locked=locked)
    got, target = fx.flexiq_evo_init(groups, score, tgt, 9, seed + 100, locked)
    assert target == sum(want[0])
    assert got.tolist() == want


@pytest.mark.parametrize("n_layers,seed,N,k,r,bp", [(1, 11, 6, 2, 3, 100), (3, 12, 8, 2, 4, 100), (6, 13, 11, 1, 5, 2500),
                                                  (4, 14, 7, 0, 7, 10000), (5, 15, 8, 8, 2, 100), (8, 16, 16, 2, 8, 0)])
def test_generations_match(n_layers, seed, N, k, r, bp):
    groups, score = _problem(n_layers, seed)
    tgt = [max(1, g // 3) for g in groups]
    locked = [1 if v < 0.1 else 0 for v in inputs.uniform(seed, 2, sum(groups))] if seed % 2 else None
    pop = ev.init_population(groups, score, tgt, N, seed=seed, locked=locked)
    target = sum(pop[0])
    got = np.array(pop, dtype=np.uint8)
    for gen in range(6):
        # any deterministic fitness serves here: the operators only see the numbers
        dist = [int(sum((i + 1) * f * (1 + s % 7) for i, (f, s) in enumerate(zip(c, score))) % 1000) for c in pop]
        pop = ev.next_generation(pop, dist, groups, score, target, k, r, bp, seed, gen, locked)
        got = fx.flexiq_evo_next_generation(got, dist, groups, score, target, k, r, bp, seed, gen, locked)
        assert got.tolist() == pop, gen
        assert all(sum(c) == target for c in pop)


def test_argument_errors():
    groups, score = [4, 4], [1] * 8
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_evo_init(groups, [-1] + [1] * 7, [2, 2], 4, 0)                  # negative score
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_evo_init(groups, score, [5, 2], 4, 0)                            # more than the layer holds
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_evo_init([0, 4], [1] * 4, [0, 2], 4, 0)                          # empty layer
    pop, target = fx.flexiq_evo_init(groups, score, [2, 2], 4, 0)
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_evo_next_generation(pop, [0] * 4, groups, score, target, 5, 2, 100, 0, 0)   # k > N
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_evo_next_generation(pop, [0] * 4, groups, score, target, 1, 0, 100, 0, 0)   # no parents
    with pytest.raises(fx.FlexiqError):
        fx.flexiq_evo_next_generation(pop, [0] * 4, groups, score, target, 1, 2, 20000, 0, 0)  # rate
