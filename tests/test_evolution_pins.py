"""Pins of the evolutionary-selection oracle (Sec. 4.2, Algorithm 1): the generator against the
published splitmix64 sequence, the operators against their stated properties, the search against
brute force on a problem small enough to enumerate."""
import itertools

import numpy as np

import helpers
from oracle import evolution as ev


def _problem(seed=3):
    rng = np.random.default_rng(seed)
    groups = [6, 8, 6]
    score = [int(v) for v in rng.integers(0, 200, sum(groups))]
    return groups, score


def test_generator_is_splitmix64():
    # first three outputs of splitmix64 from state 0 (reference values of the published generator)
    state, out = 0, []
    for _ in range(3):
        state = (state + 0x9E3779B97F4A7C15) & ev.MASK
        out.append(ev._mix(state))
    assert out == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    # counters are independent inputs: changing any one changes the draw; values look uniform
    base = ev.draw(1, 2, 3, 4)
    assert len({base, ev.draw(2, 2, 3, 4), ev.draw(1, 3, 3, 4), ev.draw(1, 2, 4, 4), ev.draw(1, 2, 3, 5)}) == 5
    v = np.array([ev.draw(7, 0, 0, n) % 10000 for n in range(20000)])
    assert abs(v.mean() - 4999.5) < 60 and abs((v < 100).mean() - 0.01) < 0.003


def test_greedy_seed_is_the_lowest_scores_of_every_layer():
    groups, score = _problem()
    tgt = [3, 4, 3]
    flags = ev.greedy_seed(groups, score, tgt)
    off = np.cumsum([0] + groups)
    for l, g in enumerate(groups):
        s = np.array(score[off[l]:off[l + 1]])
        want = set(np.argsort(s, kind="stable")[:tgt[l]].tolist())
        assert {j for j in range(g) if flags[off[l] + j]} == want


def test_seeds_have_the_target_total_and_prefer_low_scores():
    groups = [40]
    score = [0] * 20 + [9] * 20           # weight 1 against 1/10
    counts = np.zeros(40)
    N = 400
    pop = ev.init_population(groups, score, [4], N, seed=5)
    for c in pop:
        assert sum(c) == 4 and set(c) <= {0, 1}
        counts += np.array(c)
    # without replacement from 20 + 20 flags, 4 picks: low scores are picked roughly 10 times as often
    ratio = counts[:20].sum() / max(1.0, counts[20:].sum())
    assert 6.0 < ratio < 16.0


def test_crossover_is_single_point_at_a_layer_boundary():
    groups, score = _problem()
    N, k, r = 10, 2, 4
    pop = ev.init_population(groups, score, [3, 4, 3], N, seed=9)
    # give every seed the same per-layer counts so that no repair is needed, and switch mutation off
    pop = [ev.greedy_seed(groups, [(s * (i + 3)) % 211 for s in score], [3, 4, 3]) for i in range(N)]
    dist = [(i * 37) % 11 for i in range(N)]
    nxt = ev.next_generation(pop, dist, groups, score, 10, k, r, 0, seed=9, generation=0)
    order = ev.rank(dist)
    assert nxt[:k] == [pop[i] for i in order[:k]]                      # elites, unchanged, in rank order
    parents = [pop[i] for i in order[:r]]
    cuts = [6, 14]
    for child in nxt[k:]:
        assert any(child == a[:c] + b[c:] for a in parents for b in parents for c in cuts)
    assert len(nxt) == N


def test_mutation_rate_and_conservation():
    groups = [200, 200]
    score = list(range(400))
    flags = [1 if i % 2 == 0 else 0 for i in range(400)]
    changed = 0
    trials = 60
    for t in range(trials):
        out = ev.mutate(flags, groups, score, None, 200, 100, ev._Draws(11, 0, t))
        assert sum(out[:200]) == 100 and sum(out[200:]) == 100       # exchanges stay inside a layer
        changed += sum(1 for a, b in zip(flags, out) if a == 1 and b == 0)
    # 200 set flags, 1 % each: 2 cleared per trial on average
    assert 0.6 * 2 * trials < changed < 1.5 * 2 * trials


def test_mutation_repairs_the_total_and_keeps_locked_flags():
    groups, score = _problem()
    locked = [0] * 20
    locked[1] = locked[7] = locked[15] = 1
    too_many = [1] * 20
    out = ev.mutate(too_many, groups, score, locked, 8, 100, ev._Draws(1, 0, 0))
    assert sum(out) == 8 and out[1] == out[7] == out[15] == 1
    too_few = [0] * 20
    too_few[1] = too_few[7] = too_few[15] = 1
    out = ev.mutate(too_few, groups, score, locked, 8, 100, ev._Draws(1, 0, 1))
    assert sum(out) == 8 and out[1] == out[7] == out[15] == 1
    pop = ev.init_population(groups, score, [3, 3, 2], 12, seed=4, locked=locked)
    assert all(sum(c) == 8 and c[1] == c[7] == c[15] == 1 for c in pop)


def test_best_distance_never_rises_and_reaches_the_brute_force_optimum():
    # 2 layers x 6 groups, 4 low groups in total: 495 selections, enumerable.  The fitness couples
    # the layers (error amplification): the greedy per-layer choice is not the optimum.
    groups = [6, 6]
    score = [5, 1, 9, 3, 7, 2, 4, 4, 8, 1, 6, 3]
    cost = [9, 8, 9, 1, 7, 6, 2, 5, 8, 7, 6, 1]

    def fitness(flags):
        a = sum(c for c, f in zip(cost[:6], flags[:6]) if f)
        b = sum(c for c, f in zip(cost[6:], flags[6:]) if f)
        return a * a + b * b + 3 * a * b

    best = min(fitness([1 if i in sel else 0 for i in range(12)]) for sel in itertools.combinations(range(12), 4))
    greedy = fitness(ev.greedy_seed(groups, score, [2, 2]))
    assert greedy > best
    flags, dist, hist = ev.run(fitness, groups, score, [2, 2], N=12, k=2, r=6, rate_bp=1500, generations=25, seed=2)
    assert all(b <= a for a, b in zip(hist, hist[1:]))                 # elitism
    assert sum(flags) == 4 and dist == fitness(flags) == hist[-1]
    assert dist == best


def test_selection_perm_puts_selected_groups_first():
    perm, n_low = ev.selection_perm([0, 1, 1, 0, 1])
    assert perm == [1, 2, 4, 0, 3] and n_low == 3


def test_stack_fitness_reduces_to_the_8bit_chain_and_to_zero_when_lossless():
    layers, X, groups, y8 = helpers.tiny_stack()
    none = [0] * sum(groups)
    assert np.array_equal(ev.stack_forward(layers, X, none, groups), y8)        # no low group: the plain int8 chain
    allset = [1] * sum(groups)
    d = ev.sq_distance(ev.stack_forward(layers, X, allset, groups), y8)
    assert d > 0                                                                  # 4-bit groups do add error
    half = ev.greedy_seed(groups, [1] * sum(groups), [g // 2 for g in groups])
    assert 0 < ev.sq_distance(ev.stack_forward(layers, X, half, groups), y8)
    # values that fit four bits on both sides (positions 0): every selection is lossless
    layers, X, groups, y8 = helpers.tiny_stack(small=True)
    q0 = __import__("oracle").quantize(X, layers[0]["x_scale"])
    assert np.abs(q0).max() <= 7
    first = [1] * groups[0] + [0] * (sum(groups) - groups[0])
    assert ev.sq_distance(ev.stack_forward(layers, X, first, groups), y8) == 0
    assert ev.sq_distance(np.array([1, -2, 3], np.int8), np.array([-1, 2, 3], np.int8)) == 4 + 16
