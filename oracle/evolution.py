"""CPU oracle of the evolutionary selection of low-bitwidth channel groups (Sec. 4.2, Algorithm 1).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH: only the tests, the smoke check and the
CPU-baseline leg of the benchmark import this module.  It shares nothing with the CUDA
library and never imports it.  Plain Python integers and loops.

What it follows: a chromosome holds one flag per feature channel (here per channel group, the
granularity the hardware computes at), ordered by layer; 1 = low bitwidth.  A generation ranks
the population by fitness (the L2 distance of the model's outputs from those of the 8-bit model:
smaller is fitter), carries the k fittest over unchanged, and fills the rest with offspring of
the r fittest: single-point crossover at a layer boundary, then mutation (each set flag is
cleared with a small probability and as many unset flags of the same layer are set, preferring
low error scores; a total that the crossover moved away from the target is brought back).
The seeds are one greedy selection (the lowest scores of every layer at an equal ratio) and
random ones that prefer low scores.

Readings where the text is silent (each is also listed in the design notes):
  * randomness: a counter-based generator, draw(seed, generation, individual, n) = splitmix64
    finaliser of a mix of the four counters; every decision below says which draw it takes;
  * draws that favour low error scores (Sec. 4.2): integer weight 2^32 // (1 + score);
    a flag to CLEAR in a repair is drawn with weight 1 + score; weighted draws walk the
    candidates in index order with value = draw % total weight;
  * parents of a pair: two independent draws among the r fittest (they may coincide); the
    crossover point is a layer boundary 1 .. n_layers-1; pairs fill the offspring in order,
    an odd last place takes the first child only;
  * mutation probability in basis points: a flag flips when draw % 10000 < rate (100 = 1 %);
    flags that were unset before the mutation of a layer are the candidates for the flags set
    in exchange; when a layer has fewer candidates than cleared flags the first cleared flags
    (index order) are set again;
  * locked flags (the groups selected at a smaller ratio, which every larger ratio must keep:
    nested selection) are set in every seed and are never cleared;
  * ranking: ascending distance, ties by index in the population.
"""
from __future__ import annotations

MASK = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
INIT_GENERATION = 0xFFFFFFFF      # generation counter of the draws that make the seeds


def _mix(z: int) -> int:
    z &= MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK
    return z ^ (z >> 31)


def draw(seed: int, generation: int, individual: int, n: int) -> int:
    """64 random bits that depend only on the four counters."""
    z = _mix(seed * _GOLD + _GOLD)
    z = _mix(z ^ ((generation + 1) * 0xD1B54A32D192ED03 & MASK))
    z = _mix(z ^ ((individual + 1) * 0x8CB92BA72F3D8DD7 & MASK))
    return _mix(z ^ ((n + 1) * _GOLD & MASK))


class _Draws:
    def __init__(self, seed, generation, individual):
        self.key = (seed, generation, individual)
        self.n = 0

    def next(self) -> int:
        v = draw(*self.key, self.n)
        self.n += 1
        return v


def _weight_set(score: int) -> int:
    return (1 << 32) // (1 + score)


def _pick(candidates, weights, value: int) -> int:
    """Weighted choice: candidates in index order, `value` already reduced modulo the total weight."""
    acc = 0
    for c, w in zip(candidates, weights):
        acc += w
        if value < acc:
            return c
    raise AssertionError("value outside the total weight")


def _offsets(groups):
    off = [0]
    for g in groups:
        off.append(off[-1] + g)
    return off


def greedy_seed(groups, score, per_layer_target, locked=None):
    """The lowest error scores of every layer (ties by index), locked flags first."""
    off = _offsets(groups)
    flags = [0] * off[-1]
    for l, g in enumerate(groups):
        idx = list(range(off[l], off[l + 1]))
        idx.sort(key=lambda i: (0 if locked and locked[i] else 1, score[i], i))
        for i in idx[:per_layer_target[l]]:
            flags[i] = 1
        if locked:
            for i in idx:
                if locked[i]:
                    flags[i] = 1
    return flags


def _repair(flags, score, locked, target, d: _Draws):
    total = sum(flags)
    while total > target:
        cand = [i for i, f in enumerate(flags) if f and not (locked and locked[i])]
        if not cand:
            break
        w = [1 + score[i] for i in cand]
        flags[_pick(cand, w, d.next() % sum(w))] = 0
        total -= 1
    while total < target:
        cand = [i for i, f in enumerate(flags) if not f]
        if not cand:
            break
        w = [_weight_set(score[i]) for i in cand]
        flags[_pick(cand, w, d.next() % sum(w))] = 1
        total += 1
    return flags


def init_population(groups, score, per_layer_target, N, seed, locked=None):
    """N seed chromosomes: the greedy one, then random ones that prefer low scores (same total)."""
    pop = [greedy_seed(groups, score, per_layer_target, locked)]
    target = sum(pop[0])          # = sum(per_layer_target) unless a layer has more locked flags than its share
    for i in range(1, N):
        flags = [1 if locked and locked[j] else 0 for j in range(sum(groups))]
        pop.append(_repair(flags, score, locked, target, _Draws(seed, INIT_GENERATION, i)))
    return pop


def rank(distance):
    return sorted(range(len(distance)), key=lambda i: (distance[i], i))


def mutate(flags, groups, score, locked, target, rate_bp, d: _Draws):
    off = _offsets(groups)
    flags = list(flags)
    for l in range(len(groups)):
        idx = range(off[l], off[l + 1])
        unset_before = [i for i in idx if not flags[i]]
        cleared = []
        for i in idx:
            if flags[i] and not (locked and locked[i]):
                if d.next() % 10000 < rate_bp:
                    cleared.append(i)
        for i in cleared:
            flags[i] = 0
        cand = list(unset_before)
        for _ in range(min(len(cleared), len(cand))):
            w = [_weight_set(score[i]) for i in cand]
            c = _pick(cand, w, d.next() % sum(w))
            flags[c] = 1
            cand.remove(c)
        for i in cleared[:max(0, len(cleared) - len(unset_before))]:
            flags[i] = 1
    return _repair(flags, score, locked, target, d)


def next_generation(pop, distance, groups, score, target, k, r, rate_bp, seed, generation, locked=None):
    """One generation of Algorithm 1: elites + mutated crossover offspring of the r fittest."""
    N = len(pop)
    order = rank(distance)
    elites = [list(pop[i]) for i in order[:k]]
    parents = order[:r]
    off = _offsets(groups)
    n_layers = len(groups)
    children = []
    pair = 0
    while len(children) < N - k:
        d = _Draws(seed, generation, N + pair)      # the pair's own stream, apart from the children's
        a = pop[parents[d.next() % len(parents)]]
        b = pop[parents[d.next() % len(parents)]]
        if n_layers > 1:
            cut = off[1 + d.next() % (n_layers - 1)]
            c1, c2 = a[:cut] + b[cut:], b[:cut] + a[cut:]
        else:
            c1, c2 = list(a), list(b)
        children.append(c1)
        if len(children) < N - k:
            children.append(c2)
        pair += 1
    out = elites
    for j, c in enumerate(children):
        out.append(mutate(c, groups, score, locked, target, rate_bp, _Draws(seed, generation, j)))
    return out


def run(fitness, groups, score, per_layer_target, N, k, r, rate_bp, generations, seed, locked=None):
    """Algorithm 1 end to end; `fitness(flags) -> int` is the distance to the 8-bit model's outputs.
    Returns (best flags, best distance, history of the best distance per generation)."""
    pop = init_population(groups, score, per_layer_target, N, seed, locked)
    target = sum(pop[0])
    history = []
    for g in range(generations):
        dist = [fitness(c) for c in pop]
        history.append(min(dist))
        pop = next_generation(pop, dist, groups, score, target, k, r, rate_bp, seed, g, locked)
    dist = [fitness(c) for c in pop]
    history.append(min(dist))
    best = rank(dist)[0]
    return pop[best], dist[best], history


# ------------------------------------------------------------------ fitness of a chromosome on a stack of linears
def selection_perm(flags_layer):
    """Group order of a layer for a selection: the selected groups (index order), then the others;
    the number of selected groups is the layer's low-bit prefix."""
    low = [j for j, f in enumerate(flags_layer) if f]
    high = [j for j, f in enumerate(flags_layer) if not f]
    return low + high, len(low)


def stack_forward(layers, X, flags, groups):
    """int8 outputs of a chain of quantized linears under a selection (Sec. 4.2: the outputs whose
    distance from the 8-bit model's is the fitness).  layers[l] = dict(Wq [K, N] int8, w_scale, bias,
    x_scale, y_scale, G, sx_group [K/G] static activation positions per ORIGINAL group); the first
    layer quantizes the fp32 X by Eq. 1, every later layer takes the previous int8 output as its
    quantized input (y_scale of layer l is x_scale of layer l + 1)."""
    import numpy as np

    import oracle

    off = _offsets(groups)
    q = oracle.quantize(X, layers[0]["x_scale"])
    for l, L in enumerate(layers):
        perm, n_low = selection_perm(flags[off[l]:off[l + 1]])
        perm = np.asarray(perm, dtype=np.int32)
        sw = oracle.weight_positions_linear(L["Wq"], L["G"], perm)
        sx_slab = np.asarray(L["sx_group"], dtype=np.uint8)[perm].copy()
        acc = oracle.mixed_gemm_acc(q, L["Wq"], L["G"], perm, sx_slab, sw, n_low)
        q = oracle.epilogue_i8(acc, L["x_scale"], L["w_scale"], L["bias"], L["y_scale"])
    return q


def sq_distance(a, b) -> int:
    """Squared L2 distance of two int8 tensors, exact."""
    import numpy as np

    d = a.astype(np.int64) - b.astype(np.int64)
    return int((d * d).sum())
