"""Oracle of the search-side host code: cost model, two-step sampling, enumeration (test infrastructure).

Plain and slow on purpose; shares no code with the library.  Only tests/, __graft_entry__.smoke() and
bench.py's cpu_baseline leg may import it.

What it follows (ELSA, arXiv 2409.09708):
  * Sec. 3: a configuration is one level per linear module; Sec. 3.2 / appendix "settings": the cost F is the
    FLOP count (Table 1 counts multiply-accumulates), C_upper = 50 % of the dense model's.
  * Alg. 3 (two-step sampling), taken in the paper's order: draw an interval of [C_lower, C_upper] uniformly,
    then draw a configuration from the per-layer level probabilities P_t among those whose cost lies in it.
    `two_step_rejection` is that, literally (draw level by level, keep the draw if its cost fits).
    `two_step_inverse_cdf` draws from the same distribution with given uniforms so that a deterministic
    implementation can be compared choice by choice: it enumerates every configuration of the interval, and
    picks each layer's level by inverse CDF over the levels in their given order from the conditional
    distribution of that layer given the earlier picks.  Only for small L (k^L configurations are listed).
  * Sec. 2: |S|^L configurations (3^48 for 48 modules and three levels).

Costs are exact integers (multiples of the caller's quantum) and interval edges are exact fractions.  The
last interval also contains C_upper (Sec. 3.2: configurations with F <= C_upper take part).
"""
from fractions import Fraction
from itertools import product


def config_cost(cost, choice, fixed=0):
    return fixed + sum(cost[l][s] for l, s in enumerate(choice))


def cost_table_macs(shapes, levels):
    """shapes: [(rows, in, out)], levels: [(N, M)]: multiply-accumulates of the kept weights (Sec. 2)."""
    return [[Fraction(r * i * o * n, m) for (n, m) in levels] for (r, i, o) in shapes]


def interval_of(total, lower, upper, n_intervals):
    """Index of the interval that holds `total`, or None outside [lower, upper]."""
    if total < lower or total > upper:
        return None
    if total == upper:
        return n_intervals - 1
    width = Fraction(upper - lower, n_intervals)
    for i in range(n_intervals):
        if lower + i * width <= total < lower + (i + 1) * width:
            return i
    return None


def lower_cost(cost):
    return sum(min(row) for row in cost)


def two_step_rejection(cost, P, upper, n_intervals, rng, max_tries=1000000):
    """Alg. 3 as written.  rng: numpy Generator.  Returns (choice, interval)."""
    L = len(cost)
    lower = lower_cost(cost)
    interval = int(rng.integers(0, n_intervals))
    for _ in range(max_tries):
        choice = []
        for l in range(L):
            p = [float(x) for x in P[l]]
            z = sum(p)
            choice.append(int(rng.choice(len(p), p=[x / z for x in p])))
        if interval_of(config_cost(cost, choice), lower, upper, n_intervals) == interval:
            return choice, interval
    raise RuntimeError("no accepted draw")


def conditional_by_enumeration(cost, P, upper, n_intervals, interval):
    """{configuration: probability} of P restricted to the interval (normalised), by listing every configuration."""
    L, k = len(cost), len(cost[0])
    lower = lower_cost(cost)
    out = {}
    for choice in product(range(k), repeat=L):
        if interval_of(config_cost(cost, choice), lower, upper, n_intervals) != interval:
            continue
        w = 1.0
        for l, s in enumerate(choice):
            w *= float(P[l][s]) / float(sum(P[l]))
        if w > 0:
            out[choice] = w
    z = sum(out.values())
    return {c: w / z for c, w in out.items()} if z > 0 else {}


def interval_masses(cost, P, upper, n_intervals):
    L, k = len(cost), len(cost[0])
    lower = lower_cost(cost)
    mass = [0.0] * n_intervals
    for choice in product(range(k), repeat=L):
        i = interval_of(config_cost(cost, choice), lower, upper, n_intervals)
        if i is None:
            continue
        w = 1.0
        for l, s in enumerate(choice):
            w *= float(P[l][s]) / float(sum(P[l]))
        mass[i] += w
    return mass


def two_step_inverse_cdf(cost, P, upper, n_intervals, uniforms):
    """Same distribution as two_step_rejection, driven by 1 + L uniforms in [0, 1).  Returns (choice, interval),
    choice None when the interval holds no configuration of non-zero probability."""
    L, k = len(cost), len(cost[0])
    interval = min(int(uniforms[0] * n_intervals), n_intervals - 1)
    cond = conditional_by_enumeration(cost, P, upper, n_intervals, interval)
    if not cond:
        return None, interval
    prefix = ()
    for l in range(L):
        w = [sum(p for c, p in cond.items() if c[:l] == prefix and c[l] == s) for s in range(k)]
        target = uniforms[l + 1] * sum(w)
        acc, pick = 0.0, None
        for s in range(k):
            if w[s] <= 0:
                continue
            acc += w[s]
            pick = s
            if target < acc:
                break
        prefix = prefix + (pick,)
    return list(prefix), interval


def search_space_size(n_layers, n_levels):
    return n_levels ** n_layers


def config_from_index(index, n_layers, n_levels):
    """Digit l of the index in base n_levels is the level of layer l."""
    choice = []
    for _ in range(n_layers):
        choice.append(index % n_levels)
        index //= n_levels
    assert index == 0
    return choice
