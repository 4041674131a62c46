"""Search-side host code (cost model, two-step sampling, enumeration): the oracle against what the paper and the
mathematics fix, then the library against the oracle.  No GPU."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import elsa_search_oracle as so

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


@pytest.fixture(scope="module")
def lib():
    from paper_2409_09708_b200 import build
    build.build()
    from paper_2409_09708_b200 import binding
    return binding


# DeiT-B per image (Sec. 4.1: 12 blocks, dim 768, MLP 3072, 197 tokens) in the N:4 space of the main experiments
DEIT_B = [(197, 768, 2304), (197, 768, 768), (197, 768, 3072), (197, 3072, 768)] * 12
N4 = [(1, 4), (2, 4), (4, 4)]
# what stays dense (attention products, patch embedding, head), in multiply-accumulates per image
DEIT_B_FIXED = 2 * 197 * 197 * 768 * 12 + 196 * 768 * 768 + 768 * 1000


# ------------------------------------------------------------------ pins of the oracle

def test_oracle_search_space_size_is_the_papers_3_to_the_48():
    with open(os.path.join(GOLDEN, "search_space_3pow48.txt")) as f:
        value = int([ln for ln in f if not ln.startswith("#")][0])
    assert so.search_space_size(48, 3) == value
    # every index decodes to a distinct configuration and back
    seen = {tuple(so.config_from_index(i, 4, 3)) for i in range(81)}
    assert len(seen) == 81 and so.config_from_index(80, 4, 3) == [2, 2, 2, 2] and so.config_from_index(5, 4, 3) == [2, 1, 0, 0]


def test_oracle_cost_model_reproduces_table1_for_deit_b():
    cost = so.cost_table_macs(DEIT_B, N4)
    with open(os.path.join(GOLDEN, "table1_flops.txt")) as f:
        row = [ln.split() for ln in f if ln.startswith("DeiT-B")][0]
    dense = so.config_cost(cost, [2] * 48, DEIT_B_FIXED)
    half = so.config_cost(cost, [1] * 48, DEIT_B_FIXED)
    assert round(float(dense) / 1e9, 1) == float(row[1]) and round(float(half) / 1e9, 1) == float(row[2])   # 17.6 G, 9.2 G
    # 2:4 multiplies exactly half of the weights of every module (Sec. 2)
    assert all(c[1] * 2 == c[2] and c[0] * 4 == c[2] for c in cost)


def test_oracle_conditional_distribution_has_its_closed_form_on_equal_layers():
    # L equal layers, two levels costing 0 and 1, uniform P: given the total m, every set of m layers is equally
    # likely, so a layer is at the dearer level with probability m / L
    L = 6
    cost = [[0, 1]] * L
    P = [[1.0, 1.0]] * L
    cond = so.conditional_by_enumeration(cost, P, L, 2, 0)          # totals 0, 1, 2 (interval [0, 3))
    z = sum(cond.values())
    assert abs(z - 1.0) < 1e-12
    # P(total = t | interval) is proportional to C(6, t)
    by_total = {t: sum(p for c, p in cond.items() if sum(c) == t) for t in (0, 1, 2)}
    assert by_total[1] / by_total[0] == pytest.approx(6.0) and by_total[2] / by_total[0] == pytest.approx(15.0)
    marg = sum(p for c, p in cond.items() if c[0] == 1)
    assert marg == pytest.approx((6 * 1 / 6 + 15 * 2 / 6) / 22)


def test_oracle_inverse_cdf_draws_from_the_distribution_of_algorithm_3_as_written():
    # the literal rejection sampler of Alg. 3 and the enumerated conditional distribution agree in frequency
    rng = np.random.default_rng(11)
    cost = [[1, 2, 4], [3, 6, 12], [4, 8, 16], [1, 2, 4], [2, 4, 8]]
    P = [[1, 2, 1], [1, 1, 1], [3, 1, 1], [1, 1, 2], [1, 1, 1]]
    upper, n_int = 30, 4
    counts = [dict() for _ in range(n_int)]
    hits = [0] * n_int
    draws = 6000
    for _ in range(draws):
        choice, i = so.two_step_rejection(cost, P, upper, n_int, rng)
        hits[i] += 1
        counts[i][tuple(choice)] = counts[i].get(tuple(choice), 0) + 1
    assert max(hits) - min(hits) < 6 * (draws / n_int) ** 0.5            # step 1: intervals uniformly
    for i in range(n_int):
        cond = so.conditional_by_enumeration(cost, P, upper, n_int, i)
        assert set(counts[i]) <= set(cond)
        for c, p in cond.items():
            if p * hits[i] >= 30:                                           # step 2: frequencies follow P restricted to I
                assert abs(counts[i].get(c, 0) - p * hits[i]) < 5 * (p * hits[i]) ** 0.5 + 1
    # and the inverse-CDF form reproduces those probabilities when its uniforms sweep a grid
    grid = (np.arange(40) + 0.5) / 40
    freq = {}
    for u1 in grid:
        for u2 in grid:
            choice, i = so.two_step_inverse_cdf(cost[:2], P[:2], 12, 1, [0.0, u1, u2])
            freq[tuple(choice)] = freq.get(tuple(choice), 0) + 1
    cond = so.conditional_by_enumeration(cost[:2], P[:2], 12, 1, 0)
    for c, p in cond.items():
        assert abs(freq.get(c, 0) / 1600 - p) < 0.03


# ------------------------------------------------------------------ the library against the oracle

def test_library_cost_model_and_enumeration_match_the_oracle(lib):
    cost = lib.elsa_cost_table_macs(DEIT_B, N4)
    ocost = so.cost_table_macs(DEIT_B, N4)
    assert all(float(o) == c for orow, row in zip(ocost, cost) for o, c in zip(orow, row))
    rng = np.random.default_rng(5)
    for _ in range(20):
        choice = [int(v) for v in rng.integers(0, 3, 48)]
        assert lib.elsa_config_cost(cost, choice, DEIT_B_FIXED) == float(so.config_cost(ocost, choice, DEIT_B_FIXED))
    assert lib.elsa_search_space_size(48, 3) == so.search_space_size(48, 3)
    assert lib.elsa_search_space_size(96, 5) == 5 ** 96
    for index in (0, 5, 80, 3 ** 48 - 1, 3 ** 47 + 12345678901234567):
        L = 4 if index <= 80 else 48
        assert lib.elsa_config_from_index(index, L, 3) == so.config_from_index(index, L, 3)
    with pytest.raises(lib.ElsaError):
        lib.elsa_config_from_index(81, 4, 3)                         # not below 3^4


def test_library_two_step_sampler_matches_the_oracle_choice_by_choice(lib):
    rng = np.random.default_rng(21)
    checked = 0
    for case in range(12):
        L = int(rng.integers(2, 8))
        k = int(rng.integers(2, 4))
        cost = [sorted(int(v) for v in rng.integers(0, 9, k)) for _ in range(L)]
        P = [[float(v) for v in rng.integers(0, 4, k)] for _ in range(L)]
        for row in P:
            if sum(row) == 0:
                row[0] = 1.0
        lower, top = sum(min(r) for r in cost), sum(max(r) for r in cost)
        upper = int(rng.integers(lower, top + 1))
        n_int = int(rng.integers(1, 5))
        fcost = [[float(v) for v in row] for row in cost]
        omass = so.interval_masses(cost, P, upper, n_int)
        mass = lib.elsa_interval_masses(fcost, P, 0.0, float(upper), n_int, 1.0)
        assert mass == pytest.approx(omass, abs=1e-12)
        for _ in range(40):
            u = [float(v) for v in rng.random(L + 1)]
            ochoice, ointerval = so.two_step_inverse_cdf(cost, P, upper, n_int, u)
            if ochoice is None:
                with pytest.raises(lib.ElsaError):
                    lib.elsa_two_step_sample(fcost, P, 0.0, float(upper), n_int, 1.0, u)
                continue
            choice, interval = lib.elsa_two_step_sample(fcost, P, 0.0, float(upper), n_int, 1.0, u)
            assert interval == ointerval and choice == ochoice, (case, cost, P, upper, n_int, u)
            checked += 1
    assert checked > 200


def test_library_sampler_at_full_size_fills_the_cost_range_evenly(lib):
    """DeiT-B, N:4 space, C_upper = 50 % of the dense FLOPs (appendix, settings): step 1 makes the intervals
    equally likely, every draw lands in its interval, and the paper's operating points (7.0 G, 6.0 G) are reached."""
    cost = lib.elsa_cost_table_macs(DEIT_B, N4)
    P = [[1.0, 1.0, 1.0]] * 48
    dense = lib.elsa_config_cost(cost, [2] * 48, DEIT_B_FIXED)
    c_upper = 0.5 * dense
    quantum = 197 * 768 * 768 / 4.0                                    # every module's cost is a multiple of it
    lower = lib.elsa_config_cost(cost, [0] * 48, DEIT_B_FIXED)
    n_int = 8
    rng = np.random.default_rng(3)
    hits = [0] * n_int
    costs = []
    for _ in range(800):
        u = [float(v) for v in rng.random(49)]
        choice, interval = lib.elsa_two_step_sample(cost, P, DEIT_B_FIXED, c_upper, n_int, quantum, u)
        f = lib.elsa_config_cost(cost, choice, DEIT_B_FIXED)
        width = (c_upper - lower) / n_int
        assert lower + interval * width - quantum <= f <= lower + (interval + 1) * width + quantum and f <= c_upper + 1e-3
        hits[interval] += 1
        costs.append(f)
    assert max(hits) - min(hits) < 6 * (800 / n_int) ** 0.5
    assert min(costs) < 6.0e9 < 7.0e9 < max(costs)                      # Table 1's 6.0 G and 7.0 G rows lie inside
    # the vanilla sampler (one interval, no budget) piles up around the mean instead (Sec. 3.2)
    vanilla = []
    for _ in range(400):
        u = [float(v) for v in rng.random(49)]
        choice, _ = lib.elsa_two_step_sample(cost, P, DEIT_B_FIXED, dense, 1, quantum, u)
        vanilla.append(lib.elsa_config_cost(cost, choice, DEIT_B_FIXED))
    assert np.std(vanilla) < 0.5 * np.std(costs) or np.mean(vanilla) > np.mean(costs)
