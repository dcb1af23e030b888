"""The greedy marginal-utility policy: the oracle against what the paper and the mathematics fix
(the utility formula on a worked case, the marginal-drop expression, the linear-programming bound
of the multiple-choice knapsack, brute force on tiny instances), and the library's C++
implementation against the oracle."""
import itertools
from fractions import Fraction

import numpy as np
import pytest
from scipy.optimize import linprog

import workloads
from oracle import policy


@pytest.fixture(scope="module")
def kvh():
    from paper_2509_00105_b200 import _build
    _build.build()
    import paper_2509_00105_b200 as k
    k.lib()
    return k


def dyadic_instance(rng, n, max_opts=5):
    """Inputs on which binary64 arithmetic is exact: small integer frequencies, qualities in 1/256,
    sizes in multiples of 4096, power-of-two alpha and bandwidth."""
    freq = rng.integers(1, 33, size=n).astype(float).tolist()
    options, begin = [], [0]
    for _ in range(n):
        k = int(rng.integers(1, max_opts + 1))
        sizes = sorted(rng.choice(np.arange(1, 4097), size=k, replace=False) * 4096, reverse=True)
        quals = sorted(rng.integers(0, 257, size=k) / 256.0, reverse=True)
        if rng.random() < 0.3:
            rng.shuffle(quals)                             # some entries with dominated options
        options += [(int(s), float(q)) for s, q in zip(sizes, quals)]
        begin.append(len(options))
    alpha = float(2.0 ** rng.integers(-2, 4))
    bandwidth = float(2.0 ** rng.integers(18, 24))
    return freq, options, begin, alpha, bandwidth


def brute_force(freq, options, begin, alpha, bandwidth, capacity):
    best = Fraction(-10 ** 18)
    per_entry = [[(0, Fraction(0))] + [(options[k][0], policy.utility(freq[i], alpha, bandwidth, *options[k]))
                                        for k in range(begin[i], begin[i + 1])] for i in range(len(freq))]
    for combo in itertools.product(*per_entry):
        if sum(s for s, _ in combo) <= capacity:
            best = max(best, sum(u for _, u in combo))
    return best


def test_utility_formula_on_a_worked_case():
    # Freq 2, alpha 1/2, quality 0.75, 1000 bytes at 500 B/s: 2 * (0.375 - 2) = -3.25
    assert policy.utility(2, 0.5, 500, 1000, 0.75) == Fraction(-13, 4)
    assert policy.utility(3, 2, 1 << 30, 0, 1.0) == 6             # nothing to load: only quality counts
    # the marginal utility drop of the paper, written with rates m > n of an entry of `size` bytes
    size, m, n, qm, qn = 1 << 20, Fraction(9, 16), Fraction(3, 16), 0.96875, 0.75
    um = policy.utility(4, 1, 1 << 24, size * m, qm)
    un = policy.utility(4, 1, 1 << 24, size * n, qn)
    chain = policy.hull_of_entry([(int(size * m), um, 0), (int(size * n), un, 1)])
    assert [p[2] for p in chain] == [0, 1, -1]
    assert (chain[0][1] - chain[1][1]) / (chain[0][0] - chain[1][0]) == (um - un) / (size * (m - n))


def test_hull_drops_dominated_and_lp_dominated_options():
    U = Fraction
    pts = [(100, U(10), 0), (80, U(9), 1), (60, U(3), 2), (40, U(6), 3), (90, U(4), 4), (100, U(7), 5)]
    chain = policy.hull_of_entry(pts)
    # 60 and 90 lie under the hull, the second 100 is dominated; 80 is LP-dominated by the edge 100 -> 40?
    # slopes from (100, 10): to 80: 0.05, to 40: 0.0667, to 0: 0.1  => 80 is a vertex
    assert [(p[0], p[2]) for p in chain] == [(100, 0), (80, 1), (40, 3), (0, -1)]
    drops = [(chain[i][1] - chain[i + 1][1]) / (chain[i][0] - chain[i + 1][0]) for i in range(len(chain) - 1)]
    assert drops == sorted(drops) and len(set(drops)) == len(drops)        # strictly growing: concave
    # nothing worth storing: eviction at once
    assert policy.hull_of_entry([(50, U(-1), 0), (20, U(0), 1)]) == [(0, U(0), -1)]
    # the best point is not the largest one
    assert [p[2] for p in policy.hull_of_entry([(100, U(5), 0), (50, U(8), 1)])] == [1, -1]


def test_capacity_extremes_and_monotonicity():
    rng = np.random.default_rng(1)
    freq, options, begin, alpha, bw = dyadic_instance(rng, 12)
    full, used_full, total_full = policy.assign_tier(freq, options, begin, alpha, bw, 10 ** 15)
    for i, ch in enumerate(full):                        # unlimited room: every entry at its best option
        us = [policy.utility(freq[i], alpha, bw, *options[k]) for k in range(begin[i], begin[i + 1])]
        assert (max(us) <= 0 and ch == -1) or us[ch] == max(us)
    none, used0, total0 = policy.assign_tier(freq, options, begin, alpha, bw, 0)
    assert set(none) == {-1} and used0 == 0 and total0 == 0
    prev = Fraction(-1)
    for cap in np.linspace(0, used_full, 25):
        _, used, total = policy.assign_tier(freq, options, begin, alpha, bw, int(cap))
        assert used <= int(cap) and total >= prev
        prev = total


@pytest.mark.parametrize("seed", range(12))
def test_greedy_against_brute_force_and_the_lp_bound(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(2, 6))
    freq, options, begin, alpha, bw = dyadic_instance(rng, n, max_opts=4)
    biggest = sum(max(options[k][0] for k in range(begin[i], begin[i + 1])) for i in range(n))
    capacity = int(rng.integers(0, biggest + 1))
    choice, used, total = policy.assign_tier(freq, options, begin, alpha, bw, capacity)
    assert used <= capacity
    opt = brute_force(freq, options, begin, alpha, bw, capacity)
    assert total <= opt
    # LP relaxation of the multiple-choice knapsack with a library solver: x[i][k] >= 0, sum_k x <= 1
    util = [float(policy.utility(freq[i], alpha, bw, *options[k])) for i in range(n) for k in range(begin[i], begin[i + 1])]
    A = [[float(options[k][0]) for k in range(len(options))]]
    for i in range(n):
        A.append([1.0 if begin[i] <= k < begin[i + 1] else 0.0 for k in range(len(options))])
    res = linprog(c=[-u for u in util], A_ub=A, b_ub=[float(capacity)] + [1.0] * n, bounds=(0, 1), method="highs")
    assert res.status == 0
    lp = -res.fun
    assert float(opt) <= lp + 1e-6
    # the greedy is the LP solution with its one fractional entry moved a full step down: it loses at
    # most the largest single step of any chain against the LP optimum
    slack = 0.0
    for i in range(n):
        pts = [(options[k][0], policy.utility(freq[i], alpha, bw, *options[k]), k - begin[i]) for k in range(begin[i], begin[i + 1])]
        ch = policy.hull_of_entry(pts)
        slack = max([slack] + [float(ch[j][1] - ch[j + 1][1]) for j in range(len(ch) - 1)])
    assert float(total) >= lp - slack - 1e-6
    # where the greedy stops exactly at capacity the LP solution is integral, hence optimal
    if used == capacity:
        assert total == opt


def test_more_frequent_entries_keep_more(kvh):
    """Identical entries that differ only in reuse frequency: a more frequent one never ends up with
    a smaller stored form than a less frequent one."""
    n = 16
    sizes = [kvh.level_bytes(k, 32, 1024, 256) * 8 for k in range(4)]
    qual = [1.0, 0.97, 0.9, 0.6]
    options = [(s, q) for _ in range(n) for s, q in zip(sizes, qual)]
    begin = list(range(0, 4 * n + 1, 4))
    freq = [float(n - i) for i in range(n)]
    capacity = int(3.3 * sizes[0])
    choice, used, _ = policy.assign_tier(freq, options, begin, 4.0, float(1 << 26), capacity)
    stored = [sizes[c] if c >= 0 else 0 for c in choice]
    assert stored == sorted(stored, reverse=True) and used <= capacity
    assert 0 < stored.count(0) < n and len(set(stored)) >= 3      # a mix of levels, not one fixed rate


@pytest.mark.parametrize("seed", range(20))
def test_library_matches_oracle_on_exact_instances(kvh, seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 40))
    freq, options, begin, alpha, bw = dyadic_instance(rng, n)
    biggest = sum(max(options[k][0] for k in range(begin[i], begin[i + 1])) for i in range(n))
    for capacity in (0, biggest // 7, biggest // 2, biggest):
        want, used, total = policy.assign_tier(freq, options, begin, alpha, bw, capacity)
        got, got_used, got_total = kvh.policy_assign(freq, options, begin, alpha, bw, capacity)
        assert got.tolist() == want and got_used == used and got_total == float(total)
    tiers = [(alpha, bw, biggest // 5), (alpha, bw / 64, biggest // 3)]
    want_t, want_c = policy.assign_tiers(freq, options, begin, tiers)
    got_t, got_c = kvh.policy_assign_tiers(freq, options, begin, tiers)
    assert got_t.tolist() == want_t and got_c.tolist() == want_c


def test_adaptive_choice_beats_every_fixed_form_on_the_synthetic_workload(kvh):
    """size() comes from the codec (kvh_plan_chunks for the level and the kept tokens); quality
    curves are synthetic.  Under the same capacity the greedy's total utility is at least that of
    storing every entry in one fixed form, most frequent first, as far as the tier holds (the static
    baselines of the paper's comparison), up to the one step the greedy may overshoot."""
    l, c = 32, 1024
    freq, tokens, forms, quality = workloads.policy_entries(200, seed=11)
    options, begin = [], [0]
    for i, n in enumerate(tokens):
        for j, (level, keep) in enumerate(forms):
            kept = max(1, int(n * keep))
            options.append((kvh.plan_chunks(l, c, kept, level)[1], quality[i][j]))
        begin.append(len(options))
    alpha, bw = 2.0, 25e9                                 # seconds per unit of quality; bytes/s of the tier
    full = sum(options[begin[i]][0] for i in range(len(freq)))
    capacity = full // 40
    choice, used, total = kvh.policy_assign(freq, options, begin, alpha, bw, capacity)
    assert used <= capacity
    util = lambda i, j: freq[i] * (alpha * options[begin[i] + j][1] - options[begin[i] + j][0] / bw)
    step = max(util(i, 0) for i in range(len(freq)))
    order = sorted(range(len(freq)), key=lambda i: -freq[i])
    for j in range(len(forms)):
        room, fixed = capacity, 0.0
        for i in order:
            if options[begin[i] + j][0] <= room and util(i, j) > 0:
                room -= options[begin[i] + j][0]
                fixed += util(i, j)
        assert total >= fixed - step
    kept_forms = {forms[ch] for ch in choice if ch >= 0}
    assert len(kept_forms) >= 3                           # the policy mixes methods and rates
    tier_of, _ = kvh.policy_assign_tiers(freq, options, begin, [(alpha, bw, capacity), (alpha, 1e9, full // 3)])
    assert (tier_of == 0).sum() == (choice >= 0).sum() and (tier_of == 1).sum() > 0
