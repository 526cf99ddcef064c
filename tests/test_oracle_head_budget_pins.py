"""Pins of the head-level budget rule (different numbers of kept tokens per KV head; the paper's Ada-KV /
HeadKV rows, Table 1): closed forms, hand-computed small cases (tests/golden/head_budgets.txt) and invariants."""
import os

import numpy as np

from oracle import qp_oracle as orc

RNG = np.random.default_rng(424242)


def test_equal_heads_get_equal_shares():
    Bt, Hkv, L, w, n_mean = 2, 4, 512 + 32, 32, 128
    row = RNG.random(L - w)
    pooled = np.broadcast_to(row, (Bt, Hkv, L - w)).copy()      # every head has the same scores
    n = orc.head_budgets(pooled, L, w, n_mean)
    # ties go to the lower head first, so shares differ by at most the tie run; with whole units and a total
    # that may not exceed Hkv * n_mean every head lands on n_mean or one unit below
    assert n.sum(1).max() <= Hkv * n_mean and np.all((n == n_mean) | (n == n_mean - 32))
    distinct = np.stack([RNG.permutation(row) for _ in range(Hkv)])[None].repeat(Bt, 0) + 0.0
    n2 = orc.head_budgets(distinct, L, w, n_mean)                # same multiset of scores per head, no ties across
    assert np.all(n2 == n_mean)


def test_one_head_holding_all_the_mass_takes_what_the_others_can_spare():
    Hkv, L, w, n_mean = 4, 1024 + 32, 32, 128
    P = L - w
    pooled = RNG.random((1, Hkv, P)) * 1e-3
    pooled[0, 2] += 1.0                                          # head 2 outranks everything else
    n = orc.head_budgets(pooled, L, w, n_mean)[0]
    k_total = Hkv * (n_mean - w)                                 # 384 marked positions, all in head 2
    assert k_total == 384
    # raw shares: head 2 -> 384 + 32 = 416, the others -> 32 -> raised to 64 each (one unit above w):
    # total 416 + 192 = 608 > 512, so head 2 gives back 3 units: 320
    assert n.tolist() == [64, 64, 320, 64]


def test_hand_computed_cases_from_the_golden_file():
    path = os.path.join(os.path.dirname(__file__), "golden", "head_budgets.txt")
    rows = [l.split("|") for l in open(path) if l.strip() and not l.startswith("#")]
    assert rows
    for params, scores, want in rows:
        L, w, n_mean, unit, Hkv = map(int, params.split())
        pooled = np.array(list(map(float, scores.split())), np.float64).reshape(1, Hkv, L - w)
        got = orc.head_budgets(pooled, L, w, n_mean, unit)[0].tolist()
        assert got == list(map(int, want.split())), (params, got)


def test_invariants_on_random_scores_and_brute_force_counts():
    for trial in range(12):
        Hkv = int(RNG.integers(1, 7)); w = int(RNG.choice([4, 8, 32])); unit = int(RNG.choice([8, 32]))
        L = w + int(RNG.integers(3, 12)) * unit + int(RNG.integers(0, unit))
        n_mean = max(((w // unit) + 2) * unit, (int(RNG.integers(w + 1, L)) // unit) * unit)
        n_mean = min(n_mean, (L // unit) * unit)
        P = L - w
        pooled = np.round(RNG.random((2, Hkv, P)) * 6) / 6           # many ties
        n = orc.head_budgets(pooled, L, w, n_mean, unit)
        assert np.all(n % unit == 0) and np.all(n > w) and np.all(n <= L)
        n_min = (w // unit) * unit + unit
        assert np.all(n.sum(1) <= max(Hkv * n_mean, Hkv * n_min))
        # independent count of the marked positions: k-th largest value, then ties in (head, position) order
        for b in range(2):
            k_total = min(Hkv * (n_mean - w), Hkv * P)
            flat = pooled[b].ravel()
            order = np.lexsort((np.arange(flat.size), -flat))         # score desc, flat index asc
            marked = np.zeros(flat.size, bool); marked[order[:k_total]] = True
            raw = marked.reshape(Hkv, P).sum(1) + w
            floor = (raw // unit) * unit
            untouched = (floor >= n_min) & (floor <= (L // unit) * unit)
            if floor.clip(n_min, (L // unit) * unit).sum() <= Hkv * n_mean:   # no give-back happened
                assert np.array_equal(n[b][untouched], floor[untouched])
