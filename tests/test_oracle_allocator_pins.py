"""Pins for the oracle's heuristic allocator rule (CPU only): hand-worked cases, the ranking against
numpy's stable sort, a closed form for equal units, and the properties the rule's three steps imply."""
import os

import numpy as np
import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "heuristic_allocator.txt")

CENTI = np.array([1600, 800, 400, 300, 200, 158, 100], np.int64)


def read_cases():
    cases, cur = [], None
    for line in open(GOLDEN):
        line = line.split("#")[0].split()
        if not line:
            continue
        if line[0] == "case":
            cur = {"name": line[1], "args": [int(x) for x in line[2:6]], "units": []}
            cases.append(cur)
        elif line[0] == "unit":
            cur["units"].append((float(line[1]), int(line[2]), int(line[3]), int(line[4])))
        else:
            cur[line[0]] = [int(x) for x in line[1:]]
    return cases


@pytest.mark.parametrize("case", read_cases(), ids=lambda c: c["name"])
def test_hand_worked_cases(oracle, case):
    target, headroom, sb, zb = case["args"]
    sal, n, p, g = (np.array(x) for x in zip(*case["units"]))
    actions, order, total = oracle.greedy_allocate(sal, n, g, target, headroom, n_protected=p, scale_bits=sb, zero_bits=zb)
    assert order.tolist() == case["expect_order"]
    assert actions.tolist() == case["expect_actions"]
    assert total == case["expect_total"][0]


def test_ranking_is_numpy_stable_sort_descending(oracle):
    rng = np.random.default_rng(5)
    sal = rng.choice(rng.random(40).astype(np.float32), 1000)      # many equal scores
    n = np.full(1000, 64)
    _, order, _ = oracle.greedy_allocate(sal, n, n // 32, 200, 0)
    assert np.array_equal(order, np.argsort(-sal.astype(np.float64), kind="stable"))


def test_ranking_of_signed_zeros_and_negative_scores(oracle):
    sal = np.array([-1.0, 0.0, -0.0, 2.0, -np.inf, np.inf, 1e-45, -1e-45], np.float32)
    _, order, _ = oracle.greedy_allocate(sal, np.full(8, 32), np.ones(8, np.int64), 200, 0)
    assert order.tolist() == [5, 3, 6, 1, 2, 7, 0, 4]


def unit_costs(oracle, actions, n, p, g, sb, zb):
    """Eq. 6 per unit through the oracle's own accounting call (pinned by the Eq. 6 fixtures), one unit at a time."""
    out = np.zeros(len(n), np.int64)
    for u in range(len(n)):
        G = n[u] // g[u]
        out[u] = oracle.effective_bits_protected(np.array([actions[u]], np.uint8), np.array([p[u]], np.int64), int(g[u]), int(G), sb, zb)["total_centibits"]
    return out


@pytest.mark.parametrize("target", [100, 120, 158, 160, 179, 200, 230, 300, 400, 450])
def test_equal_units_closed_form(oracle, target):
    """U equal units without protection or parameter bits and no headroom: the number of moves of each
    step follows from the budget alone."""
    U, n = 50, 4096
    sal = np.arange(U, dtype=np.float32)[::-1].copy()             # unit index = rank
    actions, order, total = oracle.greedy_allocate(sal, np.full(U, n), np.full(U, n // 128), target, 0)
    assert order.tolist() == list(range(U))
    budget = target * U * n
    if target >= 200:
        # no unit moves down; k4 units at 4 bit as long as the budget holds, then at most one at 3 bit
        k4 = min(U, (budget - 200 * U * n) // (200 * n))
        rest = budget - 200 * U * n - k4 * 200 * n
        k3 = min(U - k4, rest // (100 * n))
        expect = [2] * k4 + [3] * k3 + [4] * (U - k4 - k3)
    else:
        d1 = min(U, -(-(200 * U * n - budget) // (42 * n)))        # moves of the first sweep (ceil)
        if d1 < U or 158 * U * n <= budget:
            d2 = 0
        else:
            d2 = min(U, -(-(158 * U * n - budget) // (58 * n)))
        expect = [4] * (U - d1) + [5] * (d1 - d2) + [6] * d2
        if d1 < U:
            # whatever the last move freed beyond the budget can promote the top unit only if >= 100 n
            slack = budget - (200 * (U - d1) + 158 * d1) * n
            assert slack < 42 * n
    assert actions.tolist() == expect
    assert total == int(CENTI[actions].sum()) * n


@pytest.mark.parametrize("seed", range(6))
def test_properties_of_the_three_steps(oracle, seed):
    rng = np.random.default_rng(100 + seed)
    U = 300
    G = rng.choice([32, 64, 128], U)
    g = rng.integers(1, 40, U)                                     # groups (rows) per unit
    n = G * g
    p = (n * rng.choice([0.0, 0.02, 0.03, 0.2], U)).astype(np.int64)
    sal = rng.choice(rng.random(100).astype(np.float32), U)
    target = int(rng.choice([150, 190, 200, 218, 240, 300]))
    headroom = int(rng.choice([0, 5, 20]))
    sb, zb = int(rng.choice([0, 16])), int(rng.choice([0, 8]))
    actions, order, total = oracle.greedy_allocate(sal, n, g, target, headroom, n_protected=p, scale_bits=sb, zero_bits=zb)
    N = int(n.sum())
    budget, floor = target * N, (target - headroom) * N
    assert set(actions.tolist()) <= {2, 3, 4, 5, 6}
    assert total == int(unit_costs(oracle, actions, n, p, g, sb, zb).sum())
    ranked = actions[order]
    # moved-down units are the tail of the ranking, the 1-bit units the tail of that, and a 1-bit unit
    # exists only if no unit is left above 1.58 bit
    down = ranked >= 5
    assert not down.any() or down[np.argmax(down):].all()
    one = ranked == 6
    assert not one.any() or (one[np.argmax(one):].all() and down.all())
    # step 2 stops as soon as it can: before its last move the total was above the floor
    before_promo = np.where(actions < 4, 4, actions)
    c_before = unit_costs(oracle, before_promo, n, p, g, sb, zb)
    t_before = int(c_before.sum())
    if down.any():
        last = order[np.argmax(one)] if one.any() else order[np.argmax(down)]
        undone = before_promo.copy()
        undone[last] -= 1
        assert int(unit_costs(oracle, undone, n, p, g, sb, zb).sum()) > floor
        assert t_before <= floor or (ranked == 6).all()
    else:
        assert t_before == int(unit_costs(oracle, np.full(U, 4), n, p, g, sb, zb).sum())
    # step 3 never exceeds the budget and leaves no move that still fits
    if t_before <= budget:
        assert total <= budget
    c_final = unit_costs(oracle, actions, n, p, g, sb, zb)
    for up in (3, 2):
        alt = actions.copy()
        cand = actions == up + 1
        alt[cand] = up
        c_alt = unit_costs(oracle, alt, n, p, g, sb, zb)
        assert ((total - c_final + c_alt)[cand] > budget).all()
    if t_before > budget:
        assert (actions >= 4).all()
