"""Pins of the oracle's search over the ternary assignment, and of the claim that the 1-bit fit needs none.

The paper names its low-bit operators (App. "Per-unit Scale Optimization", Sec. 3.5) without formulas; the oracle's
reading is a threshold search.  What fixes it here, independently of the oracle's own code: a case worked by hand
(tests/golden/ternary_threshold_search.txt), the exhaustive optimum over all 3^8 ternary codes of toy groups in
float64, the reduction to the 0.7 rule of the plain fit, exact power-of-two scalings, and a decoder of the packed
plan written in numpy.
"""
import itertools
import os

import numpy as np
import pytest

import windq_synth as ws

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "ternary_threshold_search.txt")


def read_cases():
    cases, cur = [], None
    with open(GOLDEN) as fh:
        for line in fh:
            t = line.split()
            if not t or t[0].startswith("#"):
                continue
            if t[0] == "case":
                cur = dict(name=t[1], cands=[])
                cases.append(cur)
            elif t[0] in ("weights", "stats", "ratios"):
                cur[t[0]] = np.array([float(x) for x in t[1:]], np.float32)
            elif t[0] == "cand":
                cur["cands"].append(dict(k=int(t[1]), alpha=float(t[3]), err=float(t[5]), trits=[int(x) for x in t[7:]]))
            elif t[0] == "best":
                cur["best"] = int(t[1])
    return cases


@pytest.mark.parametrize("case", read_cases(), ids=lambda c: c["name"])
def test_hand_worked_threshold_search(oracle, case):
    w, s = case["weights"], case["stats"]
    for c in case["cands"]:
        alpha, err, trits = oracle.ternary_candidate(w, s, float(case["ratios"][c["k"]]))
        assert alpha == c["alpha"] and err == c["err"] and trits.tolist() == c["trits"], c
    W = w.astype(np.float16)[None, :]
    out = oracle.fit_ternary_search(W, 8, s, case["ratios"])
    best = case["cands"][case["best"]]
    assert int(out["thr_idx"][0, 0]) == case["best"]
    assert float(out["alpha"][0, 0]) == best["alpha"] and float(out["group_err"][0, 0]) == best["err"]
    assert float(out["err"][0]) == best["err"]


def exhaustive_ternary(w, s):
    """Least s-weighted squared error over all codes t in {-1, 0, 1}^G with the best scale for each, in float64."""
    w, s = w.astype(np.float64), s.astype(np.float64)
    best = float((s * w * w).sum())                       # all zeros
    for t in itertools.product((-1.0, 0.0, 1.0), repeat=w.size):
        t = np.array(t)
        den = float((s * t * t).sum())
        if den == 0.0:
            continue
        alpha = float((s * t * w).sum()) / den
        if alpha <= 0.0:
            continue
        best = min(best, float((s * (w - alpha * t) ** 2).sum()))
    return best


def test_threshold_search_reaches_the_exhaustive_optimum_on_toy_groups(oracle):
    """With a threshold between every two neighbouring magnitudes the search sees every threshold support; the best
    of them must be the optimum over ALL ternary codes (the argument in the oracle: for a fixed scale the best code
    of w_j is sign(w_j) [|w_j| > alpha / 2], whatever s_j is).  A wrong sign, a wrong weighting of the scale or a
    support that is not a threshold set would leave a gap.  The scale is stored in fp16, hence the tolerance."""
    rng = np.random.default_rng(5)
    for trial in range(12):
        w = (rng.standard_normal(8) * 0.05).astype(np.float16).astype(np.float32)
        s = np.exp(rng.standard_normal(8)).astype(np.float32)
        if trial == 3:
            s[2] = 0.0
        a = np.sort(np.unique(np.abs(w)))
        mean = float(np.abs(w).astype(np.float64).sum() / 8)
        mids = np.concatenate([[a[0] * 0.5], (a[:-1] + a[1:]) / 2]) / mean
        grid = mids.astype(np.float32)
        out = oracle.fit_ternary_search(w.astype(np.float16)[None, :], 8, s, grid)
        want = exhaustive_ternary(w, s)
        got = float(out["group_err"][0, 0])
        assert got >= want * (1 - 1e-6)
        assert got <= want * (1 + 2e-3) + 1e-12, (trial, got, want)


def test_one_bit_fit_is_the_exhaustive_optimum(oracle):
    """With levels +-alpha the code sign(w_j) is the best one for every alpha > 0 and alpha has a closed form: the
    plain 1-bit fit is already the optimum over all 2^8 sign patterns, so no search is built for it."""
    rng = np.random.default_rng(6)
    for trial in range(12):
        w = (rng.standard_normal(8) * 0.05).astype(np.float16).astype(np.float32)
        s = np.exp(rng.standard_normal(8)).astype(np.float32)
        w64, s64 = w.astype(np.float64), s.astype(np.float64)
        best = np.inf
        for t in itertools.product((-1.0, 1.0), repeat=8):
            t = np.array(t)
            alpha = float((s64 * t * w64).sum() / s64.sum())
            if alpha > 0:
                best = min(best, float((s64 * (w64 - alpha * t) ** 2).sum()))
        alpha, err, bits = oracle.binary_candidate(w, s)
        assert err >= best * (1 - 1e-6) and err <= best * (1 + 2e-3) + 1e-12
        assert (bits == (w >= 0)).all() or (w == 0).any()


def test_a_grid_holding_only_the_textbook_ratio_gives_the_plain_fit(oracle):
    R, C, G = 30, 512, 128
    W = ws.weights(R, C, 8, "student_t").numpy()
    s = oracle.act_stats(ws.activations(64, C, 9).numpy())
    plain = oracle.fit_eval(W, G, s, ws.clip_grid(3))
    out = oracle.fit_ternary_search(W, G, s, np.array([0.7], np.float32))
    assert (out["thr_idx"] == 0).all()
    assert (out["group_err"].view(np.uint32) == plain["group_err"][4].view(np.uint32)).all()
    assert np.allclose(out["err"], plain["err"][:, 4], rtol=1e-6)
    acts = np.full(C // G, 5, np.uint8)
    a = oracle.apply_plan(W, G, s, ws.clip_grid(3), acts, plain["clip_idx"])
    b = oracle.apply_plan_searched(W, G, s, ws.clip_grid(3), acts, plain["clip_idx"], np.array([0.7], np.float32), out["thr_idx"])
    for key in ("codes", "scales", "zeros", "wq"):
        assert (a[key] == b[key]).all(), key
    assert (b["scales"] == out["alpha"].view(np.uint16)).all()


def test_search_never_loses_to_a_ratio_of_its_grid_and_takes_the_first_minimum(oracle):
    R, C, G = 40, 256, 64
    W = ws.weights(R, C, 18, "student_t").numpy()
    s = oracle.act_stats(ws.activations(64, C, 19).numpy())
    grid = np.linspace(0.3, 1.5, 13).astype(np.float32)
    out = oracle.fit_ternary_search(W, G, s, grid)
    for u in range(C // G):
        for r in range(0, R, 7):
            w = W[r, u * G:(u + 1) * G].astype(np.float32)
            errs = np.array([oracle.ternary_candidate(w, s[u * G:(u + 1) * G], float(p), False)[1] for p in grid], np.float32)
            k = int(out["thr_idx"][u, r])
            assert k == int(np.argmin(errs)) and out["group_err"][u, r] == errs[k]      # argmin: the first minimum
    # the textbook ratio on the grid: the searched error cannot exceed the plain fit's
    grid7 = np.array([0.4, 0.55, 0.7, 0.85, 1.0], np.float32)
    plain = oracle.fit_eval(W, G, s, ws.clip_grid(2))
    assert (oracle.fit_ternary_search(W, G, s, grid7)["group_err"] <= plain["group_err"][4]).all()


def test_power_of_two_scalings_are_exact(oracle):
    R, C, G = 16, 256, 128
    W = ws.weights(R, C, 28, "student_t")
    s = oracle.act_stats(ws.activations(64, C, 29).numpy())
    grid = np.linspace(0.3, 1.5, 9).astype(np.float32)
    a = oracle.fit_ternary_search(W.numpy(), G, s, grid)
    b = oracle.fit_ternary_search((W * 4).numpy(), G, s, grid)
    c = oracle.fit_ternary_search(W.numpy(), G, s * 8, grid)
    assert (a["thr_idx"] == b["thr_idx"]).all() and (a["thr_idx"] == c["thr_idx"]).all()
    assert (b["group_err"] == a["group_err"] * 16).all() and (c["group_err"] == a["group_err"] * 8).all()
    assert (b["alpha"].astype(np.float32) == a["alpha"].astype(np.float32) * 4).all() and (c["alpha"] == a["alpha"]).all()


def test_packed_searched_plan_decodes_to_the_scored_error(oracle):
    """A decoder written here (base-3 digits, alpha from the stored scales) turns the packed 1.58-bit plan back into
    weights; their s-weighted squared distance to W, in float64, is the error the search reported."""
    R, C, G = 12, 256, 128
    W = ws.weights(R, C, 38, "student_t").numpy()
    s = oracle.act_stats(ws.activations(64, C, 39).numpy())
    grid = np.linspace(0.3, 1.5, 9).astype(np.float32)
    fit = oracle.fit_ternary_search(W, G, s, grid)
    acts = np.full(C // G, 5, np.uint8)
    plan = oracle.apply_plan_searched(W, G, s, ws.clip_grid(2), acts, None, grid, fit["thr_idx"])
    bpg = (G + 4) // 5
    for u in range(C // G):
        base = int(plan["code_offsets"][u])
        for r in range(R):
            raw = plan["codes"][base + r * bpg: base + (r + 1) * bpg].astype(np.int64)
            digits = np.stack([(raw // 3 ** m) % 3 for m in range(5)], axis=1).reshape(-1)[:G]
            alpha = float(plan["scales"][u, r:r + 1].view(np.float16)[0])
            what = (digits - 1) * alpha
            assert (np.float16(what).view(np.uint16) == plan["wq"][r, u * G:(u + 1) * G]).all()
            e = float((s[u * G:(u + 1) * G].astype(np.float64) * (what - W[r, u * G:(u + 1) * G].astype(np.float64)) ** 2).sum())
            assert abs(e - float(fit["group_err"][u, r])) <= 1e-5 * e + 1e-12


def test_protected_search_with_infinite_thresholds_is_the_plain_search(oracle):
    R, C, G = 20, 256, 64
    W = ws.weights(R, C, 48, "student_t").numpy()
    s = oracle.act_stats(ws.activations(64, C, 49).numpy())
    grid = np.linspace(0.3, 1.5, 7).astype(np.float32)
    a = oracle.fit_ternary_search(W, G, s, grid)
    b = oracle.fit_ternary_search(W, G, s, grid, thresh=np.full(C // G, np.inf, np.float32))
    for k in ("thr_idx", "group_err", "err"):
        assert (a[k] == b[k]).all()
    assert (a["alpha"].view(np.uint16) == b["alpha"].view(np.uint16)).all()
    # a finite threshold takes the largest-key weights out: the error over what is left cannot grow
    sel = oracle.salient_select(W, G, s, 30000, want_mask=False)
    c = oracle.fit_ternary_search(W, G, s, grid, thresh=sel["thresh"])
    assert (c["err"] <= a["err"] * (1 + 1e-6)).all()
