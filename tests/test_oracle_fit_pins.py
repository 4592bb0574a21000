"""Pins for the oracle's quantizer fits (CPU only).

Nothing here compares the oracle with itself: each test checks it against a
closed form, an invariant, a hand-worked value, or an independent float64
routine written differently (direct divide-and-round form in numpy).
"""
import numpy as np
import pytest

import windq_synth as ws

BITS = (8, 4, 3, 2)


def _rand_wsx(R, C, seed, T=64):
    W = ws.weights(R, C, seed).numpy()
    X = ws.activations(T, C, seed + 1).numpy()
    s = (X.astype(np.float64) ** 2).mean(0).astype(np.float32)
    return W, s


# ------------------------------------------------------------------ fp16 conversion
def test_half_to_float_all_patterns(oracle):
    h = np.arange(65536, dtype=np.uint16)
    want = h.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(x)) for x in h], np.float32)
    same = (got.view(np.uint32) == want.view(np.uint32)) | (np.isnan(got) & np.isnan(want))
    assert same.all()


def test_float_to_half_rne(oracle):
    rng = np.random.default_rng(0)
    vals = np.concatenate([
        rng.standard_normal(4000).astype(np.float32) * np.float32(10.0) ** rng.integers(-9, 5, 4000).astype(np.float32),
        # exact ties between neighbouring halves, subnormal edge, overflow edge
        np.array([1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 2.0 ** -25, 3 * 2.0 ** -25, 2.0 ** -24, 2.0 ** -14,
                  2.0 ** -14 - 2.0 ** -25, 65504.0, 65519.99, 65520.0, 70000.0, 0.0, -0.0, -1.0 - 2.0 ** -11,
                  5.9e-8, 2.9e-8, 3.0e-8, 1e-10], np.float32),
    ])
    with np.errstate(over="ignore"):
        want = vals.astype(np.float16).view(np.uint16)
    got = np.array([oracle.float_to_half(float(v)) for v in vals], np.uint16)
    assert (got == want).all()


# ------------------------------------------------------------------ PSUM8 summation order
def test_psum8_leaf_is_left_to_right(oracle):
    big = 2.0 ** 24
    x = np.zeros(16, np.float32)
    x[:3] = [big, 1, 1]           # (2^24 + 1) -> 2^24 (tie to even), again -> 2^24
    assert oracle.psum8(x) == big
    x[:3] = [1, 1, big]           # (1 + 1) + 2^24 = 2^24 + 2
    assert oracle.psum8(x) == big + 2


def test_psum8_tree_adds_adjacent_leaves_first(oracle):
    big = 2.0 ** 24
    x = np.zeros(32, np.float32)
    x[0], x[8], x[16], x[24] = 1, big, 1, -big
    # adjacent pairs: (1 + 2^24) = 2^24 ; (1 - 2^24) = -(2^24 - 1) ; sum = 1
    # left-to-right over leaves would give 0, pairing leaves (0,2),(1,3) would give 2
    assert oracle.psum8(x) == 1.0
    x = np.zeros(64, np.float32)
    x[0], x[8], x[16], x[24], x[32], x[40], x[48], x[56] = 1, big, 1, -big, 0.5, 0.25, big, -big
    # ((1)+(0.75 + 0)) with the second half: (0.5+0.25) + (2^24 - 2^24) = 0.75 -> 1.75
    assert oracle.psum8(x) == 1.75


# ------------------------------------------------------------------ independent float64 quantizer
def brute_uniform(w, s, bits, p):
    """Direct form in float64: q = clip(round(w / scale) + z), scale as stored in fp16."""
    w = w.astype(np.float64)
    qmax = 2 ** bits - 1
    mn, mx = min(0.0, w.min()), max(0.0, w.max())
    scale32 = np.float32(np.float32(np.float32(p) * np.float32(mx - mn)) * np.float32(1.0 / qmax))
    scale = float(np.float16(scale32))
    if scale == 0.0:
        scale = 1.0
    z = float(np.clip(np.round(-(float(np.float32(p)) * mn) / scale), 0, qmax))
    q = np.clip(np.round(w / scale) + z, 0, qmax)
    deq = (q - z) * scale
    return float((s.astype(np.float64) * (deq - w) ** 2).sum()), q.astype(np.int64), scale, z


@pytest.mark.parametrize("G", [8, 32])
def test_clip_search_against_brute_force(oracle, G):
    rng = np.random.default_rng(G)
    grid = ws.clip_grid(20)
    for trial in range(12):
        R = 3
        w16 = (rng.standard_t(4, size=(R, G)) * 0.02).astype(np.float16)
        s = rng.lognormal(0, 1, G).astype(np.float32)
        out = oracle.fit_eval(w16, G, s, grid)
        for r in range(R):
            w = w16[r].astype(np.float32)
            for bi, bits in enumerate(BITS):
                es = []
                for k, p in enumerate(grid):
                    sc, z, e, codes = oracle.uniform_candidate(w, s, bits, float(p))
                    be, bq, bsc, bz = brute_uniform(w, s, bits, float(p))
                    assert sc == bsc and z == bz
                    assert e == pytest.approx(be, rel=1e-5, abs=1e-12)
                    es.append(be)
                    # codes agree except where w/scale sits within rounding of a half-integer
                    assert (codes.astype(np.int64) != bq).mean() <= 1.0 / G
                k_star = int(out["clip_idx"][bi, 0, r])
                assert out["group_err"][bi, 0, r] == pytest.approx(es[k_star], rel=1e-5, abs=1e-12)
                assert min(es) >= es[k_star] * (1 - 1e-5) - 1e-12
                # first index among equal minima
                assert all(es[k] > es[k_star] * (1 - 1e-5) - 1e-12 for k in range(k_star))


def test_8bit_round_trip_on_grid_values(oracle):
    rng = np.random.default_rng(3)
    G, R = 128, 40
    grid = ws.clip_grid(20)
    q = rng.integers(0, 256, size=(R, G))
    q[:, 0], q[:, 1] = 0, 255
    z = rng.integers(0, 256, size=(R, 1))
    w16 = ((q - z) * 2.0 ** -10).astype(np.float16)
    assert (w16.astype(np.float64) == (q - z) * 2.0 ** -10).all()
    s = rng.lognormal(0, 1, G).astype(np.float32)
    fit = oracle.fit_eval(w16, G, s, grid)
    assert (fit["clip_idx"][0] == 19).all()
    assert (fit["group_err"][0] == 0.0).all()
    assert fit["err"][0, 0] == 0.0
    plan = oracle.apply_plan(w16, G, s, grid, np.array([1], np.uint8), fit["clip_idx"])
    assert (plan["codes"].reshape(R, G) == q).all()
    assert (plan["scales"].view(np.float16) == np.float16(2.0 ** -10)).all()
    assert (plan["zeros"].view(np.float16).astype(np.int64) == z.T).all()
    assert (plan["wq"] == w16.view(np.uint16)).all()


# ------------------------------------------------------------------ ternary / binary closed forms
def _alphas(oracle, w16, s, action):
    grid = ws.clip_grid(4)
    plan = oracle.apply_plan(w16, w16.shape[1], s, grid, np.array([action], np.uint8))
    return plan["scales"].view(np.float16)[0].astype(np.float64), plan


def test_binary_closed_form(oracle):
    rng = np.random.default_rng(5)
    G, R = 128, 64
    w16 = (rng.standard_normal((R, G)) * 0.02).astype(np.float16)
    w = w16.astype(np.float64)
    for s in (np.ones(G, np.float32), rng.lognormal(0, 1, G).astype(np.float32)):
        alpha, plan = _alphas(oracle, w16, s, 6)
        s64 = s.astype(np.float64)
        want = (np.abs(w) * s64).sum(1) / s64.sum()
        assert np.allclose(alpha, want, rtol=2.0 ** -11 * 1.01, atol=0)
        assert (np.abs(alpha - want) <= np.abs(np.float16(want).astype(np.float64) - want) + 1e-12).all()
        fit = oracle.fit_eval(w16, G, s, ws.clip_grid(4))
        A2, B, Cs = (s64 * w * w).sum(1), (s64 * np.abs(w)).sum(1), s64.sum()
        E = A2 - 2 * alpha * B + alpha * alpha * Cs           # expansion of sum s (w - alpha sign w)^2
        assert np.allclose(fit["group_err"][5, 0], E, rtol=1e-5)
        # alpha is the stationary point of E before fp16 rounding
        for f in (1 - 1e-3, 1 + 1e-3):
            assert ((A2 - 2 * want * f * B + (want * f) ** 2 * Cs) >= (A2 - 2 * want * B + want ** 2 * Cs)).all()
        # signs: bit = !(w < 0)
        bits = np.unpackbits(plan["codes"].reshape(R, G // 8), axis=1, bitorder="little")
        assert (bits == (~(w16 < 0)).astype(np.uint8)).all()


def test_binary_error_fraction_for_gaussian_weights(oracle):
    # s == 1, Gaussian w: E_bin / energy -> 1 - 2/pi
    w16 = ws.weights(512, 512, 11, outlier_frac=0.0).numpy()
    fit = oracle.fit_eval(w16, 128, np.ones(512, np.float32), ws.clip_grid(2))
    ratio = fit["err"][:, 5].astype(np.float64).sum() / fit["energy"].astype(np.float64).sum()
    assert ratio == pytest.approx(1 - 2 / np.pi, rel=0.01)


def test_ternary_closed_form(oracle):
    rng = np.random.default_rng(6)
    G, R = 128, 64
    w16 = (rng.standard_normal((R, G)) * 0.02).astype(np.float16)
    w = w16.astype(np.float64)
    for s in (np.ones(G, np.float32), rng.lognormal(0, 1, G).astype(np.float32)):
        alpha, plan = _alphas(oracle, w16, s, 5)
        s64 = s.astype(np.float64)
        delta = 0.7 * np.abs(w).mean(1, keepdims=True)
        sup = np.abs(w) > delta
        safe = np.abs(np.abs(w) - delta) > 1e-6 * delta       # away from the threshold's rounding
        want = (np.abs(w) * s64 * sup).sum(1) / (s64 * sup).sum(1)
        assert np.allclose(alpha, want, rtol=2.0 ** -11 * 1.01)
        # codes: 5 trits per byte, base 3, little-endian
        codes = plan["codes"].reshape(R, 26).astype(np.int64)
        trits = np.stack([(codes // 3 ** m) % 3 for m in range(5)], axis=2).reshape(R, 130)[:, :G]
        want_t = 1 + np.sign(w).astype(np.int64) * sup
        assert (trits[safe] == want_t[safe]).all()
        assert (trits != want_t).sum() <= 2
        assert (codes[:, 25] < 27).all()                       # last byte holds 3 trits only
        fit = oracle.fit_eval(w16, G, s, ws.clip_grid(4))
        deq = (trits - 1) * alpha[:, None]
        E = (s64 * (deq - w) ** 2).sum(1)
        assert np.allclose(fit["group_err"][4, 0], E, rtol=1e-5)


def test_ternary_falls_back_to_unit_weights_when_support_has_no_activation(oracle):
    G = 32
    w16 = np.zeros((1, G), np.float16)
    w16[0, :4] = [0.5, -0.25, 0.75, 0.5]
    s = np.ones(G, np.float32)
    s[:4] = 0                                                   # the whole support has s == 0
    alpha, plan = _alphas(oracle, w16, s, 5)
    assert alpha[0] == 0.5                                      # plain mean of |w| on the support
    s[:] = 0
    alpha, _ = _alphas(oracle, w16, s, 6)
    assert alpha[0] == np.float16(2.0 / 32)                     # binary: mean |w| over the group


# ------------------------------------------------------------------ invariants
def test_error_decreases_with_bit_width(oracle):
    # Unit-level invariant, without planted outlier columns or x50 hot channels:
    # 8 < 4 < 3 < 2 < 1.58 < 1 < energy.  (Both plants can legitimately break it below 3 bits.  With
    # clip ratios limited to [0.5, 1], a 4-level grid stretched over a x20 outlier maps every ordinary
    # weight to zero; and the ternary / binary scales are s-weighted, so they follow a hot channel,
    # while the uniform grid sees s only through the choice of clip ratio.)
    for dist in ("normal", "student_t"):
        W = ws.weights(256, 1024, 21, dist=dist, outlier_frac=0.0).numpy()
        X = ws.activations(64, 1024, 22, n_hot=0).numpy()
        s = (X.astype(np.float64) ** 2).mean(0).astype(np.float32)
        fit = oracle.fit_eval(W, 128, s, ws.clip_grid(20), threads=8)
        e = fit["err"].astype(np.float64)
        assert (np.diff(e, axis=1) > 0).all()
        assert (e[:, 5] < fit["energy"]).all()
    # nested grids at a fixed clip ratio (3 | 15 | 255): per group e8 <= e4 <= e2 up to fp16 scale
    # rounding, outlier columns or not
    W, s = _rand_wsx(8, 1024, 21)
    for u in range(8):
        for r in range(8):
            w = W[r, 128 * u:128 * u + 128].astype(np.float32)
            e8, e4, e2 = (oracle.uniform_candidate(w, s[128 * u:128 * u + 128], b, 1.0)[2] for b in (8, 4, 2))
            assert e8 <= e4 * 1.001 and e4 <= e2 * 1.001


def test_power_of_two_scale_invariance(oracle):
    W, s = _rand_wsx(64, 512, 31)
    grid = ws.clip_grid(20)
    base = oracle.fit_eval(W, 128, s, grid)
    W8 = (W.astype(np.float32) * 8).astype(np.float16)
    assert (W8.astype(np.float32) == W.astype(np.float32) * 8).all()
    up = oracle.fit_eval(W8, 128, s, grid)
    assert (up["clip_idx"] == base["clip_idx"]).all()
    assert (up["group_err"] == base["group_err"] * np.float32(64)).all()
    s4 = s * np.float32(4)
    up = oracle.fit_eval(W, 128, s4, grid)
    assert (up["clip_idx"] == base["clip_idx"]).all()
    assert (up["group_err"] == base["group_err"] * np.float32(4)).all()
    acts = np.array([4, 5, 6, 2], np.uint8)
    p0 = oracle.apply_plan(W, 128, s, grid, acts)
    p1 = oracle.apply_plan(W, 128, s4, grid, acts)
    assert (p0["codes"] == p1["codes"]).all() and (p0["scales"] == p1["scales"]).all()
    p8 = oracle.apply_plan(W8, 128, s, grid, acts)
    assert (p0["codes"] == p8["codes"]).all()
    assert (p8["scales"].view(np.float16) == p0["scales"].view(np.float16) * np.float16(8)).all()


def test_degenerate_groups(oracle):
    G, grid = 64, ws.clip_grid(20)
    s = np.linspace(0.5, 2.0, G).astype(np.float32)
    # all-zero group: every error 0, scale 1, zero 0, alpha 0
    Wz = np.zeros((2, G), np.float16)
    fit = oracle.fit_eval(Wz, G, s, grid)
    assert (fit["group_err"] == 0).all() and (fit["err"] == 0).all() and (fit["energy"] == 0).all()
    assert (fit["clip_idx"] == 0).all()
    for a, want_scale in ((1, 1.0), (4, 1.0), (5, 0.0), (6, 0.0)):
        plan = oracle.apply_plan(Wz, G, s, grid, np.array([a], np.uint8))
        assert (plan["scales"].view(np.float16) == np.float16(want_scale)).all()
        assert (plan["zeros"] == 0).all() and (plan["wq"] == 0).all()
    # constant positive group: range [0, c]; at p = 1 the top code reproduces c to fp16 scale accuracy
    c = np.float16(0.37)
    Wc = np.full((1, G), c, np.float16)
    for bits in BITS:
        sc, z, e, codes = oracle.uniform_candidate(Wc[0].astype(np.float32), s, bits, 1.0)
        assert z == 0 and (codes == 2 ** bits - 1).all()
        ulp = 2.0 ** -11 * float(c)
        assert e <= s.sum() * (ulp * 1.01) ** 2
    # one large outlier in a narrow group: 2-bit search clips (k* < K-1)
    rng = np.random.default_rng(9)
    Wo = (rng.standard_normal((4, G)) * 0.01).astype(np.float16)
    Wo[:, 7] = 0.5
    fit = oracle.fit_eval(Wo, G, np.ones(G, np.float32), grid)
    assert (fit["clip_idx"][3] < 19).all()


def test_zero_is_exactly_representable(oracle):
    # the grid always contains 0: a weight that is exactly 0 is reconstructed as 0
    rng = np.random.default_rng(10)
    G = 128
    W = (rng.standard_normal((16, G)) * 0.05).astype(np.float16)
    W[:, ::5] = 0
    s = np.ones(G, np.float32)
    for a in (1, 2, 3, 4):
        plan = oracle.apply_plan(W, G, s, ws.clip_grid(20), np.array([a], np.uint8))
        assert (plan["wq"][:, ::5] & 0x7fff == 0).all()


def test_energy_is_the_weighted_sum_of_squares_in_float64(oracle):
    """energy[u] = sum over the unit of s_j w_rj^2, pinned by the closed form in float64 with statistics that differ
    from channel to channel by orders of magnitude (a dropped or misplaced s_j, or a sum over the wrong axis, shows)."""
    rng = np.random.default_rng(77)
    R, G, U = 37, 64, 3
    W = (rng.standard_normal((R, U * G)) * 0.05).astype(np.float16)
    s = np.exp(rng.standard_normal(U * G) * 2.0).astype(np.float32)
    s[5] = 0.0
    s[G + 3] *= 1000.0
    fit = oracle.fit_eval(W, G, s, ws.clip_grid(5))
    w64 = W.astype(np.float64)
    for u in range(U):
        want = float((s[u * G:(u + 1) * G].astype(np.float64)[None, :] * w64[:, u * G:(u + 1) * G] ** 2).sum())
        assert abs(float(fit["energy"][u]) - want) <= 1e-6 * want
    # scaling one channel's statistic changes the energy by exactly that channel's share
    s2 = s.copy()
    s2[7] *= 4.0
    e2 = oracle.fit_eval(W, G, s2, ws.clip_grid(5))["energy"]
    share = 3.0 * float(s[7]) * float((w64[:, 7] ** 2).sum())
    assert abs((float(e2[0]) - float(fit["energy"][0])) - share) <= 1e-5 * float(e2[0])
    assert e2[1] == fit["energy"][1] and e2[2] == fit["energy"][2]


# ------------------------------------------------------------------ a candidate's error against single terms
def test_error_is_never_below_the_term_of_one_weight(oracle):
    """With s >= 0 every term (s d) d is >= 0 and rounding is monotone, so the PSUM8 error of a candidate is at least
    the rounded term of any single weight -- the fact the GPU's eight-bit search rests on when it leaves out
    candidates.  Checked here on the oracle alone, with the terms formed independently in float64 (c * scale - w is
    exact there, so one rounding to binary32 gives the fused result), on weight-like groups, on groups whose
    statistics span sixty binary orders, and on groups with a single live channel (where the error IS the term)."""
    rng = np.random.default_rng(11)
    f32 = np.float32
    checked = tight = 0
    for G in (32, 128, 512):
        for trial in range(12):
            w = ws.weights(1, G, 500 + 13 * trial + G, "student_t").numpy()[0].astype(np.float32)
            kind = trial % 3
            if kind == 0:
                s = (rng.standard_normal(G) ** 2).astype(np.float32)
            elif kind == 1:
                s = (2.0 ** rng.integers(-40, 20, G)).astype(np.float32)
            else:
                s = np.zeros(G, np.float32)
                s[int(rng.integers(0, G))] = f32(rng.uniform(0.1, 10.0))
            for bits in BITS:
                for p in (0.5, 0.7368421, 1.0):
                    scale, zero, err, codes = oracle.uniform_candidate(w, s, bits, p)
                    c = codes.astype(np.float64) - float(zero)
                    d = (c * float(scale) - w.astype(np.float64)).astype(np.float32)          # fma(c, scale, -w)
                    t = (s.astype(np.float32) * d).astype(np.float32)                         # s * d, rounded
                    term = (t.astype(np.float64) * d.astype(np.float64)).astype(np.float32)   # fl(t * d)
                    assert (term >= 0).all()
                    assert f32(err) >= term.max(), (G, trial, bits, p)
                    checked += 1
                    if kind == 2:
                        assert f32(err) == term.max()
                        tight += 1
    assert checked == 3 * 12 * 4 * 3 and tight == 3 * 4 * 4 * 3
