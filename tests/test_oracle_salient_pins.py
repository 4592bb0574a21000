"""Pins for the oracle's salient-weight selection and Eq. 6 with protected weights (CPU only)."""
import os

import numpy as np
import pytest

import windq_synth as ws

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def numpy_selection(W, G, s, rate_ppm):
    """Independent restatement: keys in float32 with numpy, selection by a full sort."""
    R, C = W.shape
    a = np.sqrt(s.astype(np.float32))
    key = np.abs(W.astype(np.float32)) * a[None, :]
    assert key.dtype == np.float32
    U, n = C // G, R * G
    n_p = rate_ppm * n // 1_000_000
    thresh = np.full(U, np.inf, np.float32)
    mask = np.zeros((R, C), bool)
    for u in range(U):
        if n_p == 0:
            continue
        k = key[:, u * G:(u + 1) * G]
        thresh[u] = np.sort(k.ravel())[::-1][n_p - 1]
        mask[:, u * G:(u + 1) * G] = k >= thresh[u]
    return thresh, mask


def unpack_mask(mask_bytes, C):
    return np.unpackbits(mask_bytes, axis=1, bitorder="little")[:, :C].astype(bool)


@pytest.mark.parametrize("R,C,G,rate", [(64, 256, 128, 30000), (33, 128, 32, 20000), (100, 512, 256, 123456), (7, 64, 64, 500000)])
def test_selection_against_a_full_sort(oracle, R, C, G, rate):
    W = ws.weights(R, C, 900 + R, "student_t").numpy()
    s = ws.activations(64, C, 901).numpy().astype(np.float32)
    s = (s * s).mean(0).astype(np.float32)
    got = oracle.salient_select(W, G, s, rate)
    thresh, mask = numpy_selection(W, G, s, rate)
    assert (got["thresh"] == thresh).all()
    assert (unpack_mask(got["mask"], C) == mask).all()
    assert (got["count"] == mask.reshape(R, C // G, G).sum((0, 2))).all()
    assert (got["count"] >= rate * R * G // 1_000_000).all()


def test_count_arithmetic_and_extremes(oracle):
    for line in open(os.path.join(GOLDEN, "eq6_protected.txt")):
        t = line.split()
        if t and t[0] == "count":
            rate, R, G, want = map(int, t[1:])
            assert rate * R * G // 1_000_000 == want
            # a unit of that size whose keys are all different: exactly `want` weights are protected.
            # |w| takes 1024 values, the channel scales are 128 distinct powers of two apart by far more
            # than the spread of |w|, rows repeat |w| with a period that no two rows share a (value, channel)
            Wd = (1.0 + ((np.arange(R)[:, None] * 37 + np.arange(G)[None, :] * 5) % 1024) / 1024.0).astype(np.float16)
            got = oracle.salient_select(Wd, G, (4.0 ** (np.arange(G) - 64)).astype(np.float32), rate)
            assert got["count"][0] >= want
            keys = np.abs(Wd.astype(np.float32)) * np.sqrt((4.0 ** (np.arange(G) - 64)).astype(np.float32))[None, :]
            assert got["count"][0] == (keys >= np.sort(keys.ravel())[::-1][want - 1]).sum()
    ones = oracle.salient_select(np.ones((64, 128), np.float16), 128, np.ones(128, np.float32), 30000)
    assert ones["count"][0] == 64 * 128 and ones["thresh"][0] == np.float32(1.0)   # all keys tie: everything is in
    W = ws.weights(40, 128, 5, "normal").numpy()
    s = np.linspace(0.5, 2.0, 128).astype(np.float32)
    none = oracle.salient_select(W, 128, s, 0)
    assert np.isinf(none["thresh"]).all() and (none["count"] == 0).all() and not none["mask"].any()
    every = oracle.salient_select(W, 128, s, 1_000_000)
    assert (every["count"] == 40 * 128).all() and (np.unpackbits(every["mask"]).sum() == 40 * 128)
    tiny = oracle.salient_select(W, 128, s, 100)                                # 0.01 % of 5120 = 0 weights
    assert (tiny["count"] == 0).all()


def test_planted_salient_weights_are_found(oracle):
    R, C, G = 64, 256, 128
    rng = np.random.default_rng(3)
    W = (rng.standard_normal((R, C)) * 0.01).astype(np.float16)
    s = np.ones(C, np.float32)
    s[130] = 400.0                                   # hot channel: scale 20
    rows = rng.choice(R, 9, replace=False)
    W[rows, 130] = 0.5                               # 9 weights with key 10, everything else below 0.06 * 20
    W[5, 7] = -3.0                                   # one big weight on an ordinary channel of unit 0
    n_p = 9
    rate = (n_p * 1_000_000 + R * G - 1) // (R * G)
    assert rate * R * G // 1_000_000 == n_p
    got = oracle.salient_select(W, G, s, rate)
    mask = unpack_mask(got["mask"], C)
    assert got["count"][1] == 9 and set(np.flatnonzero(mask[:, 130])) == set(rows) and mask[:, 128:].sum() == 9
    assert got["thresh"][1] == np.float32(10.0)
    assert mask[5, 7] and got["thresh"][0] <= np.float32(3.0)


def test_power_of_two_invariance_and_monotone_rate(oracle):
    R, C, G = 48, 256, 64
    W = ws.weights(R, C, 11, "student_t").numpy()
    s = (np.random.default_rng(4).random(C).astype(np.float32) + 0.1)
    base = oracle.salient_select(W, G, s, 30000)
    scaled_s = oracle.salient_select(W, G, s * np.float32(4.0), 30000)       # a_j doubles exactly
    assert (scaled_s["mask"] == base["mask"]).all() and (scaled_s["thresh"] == base["thresh"] * np.float32(2)).all()
    scaled_w = oracle.salient_select((W.astype(np.float32) * 2).astype(np.float16), G, s, 30000)
    assert (scaled_w["mask"] == base["mask"]).all()
    more = oracle.salient_select(W, G, s, 60000)
    assert ((base["mask"] & ~more["mask"]) == 0).all() and (more["thresh"] <= base["thresh"]).all()


def test_eq6_with_protected_weights(oracle):
    rows = []
    for line in open(os.path.join(GOLDEN, "eq6_protected.txt")):
        t = line.split()
        if t and t[0].isdigit():
            rows.append((int(t[0]), int(t[2]), int(t[3]), int(t[4])))
    assert len(rows) >= 10
    for a, n, n_p, want in rows:
        R, G = (n // 128, 128) if n % 128 == 0 else (n // 8, 8)
        # G = 8 is not a chunk width of the library; the accounting only needs n = R * G
        got = oracle.effective_bits_protected(np.array([a], np.uint8), np.array([n_p]), R, G, 0, 0)
        assert got["unit_centibits"][0] == want and got["total_centibits"] == want
    # with no protected weights it is the plain accounting, overhead included
    acts = np.arange(7, dtype=np.uint8)
    plain = oracle.effective_bits(acts, 96, 128)
    prot = oracle.effective_bits_protected(acts, np.zeros(7, np.int64), 96, 128)
    assert (plain["unit_centibits"] == prot["unit_centibits"]).all() and plain["total_centibits"] == prot["total_centibits"]
    # 8-bit units cost the same whatever is protected; the average is sum B_i / sum n_i
    a8 = oracle.effective_bits_protected(np.array([1, 1], np.uint8), np.array([0, 500]), 96, 128, 0, 0)
    assert a8["unit_centibits"][0] == a8["unit_centibits"][1]
    mix = oracle.effective_bits_protected(np.array([4, 6], np.uint8), np.array([369, 369]), 96, 128, 0, 0)
    n = 96 * 128
    assert mix["total_centibits"] == 200 * (n - 369) + 800 * 369 + 100 * (n - 369) + 800 * 369
    with pytest.raises(ValueError):
        oracle.effective_bits_protected(np.array([4], np.uint8), np.array([n + 1]), 96, 128)


# ------------------------------------------------------------------ fits with the protected weights left out
def test_protected_fit_reduces_to_the_plain_fit(oracle):
    R, C, G = 24, 256, 128
    W = ws.weights(R, C, 21, "normal").numpy()
    s = (np.random.default_rng(6).random(C).astype(np.float32) + 0.2)
    grid = ws.clip_grid(20)
    plain = oracle.fit_eval(W, G, s, grid)
    nothing = oracle.fit_eval(W, G, s, grid, thresh=np.full(C // G, np.inf, np.float32))
    for k in plain:
        assert (plain[k].view(np.uint32 if plain[k].dtype == np.float32 else plain[k].dtype) ==
                nothing[k].view(np.uint32 if nothing[k].dtype == np.float32 else nothing[k].dtype)).all()
    # a column whose every weight is protected: the same as the plain fit of the matrix with that column
    # zeroed and its activation weight zero (the masking is per weight, so this is the case the plain call
    # can express)
    W2 = W.copy()
    W2[:, 40] = np.float16(0.75)                       # far above everything else in unit 0
    sel = oracle.salient_select(W2, G, s, R * 1_000_000 // (R * G))     # n_p = R weights per unit
    mask = np.unpackbits(sel["mask"], axis=1, bitorder="little").astype(bool)
    assert mask[:, 40].all() and mask[:, :G].sum() == R
    prot = oracle.fit_eval(W2, G, s, grid, thresh=sel["thresh"], units=(0, 1))
    W3, s3 = W2.copy(), s.copy()
    W3[:, 40] = 0
    s3[40] = 0
    want = oracle.fit_eval(W3, G, s3, grid, units=(0, 1))
    assert (prot["clip_idx"][:, 0] == want["clip_idx"][:, 0]).all()
    assert (prot["group_err"][:, 0].view(np.uint32) == want["group_err"][:, 0].view(np.uint32)).all()
    assert prot["energy"][0] == want["energy"][0] and (prot["err"][0] == want["err"][0]).all()
    # protecting the outlier column is the point of the method: the low-bit errors of the unit drop
    unprot = oracle.fit_eval(W2, G, s, grid, units=(0, 1))
    assert (prot["err"][0, 1:4] < 0.5 * unprot["err"][0, 1:4]).all()
    # everything protected: nothing is left to fit
    allp = oracle.fit_eval(W, G, s, grid, thresh=np.zeros(C // G, np.float32))
    assert not allp["err"].any() and not allp["energy"].any()


# ------------------------------------------------------------------ unit saliency and the fallback rule
def test_unit_saliency_closed_forms(oracle):
    R, G = 30, 32
    W = np.full((R, 2 * G), 0.5, np.float16)
    W[:, G:] = -0.25
    s = np.full(2 * G, 4.0, np.float32)
    s[G:] = 9.0
    assert (oracle.unit_saliency(W, G, s) == np.array([1.0, 0.75], np.float32)).all()     # 2 * 0.5, 3 * 0.25
    rng = np.random.default_rng(9)
    W = (rng.standard_normal((R, 4 * G)) * 0.02).astype(np.float16)
    s = (rng.random(4 * G) + 0.1).astype(np.float32)
    want = (np.abs(W.astype(np.float64)) * np.sqrt(s)[None, :].astype(np.float64)).reshape(R, 4, G).mean((0, 2))
    assert np.allclose(oracle.unit_saliency(W, G, s), want, rtol=1e-6)
    hot = s.copy()
    hot[G:2 * G] *= 4                                   # activation scale of unit 1 doubles
    got = oracle.unit_saliency(W, G, hot)
    assert np.allclose(got[1], 2 * want[1], rtol=1e-6) and np.allclose(got[[0, 2, 3]], want[[0, 2, 3]], rtol=1e-6)


def test_fallback_rule(oracle):
    #            8     4     3     2    1.58   1
    err = np.array([[0.0, 0.1, 0.2, 0.4, 0.6, 0.8],
                    [0.0, 0.1, 0.2, 0.4, 0.6, 0.8],
                    [0.3, 0.3, 0.3, 0.3, 0.3, 0.3],
                    [0.0, 0.0, 0.0, 0.0, 0.0, 0.0]], np.float32)
    energy = np.array([1.0, 2.0, 1.0, 0.0], np.float32)
    acts = np.array([6, 6, 4, 5], np.uint8)
    out, n = oracle.fallback(err, energy, acts, 0.25)
    # unit 0: 1-bit 0.8 > 0.25 -> 1.58 (0.6) -> 2 (0.4) -> 3 (0.2) passes; unit 1: limit 0.5: 1-bit 0.8, 1.58 0.6 fail, 2-bit 0.4 passes;
    # unit 2: every quantised action fails -> skip; unit 3: zero energy, zero error: 0 > 0 is false, stays
    assert out.tolist() == [3, 4, 0, 5] and n == 3
    same, n0 = oracle.fallback(err, energy, acts, np.inf)
    assert (same == acts).all() and n0 == 0
    strict, _ = oracle.fallback(err, energy, acts, 0.0)
    assert strict.tolist() == [1, 1, 0, 5]              # 8-bit has zero error in units 0 and 1
    # monotone in theta: a larger tolerance never asks for more precision
    rng = np.random.default_rng(10)
    e = np.sort(rng.random((50, 6)).astype(np.float32), axis=1)
    en = np.ones(50, np.float32)
    a = rng.integers(0, 7, 50).astype(np.uint8)
    lo, _ = oracle.fallback(e, en, a, 0.2)
    hi, _ = oracle.fallback(e, en, a, 0.6)
    assert (hi >= lo).all() and (lo <= a).all()


# ------------------------------------------------------------------ applying a plan with protected weights
def test_apply_plan_protected(oracle):
    R, C, G = 20, 1024, 128
    rng = np.random.default_rng(13)
    W = (rng.standard_normal((R, C)) * 0.02).astype(np.float16)          # no planted outlier columns here
    s = (rng.random(C).astype(np.float32) + 0.2)
    grid = ws.clip_grid(20)
    acts = np.array([0, 1, 2, 3, 4, 5, 6, 4], np.uint8)
    plain = oracle.apply_plan(W, G, s, grid, acts)
    nothing = oracle.apply_plan(W, G, s, grid, acts, thresh=np.full(C // G, np.inf, np.float32))
    for k in ("codes", "scales", "zeros", "wq"):
        assert (plain[k] == nothing[k]).all(), k
    assert nothing["prot_q"].size == 0 and not nothing["prot_offsets"].any()

    # a hot column in every unit, fully protected (n_p = R weights per unit)
    W2 = W.copy()
    hot = [u * G + 17 for u in range(C // G)]
    vals = np.linspace(0.3, 0.9, R).astype(np.float16) * np.where(np.arange(R) % 2 == 0, 1, -1).astype(np.float16)
    for c in hot:
        W2[:, c] = vals
    sel = oracle.salient_select(W2, G, s, (R * 1_000_000 + R * G - 1) // (R * G))      # n_p = R weights per unit
    mask = np.unpackbits(sel["mask"], axis=1, bitorder="little").astype(bool)
    assert all(mask[:, c].all() for c in hot) and mask.sum() == R * (C // G)
    got = oracle.apply_plan(W2, G, s, grid, acts, thresh=sel["thresh"])
    # everything but the protected column: the plain plan on the matrix with that column zero and unweighted
    W3, s3 = W2.copy(), s.copy()
    for u, c in enumerate(hot):
        if acts[u] != 0:
            W3[:, c] = 0
            s3[c] = 0
    want = oracle.apply_plan(W3, G, s3, grid, acts)
    assert (got["codes"] == want["codes"]).all() and (got["scales"] == want["scales"]).all() and (got["zeros"] == want["zeros"]).all()
    others = np.ones(C, bool)
    others[hot] = False
    assert (got["wq"][:, others] == want["wq"][:, others]).all()
    # the protected column: one INT8 grid per unit, restated in float64
    offs = got["prot_offsets"]
    assert offs[0] == 0 and (np.diff(offs) == np.where(acts != 0, R, 0)).all()       # a skipped unit protects nothing
    for u, c in enumerate(hot):
        col = W2[:, c].astype(np.float64)
        if acts[u] == 0:
            assert (got["wq"][:, c] == W2[:, c].view(np.uint16)).all() and got["prot_scale"][u] == 0
            continue
        sigma = np.float64(np.float16(np.float32(np.abs(col).max()) / np.float32(127.0)))
        assert got["prot_scale"][u] == np.float16(sigma).view(np.uint16)
        q = np.clip(np.rint(col / sigma), -127, 127)
        assert (got["prot_q"][offs[u]:offs[u + 1]] == q.astype(np.int8)).all()          # row order
        assert (got["wq"][:, c] == (q * sigma).astype(np.float16).view(np.uint16)).all()
        assert (np.abs(q * sigma - col) <= 0.5 * sigma * (1 + 1e-3)).all()
    # 8-bit round trip of the side grid: the largest protected magnitude is reproduced to within half a step
    assert np.abs(got["prot_q"]).max() == 127
