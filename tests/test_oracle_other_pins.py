"""Pins for the oracle's statistics, features, bit accounting and packing (CPU only)."""
import os

import numpy as np
import pytest

import windq_synth as ws

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ act_stats
def test_act_stats_closed_forms(oracle):
    T, C = 37, 24
    c = np.float16(1.5)
    assert (oracle.act_stats(np.full((T, C), c, np.float16)) == np.float32(2.25)).all()
    X = np.zeros((T, C), np.float16)
    X[5, 7] = 3.0
    s = oracle.act_stats(X)
    assert s[7] == np.float32(9.0 / T) and s.sum() == s[7]
    # two half batches average
    rng = np.random.default_rng(0)
    X = (rng.standard_normal((64, C)) * 3).astype(np.float16)
    full = oracle.act_stats(X).astype(np.float64)
    halves = 0.5 * (oracle.act_stats(X[:32]).astype(np.float64) + oracle.act_stats(X[32:]).astype(np.float64))
    assert np.allclose(full, halves, rtol=1e-6)
    assert np.allclose(full, (X.astype(np.float64) ** 2).mean(0), rtol=1e-6)
    # columns, not rows
    X = np.zeros((4, 6), np.float16)
    X[:, 2] = 2.0
    assert (oracle.act_stats(X) == np.array([0, 0, 4, 0, 0, 0], np.float32)).all()


# ------------------------------------------------------------------ unit_features (Table 1)
def test_unit_features_closed_forms(oracle):
    R, G = 50, 32
    s = np.arange(2 * G, dtype=np.float32)
    # unit 0: constant c ; unit 1: +-c alternating
    W = np.zeros((R, 2 * G), np.float16)
    W[:, :G] = 0.25
    W[:, G:] = np.where(np.arange(G) % 2 == 0, 0.5, -0.5)
    f = oracle.unit_features(W, G, s)
    assert np.allclose(f[0, :5], [0.25, 0.0, 0.25, 0.0, 1.0])       # every |w| > 0.5 * P99
    assert np.allclose(f[1, :5], [0.0, 0.5, 0.5, 0.0, 1.0])
    # calibration statistics of the unit's own channels: 0..31 and 32..63
    assert np.allclose(f[0, 5:], [15.5, np.sqrt((G * G - 1) / 12.0), 31.0])
    assert np.allclose(f[1, 5:], [47.5, np.sqrt((G * G - 1) / 12.0), 63.0])


def test_unit_features_p99_is_nearest_rank(oracle):
    # n = 200 distinct magnitudes 1..200 (scaled): k = ceil(0.99 * 200) = 198 -> P99 = 198,
    # threshold 99: outliers are 100..200 -> 101 of 200.  Interpolated percentiles would give 198.01.
    R, G = 25, 8
    mags = np.arange(1, 201, dtype=np.float64).reshape(R, G) / 256.0
    rng = np.random.default_rng(1)
    W = (mags * rng.choice([-1.0, 1.0], size=mags.shape)).astype(np.float16)
    W = W.reshape(-1)[rng.permutation(200)].reshape(R, G)
    f = oracle.unit_features(W, G, np.ones(G, np.float32))
    assert f[0, 4] == np.float32(101 / 200)
    assert f[0, 2] == pytest.approx(100.5 / 256.0, rel=1e-6)
    # n = 150: k = ceil(148.5) = 149 -> P99 = 149, threshold 74.5 -> 75..150 = 76 outliers
    W = (np.arange(1, 151, dtype=np.float64).reshape(25, 6) / 256.0)
    W = np.concatenate([W, W[:, :2]], axis=1)[:, :6]                 # keep n = 150, G = 6 is not needed:
    W2 = np.zeros((75, 8), np.float16)                                # use G = 8 with R = 75 -> n = 600
    vals = np.arange(1, 601, dtype=np.float64) / 1024.0
    W2[:] = vals.reshape(75, 8)
    f = oracle.unit_features(W2, 8, np.ones(8, np.float32))
    k = (99 * 600 + 99) // 100                                        # 594
    assert f[0, 4] == np.float32((600 - int(np.floor(k / 2))) / 600)  # |w| > 297/1024 -> 298..600


def test_unit_features_against_numpy(oracle):
    R, C, G = 96, 512, 128
    W = ws.weights(R, C, 41, dist="student_t").numpy()
    W[::7, ::3] = 0                                                   # planted exact zeros
    s = np.random.default_rng(2).lognormal(0, 1, C).astype(np.float32)
    f = oracle.unit_features(W, G, s)
    for u in range(C // G):
        w = W[:, u * G:(u + 1) * G].astype(np.float64).ravel()
        a = np.sort(np.abs(w))
        n = a.size
        p99 = a[int(np.ceil(0.99 * n)) - 1]
        want = [w.mean(), w.std(), np.abs(w).mean(), (np.abs(w) < 1e-6).mean(), (np.abs(w) > 0.5 * p99).mean()]
        su = s[u * G:(u + 1) * G].astype(np.float64)
        want += [su.mean(), su.std(), su.max()]
        assert np.allclose(f[u], want, rtol=1e-6, atol=1e-9)
        assert f[u, 3] * n >= (W[::7, u * G:(u + 1) * G:1][:, (np.arange(G) + u * G) % 3 == 0]).size


def test_outlier_fraction_of_half_normal(oracle):
    # |w| half-normal: 0.5 * P99 = 1.288 sigma -> P(|w| > 1.288 sigma) = 0.1977
    W = ws.weights(2048, 256, 43, outlier_frac=0.0).numpy()
    f = oracle.unit_features(W, 128, np.ones(256, np.float32))
    assert f[:, 4] == pytest.approx(0.1977, abs=0.003)
    assert f[:, 1] == pytest.approx(0.02, rel=0.01) and f[:, 2] == pytest.approx(0.02 * np.sqrt(2 / np.pi), rel=0.01)


# ------------------------------------------------------------------ effective bits (Eq. 6)
def _golden_rows():
    rows, units = [], None
    with open(os.path.join(GOLDEN, "eq6_effective_bits.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            t = line.split()
            if t[0] == "units":
                units = [int(x) for x in t[1:]]
            else:
                rows.append((int(t[0]), float(t[1]), int(t[2]), int(t[3])))
    return rows, units


def test_effective_bits_reduces_to_eq6_without_overhead(oracle):
    rows, units = _golden_rows()
    for action, nominal, n, centibits in rows:
        assert centibits == round(nominal * 100) * n                  # the fixture is Eq. 6 itself
        G = 128
        R = n // G
        out = oracle.effective_bits(np.array([action], np.uint8), R, G, 0, 0)
        assert out["total_centibits"] == centibits and out["unit_centibits"][0] == centibits
    layers, proj, hidden, chunk, n_units = units
    assert layers * proj * (hidden // chunk) == n_units


def test_effective_bits_average_and_overhead(oracle):
    # b_bar = sum B_i / sum n_i with 16 + 16 overhead bits per (row, chunk) group
    per_weight = {128: [16.0, 8.25, 4.25, 3.25, 2.25, 1.705, 1.125],
                  64: [16.0, 8.5, 4.5, 3.5, 2.5, 1.83, 1.25],
                  256: [16.0, 8.125, 4.125, 3.125, 2.125, 1.6425, 1.0625]}
    R = 40
    for G, costs in per_weight.items():
        for a, c in enumerate(costs):
            out = oracle.effective_bits(np.full(5, a, np.uint8), R, G)
            assert out["total_centibits"] / (100.0 * 5 * R * G) == pytest.approx(c, abs=1e-12)
        acts = np.arange(7, dtype=np.uint8)
        out = oracle.effective_bits(acts, R, G)
        assert out["total_centibits"] == out["unit_centibits"].sum()
        assert out["total_centibits"] / (100.0 * 7 * R * G) == pytest.approx(np.mean(costs), abs=1e-12)
    # mix reaching 1.58 at G = 128: x binary + (1 - x) ternary with 1.125 x + 1.705 (1 - x) = 1.58
    x = (1.705 - 1.58) / (1.705 - 1.125)
    assert 0.21 < x < 0.22


def test_code_offsets_and_packed_bytes(oracle):
    R, G = 24, 128
    acts = np.array([0, 1, 2, 3, 4, 5, 6, 5], np.uint8)
    out = oracle.effective_bits(acts, R, G)
    per_group = [256, 128, 64, 48, 32, 26, 16, 26]
    offs = [0]
    for b in per_group:
        offs.append(offs[-1] + (R * b + 15) // 16 * 16)
    assert out["code_offsets"].tolist() == offs
    n_scales, n_zeros = 7 * R, 4 * R
    assert out["total_packed_bytes"] == offs[-1] + 2 * (n_scales + n_zeros)
    # an odd row count leaves padding after the ternary block (26 R not a multiple of 16)
    out = oracle.effective_bits(np.array([5, 6], np.uint8), 3, 128)
    assert out["code_offsets"].tolist() == [0, 80, 128]


# ------------------------------------------------------------------ packing
def _weights_with_codes(q, bits, z, shift=-10):
    """Weights whose p = 1 fit has exactly the codes q (both 0 and qmax present in every row)."""
    w = (q.astype(np.float64) - z) * 2.0 ** shift
    w16 = w.astype(np.float16)
    assert (w16.astype(np.float64) == w).all()
    return w16


def _unpack(action, G, blob):
    """Independent unpacker (python integers), one row-group."""
    blob = [int(b) for b in blob]
    if action == 1:
        return blob[:G]
    if action == 5:
        out = []
        for b in blob:
            for _ in range(5):
                out.append(b % 3)
                b //= 3
        return out[:G]
    bits = {2: 4, 3: 3, 4: 2, 6: 1}[action]
    big = sum(b << (8 * i) for i, b in enumerate(blob))
    return [(big >> (bits * j)) & ((1 << bits) - 1) for j in range(G)]


def test_packing_hand_worked_bytes(oracle):
    G = 32
    one = np.array([1.0], np.float32)
    s = np.ones(G, np.float32)
    # 3-bit codes 0..7 repeated: elements at bits [3j, 3j+3) -> 0x88 0xC6 0xFA per 8 codes
    q = np.tile(np.arange(8), 4)[None, :]
    plan = oracle.apply_plan(_weights_with_codes(q, 3, 3), G, s, one, np.array([3], np.uint8))
    assert plan["codes"].tolist() == [0x88, 0xC6, 0xFA] * 4 + [0] * 4       # 12 bytes + pad to 16
    # 4-bit: low nibble first
    q = np.tile(np.array([0, 15, 1, 2, 3, 4, 10, 5]), 4)[None, :]
    plan = oracle.apply_plan(_weights_with_codes(q, 4, 7), G, s, one, np.array([2], np.uint8))
    assert plan["codes"].tolist() == [0xF0, 0x21, 0x43, 0x5A] * 4
    # 2-bit: element m of a byte at bits [2m, 2m+2)
    q = np.tile(np.array([0, 3, 1, 2]), 8)[None, :]
    plan = oracle.apply_plan(_weights_with_codes(q, 2, 1), G, s, one, np.array([4], np.uint8))
    assert plan["codes"].tolist() == [0b10011100] * 8 + [0] * 8
    # 8-bit: identity
    q = (np.arange(32) * 8 + 7)[None, :]
    q[0, 0] = 0
    plan = oracle.apply_plan(_weights_with_codes(q, 8, 100), G, s, one, np.array([1], np.uint8))
    assert plan["codes"].tolist() == q[0].tolist()
    # 1-bit: bit j%8 of byte j/8 is set unless w < 0
    w = np.where(np.arange(G) % 3 == 0, -0.5, 0.5).astype(np.float16)[None, :]
    plan = oracle.apply_plan(w, G, s, one, np.array([6], np.uint8))
    want = [sum(((8 * i + m) % 3 != 0) << m for m in range(8)) for i in range(4)]
    assert plan["codes"].tolist() == want + [0] * 12
    # ternary: trits (-,0,+) -> (0,1,2), five per byte in base 3; 32 elements -> 7 bytes, last holds 2
    t = np.tile(np.array([0, 1, 2, 2, 1]), 7)[:G]
    w = ((t - 1) * 0.5).astype(np.float16)[None, :]
    plan = oracle.apply_plan(w, G, s, one, np.array([5], np.uint8))
    full = 0 + 1 * 3 + 2 * 9 + 2 * 27 + 1 * 81
    assert plan["codes"].tolist() == [full] * 6 + [0 + 1 * 3] + [0] * 9
    assert plan["scales"].view(np.float16)[0, 0] == np.float16(0.5)
    # skip: the raw fp16 bytes
    plan = oracle.apply_plan(w, G, s, one, np.array([0], np.uint8))
    assert plan["codes"].tobytes() == w.tobytes()
    assert plan["scales"][0, 0] == 0 and plan["zeros"][0, 0] == 0 and (plan["wq"] == w.view(np.uint16)).all()


def test_pack_unpack_dequant_identity(oracle):
    R, C, G = 40, 1024, 128
    W = ws.weights(R, C, 51, dist="student_t").numpy()
    s = np.random.default_rng(3).lognormal(0, 1, C).astype(np.float32)
    grid = ws.clip_grid(20)
    acts = np.array([0, 1, 2, 3, 4, 5, 6, 4], np.uint8)
    fit = oracle.fit_eval(W, G, s, grid, threads=8)
    plan = oracle.apply_plan(W, G, s, grid, acts, fit["clip_idx"])
    again = oracle.apply_plan(W, G, s, grid, acts, None)              # re-search gives the same clip index
    for key in ("codes", "scales", "zeros", "wq"):
        assert (plan[key] == again[key]).all()
    offs = plan["code_offsets"]
    assert plan["codes"].size == offs[-1]
    per_group = [256, 128, 64, 48, 32, 26, 16]
    for u, a in enumerate(acts):
        a = int(a)
        blk = plan["codes"][offs[u]:offs[u + 1]]
        assert (blk[R * per_group[a]:] == 0).all()                    # padding
        sc = plan["scales"][u].view(np.float16).astype(np.float32)
        zp = plan["zeros"][u].view(np.float16).astype(np.float32)
        wq = plan["wq"][:, u * G:(u + 1) * G]
        if a == 0:
            assert blk.tobytes() == W[:, u * G:(u + 1) * G].tobytes()
            continue
        for r in range(R):
            q = np.array(_unpack(a, G, blk[r * per_group[a]:(r + 1) * per_group[a]]), np.float32)
            if a <= 4:
                assert q.max() <= 2 ** (8, 4, 3, 2)[a - 1] - 1
                deq = ((q - zp[r]) * sc[r]).astype(np.float16)
            elif a == 5:
                deq = ((q - 1) * sc[r]).astype(np.float16)
            else:
                deq = ((2 * q - 1) * sc[r]).astype(np.float16)
            assert (deq.view(np.uint16) == wq[r]).all()
        # stored parameters reproduce the scored error
        deq = wq.view(np.float16).astype(np.float64)
        e = (s[u * G:(u + 1) * G].astype(np.float64) * (deq - W[:, u * G:(u + 1) * G].astype(np.float64)) ** 2).sum()
        # fake-quantised weights are rounded to fp16 once more, so only approximately
        assert e == pytest.approx(fit["err"][u, a - 1], rel=2e-2)
