"""Pins for the oracle's step-size refinement (CPU only): a trace worked by hand, the warm start equal
to the clip-grid fit, the properties of keeping the best iterate, the first Adam step in closed form,
and the early stop."""
import os

import numpy as np
import pytest

import windq_synth as ws

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "step_size_refinement.txt")


def test_trace_worked_by_hand(oracle):
    cfg, steps = {}, []
    for line in open(GOLDEN):
        f = line.split("#")[0].split()
        if not f:
            continue
        if f[0] == "step":
            steps.append(f[1:])
        else:
            cfg[f[0]] = f[1:]
    w = np.array([float(x) for x in cfg["weights"]], np.float32)
    sc, lo, gr = oracle.refine_trace(w, np.ones_like(w), int(cfg["bits"][0]), float(cfg["scale0"][0]), float(cfg["zero"][0]),
                                     len(steps) - 1, float(cfg["lr"][0]))
    assert len(sc) == len(steps)
    for t, (_, scale, loss, g) in enumerate(steps):
        assert sc[t] == np.float32(float(scale)), t
        if loss != "-":
            assert lo[t] == pytest.approx(float(loss), rel=2e-6)
            assert gr[t] == pytest.approx(float(g), rel=2e-6)


def case(R, C, seed):
    W = ws.weights(R, C, seed, "student_t").numpy()
    X = ws.activations(64, C, seed + 1).numpy()
    return W, X


@pytest.mark.parametrize("G", [32, 128])
def test_no_steps_is_the_clip_grid_fit(oracle, G):
    W, X = case(24, 256, 11)
    s = oracle.act_stats(X)
    grid = ws.clip_grid(20)
    fit = oracle.fit_eval(W, G, s, grid)
    ref = oracle.fit_refine(W, G, s, grid, fit["clip_idx"], T=0, lr=0.01)
    assert np.array_equal(ref["group_err"], fit["group_err"][:4])
    assert np.allclose(ref["err"], fit["err"][:, :4], rtol=1e-6)
    plan = oracle.apply_plan(W, G, s, grid, np.full(256 // G, 2, np.uint8), fit["clip_idx"])   # all 4 bit
    assert np.array_equal(ref["scale"][1].view(np.uint16), plan["scales"].view(np.uint16))


def test_best_iterate_properties(oracle):
    W, X = case(16, 256, 21)
    s = oracle.act_stats(X)
    grid = ws.clip_grid(20)
    fit = oracle.fit_eval(W, 64, s, grid)
    prev = fit["group_err"][:4]
    improved = 0
    for T in (1, 3, 10):
        ref = oracle.fit_refine(W, 64, s, grid, fit["clip_idx"], T=T, lr=0.02)
        # the trajectory of T steps is a prefix of a longer one, so the best loss can only fall
        assert (ref["group_err"] <= prev).all()
        improved += int((ref["group_err"] < prev).sum())
        prev = ref["group_err"]
    assert improved > 0
    # the returned scale reproduces the returned error
    bits = [8, 4, 3, 2]
    for bi, u, r in [(0, 0, 0), (1, 2, 5), (2, 3, 15), (3, 1, 7)]:
        w = W[r, u * 64:(u + 1) * 64].astype(np.float32)
        su = s[u * 64:(u + 1) * 64]
        # zero point of the warm start, from the plan the oracle itself packs
        plan = oracle.apply_plan(W, 64, s, grid, np.full(4, bi + 1, np.uint8), fit["clip_idx"])
        zf = float(plan["zeros"].view(np.float16)[u, r])
        scs, los, _ = oracle.refine_trace(w, su, bits[bi], float(ref["scale"][bi, u, r]), zf, 0, 0.0)
        assert los[0] == ref["group_err"][bi, u, r]


def test_first_adam_step_is_one_learning_rate(oracle):
    """After one step m-hat = g and v-hat = g^2, so the step is lr * Delta_0 * sign(g) whatever |g| is."""
    rng = np.random.default_rng(3)
    for trial in range(20):
        w = rng.standard_normal(32).astype(np.float16).astype(np.float32)
        s = (rng.random(32) * 10.0 ** rng.integers(-2, 3)).astype(np.float32)
        scale0 = float(np.float16((w.max() - w.min()) / 15))
        zf = float(np.clip(np.rint(-w.min() / scale0), 0, 15))
        sc, lo, gr = oracle.refine_trace(w, s, 4, scale0, zf, 1, 0.05)
        assert gr[0] != 0
        want = scale0 * (1 - 0.05 * np.sign(gr[0]))
        assert abs(float(sc[1]) - want) <= 2.0 ** -10 * want       # fp16 spacing is at most 2^-10 relative


def test_in_range_weights_only_shrink_the_step(oracle):
    """With nothing clipped every term (s d) psi = s Delta (rne(x) - x)^2 is non-negative."""
    rng = np.random.default_rng(4)
    w = (rng.random(64) * 14 + 0.2).astype(np.float16).astype(np.float32)     # inside (0, 15) * scale 1
    _, _, gr = oracle.refine_trace(w, np.ones(64, np.float32), 4, 1.0, 0.0, 0, 0.0)
    assert gr[0] > 0
    x = w.astype(np.float64)
    assert gr[0] == pytest.approx(((np.rint(x) - x) ** 2).sum(), rel=1e-5)


def test_stops_when_the_step_size_leaves_the_positive_range(oracle):
    w = (np.arange(32) % 4 + 0.4).astype(np.float32)              # in range, off the grid: g > 0
    sc, lo, gr = oracle.refine_trace(w, np.ones(32, np.float32), 2, 1.0, 0.0, 5, 1.0)
    assert gr[0] > 0
    assert len(sc) == 1                                            # Delta_1 = 1 - 1 * 1 rounds to a non-positive fp16
    sc, _, _ = oracle.refine_trace(w, np.ones(32, np.float32), 2, 1.0, 0.0, 5, 0.1)
    assert len(sc) == 6 and (np.diff(sc[:2]) < 0).all()


def test_refined_plan_reproduces_the_refined_errors(oracle):
    """Packing with the refined scales: the 8-bit codes, zero points and scales of the plan, decoded here,
    give back the group errors the refinement reported."""
    W, X = case(16, 256, 31)
    s = oracle.act_stats(X)
    grid = ws.clip_grid(20)
    fit = oracle.fit_eval(W, 64, s, grid)
    ref = oracle.fit_refine(W, 64, s, grid, fit["clip_idx"], T=10, lr=0.02)
    plan = oracle.apply_plan(W, 64, s, grid, np.full(4, 1, np.uint8), fit["clip_idx"], scale_in=ref["scale"])
    assert np.array_equal(plan["scales"], ref["scale"][0].view(np.uint16))
    offs = plan["code_offsets"]
    for u in range(4):
        q = plan["codes"][offs[u]:offs[u] + 16 * 64].reshape(16, 64).astype(np.float64)
        z = plan["zeros"].view(np.float16)[u].astype(np.float64)[:, None]
        sc = plan["scales"].view(np.float16)[u].astype(np.float64)[:, None]
        d = (q - z) * sc - W[:, u * 64:(u + 1) * 64].astype(np.float64)
        e = (s[u * 64:(u + 1) * 64].astype(np.float64)[None, :] * d * d).sum(1)
        np.testing.assert_allclose(e, ref["group_err"][0, u], rtol=1e-5)


def test_protected_refinement_reduces_to_its_parts(oracle):
    """With the salient weights taken out: no steps give the protected fit; thresholds of +infinity give the
    plain refinement; the packed 8-bit plan decodes to the refined errors over the unprotected weights."""
    W, X = case(16, 256, 51)
    s = oracle.act_stats(X)
    grid = ws.clip_grid(20)
    sel = oracle.salient_select(W, 64, s, 30000)
    fitp = oracle.fit_eval(W, 64, s, grid, thresh=sel["thresh"])
    r0 = oracle.fit_refine(W, 64, s, grid, fitp["clip_idx"], T=0, thresh=sel["thresh"])
    assert np.array_equal(r0["group_err"], fitp["group_err"][:4])
    fit = oracle.fit_eval(W, 64, s, grid)
    a = oracle.fit_refine(W, 64, s, grid, fit["clip_idx"], T=10, lr=0.02)
    b = oracle.fit_refine(W, 64, s, grid, fit["clip_idx"], T=10, lr=0.02, thresh=np.full(4, np.inf, np.float32))
    assert np.array_equal(a["scale"].view(np.uint16), b["scale"].view(np.uint16))
    assert np.array_equal(a["group_err"], b["group_err"])
    r = oracle.fit_refine(W, 64, s, grid, fitp["clip_idx"], T=10, lr=0.02, thresh=sel["thresh"])
    assert (r["group_err"] <= fitp["group_err"][:4]).all()
    plan = oracle.apply_plan(W, 64, s, grid, np.full(4, 1, np.uint8), fitp["clip_idx"], thresh=sel["thresh"], scale_in=r["scale"])
    assert plan["prot_q"].size == int(sel["count"].sum())
    mask = np.unpackbits(sel["mask"], axis=1, bitorder="little")[:, :256].astype(bool)
    offs = plan["code_offsets"]
    for u in range(4):
        q = plan["codes"][offs[u]:offs[u] + 16 * 64].reshape(16, 64).astype(np.float64)
        z = plan["zeros"].view(np.float16)[u].astype(np.float64)[:, None]
        sc = plan["scales"].view(np.float16)[u].astype(np.float64)[:, None]
        keep = ~mask[:, u * 64:(u + 1) * 64]
        d = ((q - z) * sc - W[:, u * 64:(u + 1) * 64].astype(np.float64)) * keep
        e = (s[u * 64:(u + 1) * 64].astype(np.float64)[None, :] * d * d).sum(1)
        np.testing.assert_allclose(e, r["group_err"][0, u], rtol=1e-5, atol=1e-12)
