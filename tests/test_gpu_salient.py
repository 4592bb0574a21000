"""GPU parity of salient-weight selection and Eq. 6 with protected weights against the CPU oracle.
Thresholds, counts, mask bytes and bit totals are integers or bit patterns: all compared exactly."""
import numpy as np
import pytest
import torch

import windq_synth as ws

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def wq():
    import paper_2605_26660_b200 as wq
    return wq


@pytest.fixture(scope="module")
def ctx(wq):
    c = wq.windq_create(0)
    yield c
    wq.windq_destroy(c)


def run(wq, ctx, W, G, s, rate):
    out = wq.windq_salient_select(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), rate)
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


@pytest.mark.parametrize("R,C,G,rate", [(300, 512, 128, 30000), (97, 256, 64, 20000), (64, 128, 32, 123456),
                                        (1000, 1024, 256, 30000), (33, 1024, 512, 500000), (50, 256, 128, 1000000),
                                        (4096, 512, 128, 30000), (3, 128, 128, 30000)])
def test_salient_select(wq, ctx, oracle, R, C, G, rate):
    W = ws.weights(R, C, 700 + R, "student_t")
    W[::3, ::5] = 0
    X = ws.activations(64, C, 701)
    s = oracle.act_stats(X.numpy())
    want = oracle.salient_select(W.numpy(), G, s, rate)
    got = run(wq, ctx, W, G, s, rate)
    assert (got["thresh"].view(np.uint32) == want["thresh"].view(np.uint32)).all()
    assert (got["count"] == want["count"]).all()
    assert (got["mask"] == want["mask"]).all()


def test_salient_select_ties_zero_rate_and_strides(wq, ctx, oracle):
    G, R = 128, 40
    W = torch.full((R, 3 * G), 0.25, dtype=torch.float16)       # unit 0: every key equal
    W[:, G:2 * G] = 0                                           # unit 1: every key zero
    W[:, 2 * G:] = ws.weights(R, G, 3, "normal")
    s = np.ones(3 * G, np.float32)
    s[2 * G:2 * G + 5] = 0                                      # channels that never fire: key 0
    want = oracle.salient_select(W.numpy(), G, s, 30000)
    got = run(wq, ctx, W, G, s, 30000)
    assert (got["count"] == want["count"]).all() and got["count"][0] == R * G and got["count"][1] == R * G
    assert (got["thresh"].view(np.uint32) == want["thresh"].view(np.uint32)).all() and (got["mask"] == want["mask"]).all()
    none = run(wq, ctx, W, G, s, 0)
    assert np.isinf(none["thresh"]).all() and (none["count"] == 0).all() and not none["mask"].any()
    wide = torch.zeros((R, 4 * G), dtype=torch.float16, device="cuda")
    wide[:, G:] = W.cuda()
    out = wq.windq_salient_select(ctx, wide[:, G:], G, torch.from_numpy(s).cuda(), 30000)
    assert (out["mask"].cpu().numpy() == want["mask"]).all()
    with pytest.raises(wq.WindqError) as e:
        wq.windq_salient_select(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), 1000001)
    assert e.value.status == 4


def test_effective_bits_protected(wq, ctx, oracle):
    rng = np.random.default_rng(5)
    for U, R, G in ((86, 4096, 128), (1, 7, 32), (3000, 50, 64)):
        acts = rng.integers(0, 7, U).astype(np.uint8)
        n_p = rng.integers(0, R * G // 20 + 1, U).astype(np.int64)
        for sb, zb in ((16, 16), (0, 0)):
            want = oracle.effective_bits_protected(acts, n_p, R, G, sb, zb)
            got = wq.windq_effective_bits_protected(ctx, torch.from_numpy(acts).cuda(), torch.from_numpy(n_p).cuda(), R, G, sb, zb)
            assert (got["unit_centibits"].cpu().numpy() == want["unit_centibits"]).all()
            assert int(got["total_centibits"].item()) == want["total_centibits"]
    bad = wq.windq_effective_bits_protected(ctx, torch.tensor([4, 9], dtype=torch.uint8, device="cuda"),
                                            torch.tensor([0, 0], dtype=torch.int64, device="cuda"), 8, 128)
    assert int(bad["total_centibits"].item()) == -1


def test_full_size_selection_feeds_eq6(wq, ctx, oracle):
    """11008 x 4096 Student-t matrix of the 7B-shaped sweep at the paper's 3 % rate: sampled units against
    the oracle, counts into Eq. 6, and the average bits of an all-2-bit plan with protection."""
    spec = ws.CONFIGS["cfg3_llama7b_model"]
    m = spec.block_matrices()[4]
    W = ws.block_weight(spec, 0, 0, m, device="cuda")
    X = ws.block_input(spec, 0, 0, m.x_id, device="cuda")
    s = wq.windq_act_stats(ctx, X)
    G, U = 128, m.C // 128
    out = wq.windq_salient_select(ctx, W, G, s, 30000)
    n_p = 30000 * m.R * G // 1_000_000
    count = out["count"].cpu().numpy()
    assert (count >= n_p).all() and (count <= n_p + 64).all()      # ties at the threshold are rare on this data
    bits_set = np.unpackbits(out["mask"].cpu().numpy(), axis=1, bitorder="little").reshape(m.R, U, G).sum((0, 2))
    assert (bits_set == count).all()
    s_h = s.cpu().numpy()
    for u in (0, 17, U - 1):
        want = oracle.salient_select(W[:, u * G:(u + 1) * G].cpu().numpy(), G, s_h[u * G:(u + 1) * G], 30000)
        assert out["thresh"][u].cpu().numpy().view(np.uint32) == want["thresh"].view(np.uint32)[0]
        assert count[u] == want["count"][0]
        assert (out["mask"][:, u * G // 8:(u + 1) * G // 8].cpu().numpy() == want["mask"]).all()
    acts = torch.full((U,), 4, dtype=torch.uint8, device="cuda")
    eb = wq.windq_effective_bits_protected(ctx, acts, out["count"], m.R, G, 0, 0)
    avg = int(eb["total_centibits"].item()) / (100.0 * m.R * m.C)
    assert abs(avg - (2 * 0.97 + 8 * 0.03)) < 1e-3                  # 2.18 bits: the paper's accounting at 3 %


# ------------------------------------------------------------------ fits with the protected weights left out
def fit(wq, ctx, W, G, s, grid, thresh=None):
    out = wq.windq_fit_eval(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(), want_group_err=True,
                            thresh=None if thresh is None else torch.from_numpy(thresh).cuda())
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in out.items()}


def same_fit(got, want):
    assert (got["clip_idx"] == want["clip_idx"]).all()
    assert (got["group_err"].view(np.uint32) == want["group_err"].view(np.uint32)).all()
    for k in ("err", "energy"):
        assert (np.abs(got[k] - want[k]) <= 1e-4 * np.abs(want[k]) + 1e-6).all(), k


@pytest.mark.parametrize("G,R,C,rate", [(128, 70, 512, 30000), (64, 37, 256, 30000), (32, 33, 128, 100000),
                                        (256, 19, 1024, 20000), (512, 9, 1024, 30000)])
def test_fit_eval_protected(wq, ctx, oracle, G, R, C, rate):
    W = ws.weights(R, C, 800 + G, "student_t")
    X = ws.activations(64, C, 801)
    s = oracle.act_stats(X.numpy())
    grid = ws.clip_grid(20)
    sel = oracle.salient_select(W.numpy(), G, s, rate)
    want = oracle.fit_eval(W.numpy(), G, s, grid, threads=8, thresh=sel["thresh"])
    same_fit(fit(wq, ctx, W, G, s, grid, sel["thresh"]), want)
    # thresholds from the GPU selection are the same bits, so the two calls chain on the device
    dev = wq.windq_salient_select(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), rate, want_mask=False)
    out = wq.windq_fit_eval(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(), thresh=dev["thresh"])
    assert (out["clip_idx"].cpu().numpy() == want["clip_idx"]).all()


def test_fit_eval_protected_limits(wq, ctx, oracle):
    G, R, C = 128, 40, 256
    W = ws.weights(R, C, 810, "normal")
    s = (np.random.default_rng(8).random(C).astype(np.float32) + 0.2)
    grid = ws.clip_grid(20)
    plain = fit(wq, ctx, W, G, s, grid)
    nothing = fit(wq, ctx, W, G, s, grid, np.full(C // G, np.inf, np.float32))
    for k in plain:
        assert (plain[k] == nothing[k]).all() or k in ("err", "energy")
    assert (plain["group_err"].view(np.uint32) == nothing["group_err"].view(np.uint32)).all()
    everything = fit(wq, ctx, W, G, s, grid, np.zeros(C // G, np.float32))
    assert not everything["err"].any() and not everything["energy"].any() and not everything["group_err"].any()
    same_fit(everything, oracle.fit_eval(W.numpy(), G, s, grid, thresh=np.zeros(C // G, np.float32)))


# ------------------------------------------------------------------ unit saliency and the fallback rule
@pytest.mark.parametrize("R,C,G", [(300, 512, 128), (4096, 1024, 256), (37, 128, 32), (11008, 512, 64), (5, 1024, 512)])
def test_unit_saliency(wq, ctx, oracle, R, C, G):
    W = ws.weights(R, C, 900 + R, "student_t")
    s = oracle.act_stats(ws.activations(64, C, 901).numpy())
    want = oracle.unit_saliency(W.numpy(), G, s)
    got = wq.windq_unit_saliency(ctx, W.cuda(), G, torch.from_numpy(s).cuda()).cpu().numpy()
    assert (np.abs(got - want) <= 1e-5 * np.abs(want) + 1e-9).all()


def test_fallback(wq, ctx, oracle):
    G, R, C = 128, 200, 2048
    W = ws.weights(R, C, 910, "student_t")
    s = oracle.act_stats(ws.activations(64, C, 911).numpy())
    grid = torch.from_numpy(ws.clip_grid(20)).cuda()
    fitd = wq.windq_fit_eval(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), grid)
    err, energy = fitd["err"].cpu().numpy(), fitd["energy"].cpu().numpy()
    rng = np.random.default_rng(12)
    acts = rng.integers(0, 7, C // G).astype(np.uint8)
    for theta in (0.0, 0.01, 0.1, 0.4, np.inf):
        want, n = oracle.fallback(err, energy, acts, theta)
        got = wq.windq_fallback(ctx, fitd["err"], fitd["energy"], torch.from_numpy(acts).cuda(), theta)
        assert (got["actions"].cpu().numpy() == want).all() and int(got["n_changed"].item()) == n
    odd = acts.copy()
    odd[::3] = [7, 200, 255, 9, 7, 8][:len(odd[::3])]          # not action codes: copied as they are
    want, n = oracle.fallback(err, energy, odd, 0.05)
    got = wq.windq_fallback(ctx, fitd["err"], fitd["energy"], torch.from_numpy(odd).cuda(), 0.05)
    assert (got["actions"].cpu().numpy() == want).all() and int(got["n_changed"].item()) == n
    assert (want[::3] == odd[::3]).all()
    with pytest.raises(wq.WindqError):
        wq.windq_fallback(ctx, fitd["err"], fitd["energy"], torch.from_numpy(acts).cuda(), -1.0)


# ------------------------------------------------------------------ applying a plan with protected weights
def u16(t):
    return t.cpu().view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("G,R,rate", [(128, 70, 30000), (64, 133, 30000), (32, 200, 50000), (256, 19, 20000), (512, 67, 30000),
                                      (128, 3, 100000)])
def test_apply_plan_protected(wq, ctx, oracle, G, R, rate):
    C = 8 * G
    W = ws.weights(R, C, 1000 + G + R, "student_t")
    s = oracle.act_stats(ws.activations(64, C, 1001).numpy())
    grid = ws.clip_grid(20)
    acts = np.array([0, 1, 2, 3, 4, 5, 6, 5], np.uint8)
    sel = oracle.salient_select(W.numpy(), G, s, rate)
    fitp = oracle.fit_eval(W.numpy(), G, s, grid, threads=8, want_group_err=False, thresh=sel["thresh"])
    want = oracle.apply_plan(W.numpy(), G, s, grid, acts, fitp["clip_idx"], thresh=sel["thresh"])
    Wd, s_d, grid_d, a_d = W.cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(), torch.from_numpy(acts).cuda()
    th_d = torch.from_numpy(sel["thresh"]).cuda()
    eb = wq.windq_effective_bits(ctx, a_d, R, G)
    n_codes = int(eb["code_offsets"][-1].item())
    cap = int(sel["count"].sum())
    for clip_idx in (torch.from_numpy(fitp["clip_idx"]).cuda(), None):
        codes = torch.full((n_codes,), 0xAB, dtype=torch.uint8, device="cuda")
        prot_q = torch.full((cap + 64,), 99, dtype=torch.int8, device="cuda")
        got = wq.windq_apply_plan_protected(ctx, Wd, G, s_d, grid_d, a_d, eb["code_offsets"], codes, th_d, prot_q, clip_idx)
        torch.cuda.synchronize()
        assert (codes.cpu().numpy() == want["codes"]).all()
        assert (u16(got["scales"]) == want["scales"]).all() and (u16(got["zeros"]) == want["zeros"]).all()
        assert (u16(got["wq"]) == want["wq"]).all()
        assert (u16(got["prot_scale"]) == want["prot_scale"]).all()
        assert (got["prot_offsets"].cpu().numpy() == want["prot_offsets"]).all()
        n = int(want["prot_offsets"][-1])
        assert (prot_q[:n].cpu().numpy() == want["prot_q"]).all() and bool((prot_q[n:] == 99).all())
    # too small a list: nothing beyond its end is touched, and the offsets still tell how many there are
    small = torch.full((max(n // 2, 1) + 32,), 99, dtype=torch.int8, device="cuda")
    got = wq.windq_apply_plan_protected(ctx, Wd, G, s_d, grid_d, a_d, eb["code_offsets"], codes, th_d, small[:max(n // 2, 1)])
    torch.cuda.synchronize()
    assert int(got["prot_offsets"][-1].item()) == n and bool((small[max(n // 2, 1):] == 99).all())


def test_apply_plan_protected_without_protection_is_the_plain_plan(wq, ctx):
    G, R, C = 128, 96, 1024
    W = ws.weights(R, C, 1100, "student_t").cuda()
    s = torch.rand(C, device="cuda") + 0.1
    grid = torch.from_numpy(ws.clip_grid(20)).cuda()
    acts = torch.tensor([4, 3, 5, 6, 1, 2, 0, 4], dtype=torch.uint8, device="cuda")
    fitd = wq.windq_fit_eval(ctx, W, G, s, grid)
    eb = wq.windq_effective_bits(ctx, acts, R, G)
    n_codes = int(eb["code_offsets"][-1].item())
    c1 = torch.empty(n_codes, dtype=torch.uint8, device="cuda")
    c2 = torch.empty(n_codes, dtype=torch.uint8, device="cuda")
    plain = wq.windq_apply_plan(ctx, W, G, s, grid, acts, eb["code_offsets"], c1, fitd["clip_idx"])
    inf = torch.full((C // G,), float("inf"), device="cuda")
    prot = wq.windq_apply_plan_protected(ctx, W, G, s, grid, acts, eb["code_offsets"], c2, inf,
                                         torch.empty(16, dtype=torch.int8, device="cuda"), fitd["clip_idx"])
    assert torch.equal(c1, c2)
    for k in ("scales", "zeros", "wq"):
        assert torch.equal(plain[k].view(torch.int16), prot[k].view(torch.int16))
    assert int(prot["prot_offsets"][-1].item()) == 0
