"""GPU parity of the searched 1.58-bit fit and of plan application with its thresholds, through the C ABI.

Threshold indices, fp16 scales, group errors, packed bytes and fake-quantised weights are compared with the CPU
oracle bit for bit; unit sums within 1e-4 relative + 1e-6 absolute.
"""
import numpy as np
import pytest
import torch

import windq_synth as ws

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-4, 1e-6


@pytest.fixture(scope="module")
def wq():
    import paper_2605_26660_b200 as wq
    return wq


@pytest.fixture(scope="module")
def ctx(wq):
    c = wq.windq_create(0)
    yield c
    wq.windq_destroy(c)


def close(g, o):
    g, o = np.asarray(g, np.float64), np.asarray(o, np.float64)
    return np.abs(g - o) <= RTOL * np.abs(o) + ATOL


def u16(t):
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def check_search(got, want):
    assert np.array_equal(got["thr_idx"].cpu().numpy(), want["thr_idx"])
    assert np.array_equal(u16(got["alpha"]), want["alpha"].view(np.uint16))
    assert np.array_equal(got["group_err"].cpu().numpy().view(np.uint32), want["group_err"].view(np.uint32))
    assert close(got["err"].cpu().numpy(), want["err"]).all()


GRID = np.linspace(0.3, 1.5, 13).astype(np.float32)


@pytest.mark.parametrize("G,R,C,Kt", [(128, 70, 512, 13), (64, 37, 256, 13), (32, 33, 128, 13), (256, 19, 1024, 13),
                                      (512, 9, 1024, 13), (128, 8, 256, 1), (64, 40, 128, 64), (128, 1, 128, 3)])
def test_ternary_search_small(wq, ctx, oracle, G, R, C, Kt):
    W = ws.weights(R, C, 900 + G + Kt, "student_t")
    s = oracle.act_stats(ws.activations(96, C, 901 + G).numpy())
    grid = np.linspace(0.2, 2.5, Kt).astype(np.float32) if Kt > 1 else np.array([0.7], np.float32)
    want = oracle.fit_ternary_search(W.numpy(), G, s, grid, threads=8)
    got = wq.windq_fit_ternary_search(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(),
                                      want_group_err=True)
    torch.cuda.synchronize()
    check_search(got, want)


def test_ternary_search_degenerate_inputs(wq, ctx, oracle):
    G, R = 128, 24
    W = ws.weights(R, 5 * G, 9, "normal")
    W[:, :G] = 0                                   # all-zero unit
    W[:, G:2 * G] = 0.37                           # constant unit: no |w| exceeds a threshold at or above the mean
    W[0, 2 * G:3 * G] = -0.0
    W[1, 2 * G:3 * G] = 6.0e-8                     # fp16 subnormals
    s = np.ones(5 * G, np.float32)
    s[3 * G:4 * G] = 0                             # no activation weight at all
    s[4 * G:4 * G + 100] = 0                       # little activation weight: some supports carry none
    grid = np.array([0.05, 0.5, 0.7, 1.0, 1.5, 4.0, 40.0], np.float32)      # the last ones empty every support
    want = oracle.fit_ternary_search(W.numpy(), G, s, grid)
    got = wq.windq_fit_ternary_search(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(),
                                      want_group_err=True)
    torch.cuda.synchronize()
    check_search(got, want)


def test_one_ratio_gives_the_plain_fit(wq, ctx):
    W = ws.weights(300, 1024, 77, "student_t").cuda()
    s = torch.rand(1024, device="cuda") + 0.1
    plain = wq.windq_fit_eval(ctx, W, 128, s, torch.from_numpy(ws.clip_grid(4)).cuda(), want_group_err=True)
    got = wq.windq_fit_ternary_search(ctx, W, 128, s, torch.tensor([0.7], device="cuda"), want_group_err=True)
    torch.cuda.synchronize()
    assert torch.equal(got["group_err"].view(torch.int32), plain["group_err"][4].view(torch.int32))
    assert bool((got["thr_idx"] == 0).all())


def test_protected_ternary_search(wq, ctx, oracle):
    R, C, G = 120, 512, 128
    W = ws.weights(R, C, 55, "student_t")
    s = oracle.act_stats(ws.activations(96, C, 56).numpy())
    sel = oracle.salient_select(W.numpy(), G, s, 30000, want_mask=False)
    Wd, sd, gd = W.cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(GRID).cuda()
    want = oracle.fit_ternary_search(W.numpy(), G, s, GRID, thresh=sel["thresh"], threads=4)
    got = wq.windq_fit_ternary_search(ctx, Wd, G, sd, gd, thresh=torch.from_numpy(sel["thresh"]).cuda(), want_group_err=True)
    torch.cuda.synchronize()
    check_search(got, want)
    inf = torch.full((C // G,), float("inf"), device="cuda")
    a = wq.windq_fit_ternary_search(ctx, Wd, G, sd, gd, thresh=inf, want_group_err=True)
    b = wq.windq_fit_ternary_search(ctx, Wd, G, sd, gd, want_group_err=True)
    torch.cuda.synchronize()
    for k in ("thr_idx", "alpha", "group_err", "err"):
        assert torch.equal(a[k].view(torch.uint8), b[k].view(torch.uint8)), k


@pytest.mark.parametrize("G,R", [(128, 70), (64, 133), (32, 200), (256, 19), (512, 67), (128, 3)])
def test_apply_plan_searched_all_actions(wq, ctx, oracle, G, R):
    C = 8 * G
    W = ws.weights(R, C, 950 + G + R, "student_t")
    s = oracle.act_stats(ws.activations(96, C, 951 + G).numpy())
    grid = ws.clip_grid(20)
    acts = np.array([5, 1, 5, 3, 4, 5, 6, 0], np.uint8)
    fit = oracle.fit_eval(W.numpy(), G, s, grid, threads=8, want_group_err=False)
    search = oracle.fit_ternary_search(W.numpy(), G, s, GRID, threads=8)
    want = oracle.apply_plan_searched(W.numpy(), G, s, grid, acts, fit["clip_idx"], GRID, search["thr_idx"])
    a_d = torch.from_numpy(acts).cuda()
    eb = wq.windq_effective_bits(ctx, a_d, R, G)
    n = int(eb["code_offsets"][-1].item())
    assert n == want["codes"].size
    codes = torch.full((n,), 0xEE, dtype=torch.uint8, device="cuda")
    g_search = wq.windq_fit_ternary_search(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(GRID).cuda())
    got = wq.windq_apply_plan_searched(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(), a_d,
                                       eb["code_offsets"], codes, torch.from_numpy(fit["clip_idx"]).cuda(),
                                       torch.from_numpy(GRID).cuda(), g_search["thr_idx"])
    torch.cuda.synchronize()
    assert np.array_equal(codes.cpu().numpy(), want["codes"])
    assert np.array_equal(u16(got["scales"]), want["scales"]) and np.array_equal(u16(got["zeros"]), want["zeros"])
    assert np.array_equal(u16(got["wq"]), want["wq"])
    # the stored scale of a 1.58-bit group is the scale the search reported
    for u in np.flatnonzero(acts == 5):
        assert np.array_equal(u16(got["scales"][u]), u16(g_search["alpha"][u]))


def test_ternary_search_on_a_full_size_matrix(wq, ctx, oracle):
    """gate_proj of the 7B-shaped model (11008 x 4096, Student-t) at chunk width 128: sampled units against the
    oracle, and the searched error never above the plain 1.58-bit error when 0.7 is on the grid."""
    spec = ws.CONFIGS["cfg3_llama7b_model"]
    m = spec.block_matrices()[4]
    W = ws.block_weight(spec, 0, 0, m, device="cuda")
    s = wq.windq_act_stats(ctx, ws.block_input(spec, 0, 0, m.x_id, device="cuda"))
    grid = np.array([0.4, 0.5, 0.6, 0.7, 0.8, 0.9, 1.0, 1.1, 1.2], np.float32)
    got = wq.windq_fit_ternary_search(ctx, W, 128, s, torch.from_numpy(grid).cuda(), want_group_err=True)
    plain = wq.windq_fit_eval(ctx, W, 128, s, torch.from_numpy(ws.clip_grid(20)).cuda(), want_group_err=True)
    torch.cuda.synchronize()
    assert bool((got["group_err"] <= plain["group_err"][4]).all())
    s_h = s.cpu().numpy()
    for u in (0, 13, 31):
        want = oracle.fit_ternary_search(W[:, u * 128:(u + 1) * 128].cpu().numpy(), 128, s_h[u * 128:(u + 1) * 128], grid, threads=1)
        assert np.array_equal(got["thr_idx"][u].cpu().numpy(), want["thr_idx"][0])
        assert np.array_equal(u16(got["alpha"][u]), want["alpha"][0].view(np.uint16))
        assert close(got["err"][u].item(), want["err"][0])
    gain = float(got["err"].double().sum() / plain["err"][:, 4].double().sum())
    print("\n[ternary search, 11008 x 4096, 9 ratios] error relative to the 0.7 rule: %.4f" % gain)
    assert gain <= 1.0


def test_ternary_search_argument_errors(wq, ctx):
    W = torch.zeros((16, 256), dtype=torch.float16, device="cuda")
    s = torch.ones(256, device="cuda")
    with pytest.raises(wq.WindqError) as e:
        wq.windq_fit_ternary_search(ctx, W, 128, s, torch.ones(65, device="cuda"))
    assert e.value.status == 4
    with pytest.raises(wq.WindqError) as e:
        wq.windq_fit_ternary_search(ctx, W, 100, s, torch.ones(3, device="cuda"))
    assert e.value.status == 4
    out = wq.windq_fit_ternary_search(ctx, W, 128, s, torch.ones(3, device="cuda"))
    assert float(out["err"].abs().sum()) == 0.0
