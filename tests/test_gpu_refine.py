"""GPU parity of the step-size refinement against the CPU oracle.  Scales (fp16) and group errors (a
fixed sequence of binary32 operations) are compared bit for bit; unit sums within 1e-4 relative."""
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


def inputs(oracle, R, C, seed, K=20, kind="student_t"):
    W = ws.weights(R, C, seed, kind)
    X = ws.activations(64, C, seed + 1)
    s = oracle.act_stats(X.numpy())
    grid = ws.clip_grid(K)
    return W, s, grid


def both(wq, ctx, oracle, W, G, s, grid, T, lr, clip_idx=None):
    Wd, sd, gd = W.cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda()
    if clip_idx is None:
        fit = wq.windq_fit_eval(ctx, Wd, G, sd, gd, want_group_err=True)
        clip_idx_d = fit["clip_idx"]
        clip_idx = clip_idx_d.cpu().numpy()
    else:
        fit = None
        clip_idx_d = torch.from_numpy(clip_idx).cuda()
    got = wq.windq_fit_refine(ctx, Wd, G, sd, gd, clip_idx_d, T, lr, want_group_err=True)
    torch.cuda.synchronize()
    want = oracle.fit_refine(W.numpy(), G, s, grid, clip_idx, T=T, lr=lr)
    return got, want, fit


def compare(got, want):
    gs = got["scale"].cpu().numpy().view(np.uint16)
    assert np.array_equal(gs, want["scale"].view(np.uint16)), "scales"
    ge = got["group_err"].cpu().numpy()
    assert np.array_equal(ge.view(np.uint32), want["group_err"].view(np.uint32)), "group errors"
    np.testing.assert_allclose(got["err"].cpu().numpy(), want["err"], rtol=1e-4, atol=1e-6)


@pytest.mark.parametrize("R,C,G", [(37, 256, 32), (70, 256, 64), (45, 512, 128), (19, 512, 256), (9, 1024, 512)])
@pytest.mark.parametrize("T,lr", [(10, 0.01), (3, 0.05)])
def test_refine_matches_oracle(wq, ctx, oracle, R, C, G, T, lr):
    W, s, grid = inputs(oracle, R, C, 300 + G)
    got, want, _ = both(wq, ctx, oracle, W, G, s, grid, T, lr)
    compare(got, want)


def test_no_steps_returns_the_clip_grid_fit(wq, ctx, oracle):
    W, s, grid = inputs(oracle, 50, 512, 41)
    got, want, fit = both(wq, ctx, oracle, W, 128, s, grid, 0, 0.01)
    compare(got, want)
    assert torch.equal(got["group_err"], fit["group_err"][:4])


def test_refined_errors_never_exceed_the_clip_grid_errors(wq, ctx, oracle):
    W, s, grid = inputs(oracle, 200, 1024, 42)
    got, want, fit = both(wq, ctx, oracle, W, 128, s, grid, 10, 0.02)
    compare(got, want)
    assert (got["group_err"] <= fit["group_err"][:4]).all()
    assert (got["err"].sum(0) < fit["err"][:, :4].sum(0)).all()


def test_maximum_steps_and_large_learning_rate(wq, ctx, oracle):
    """32 steps at lr = 0.5 drives many groups to a non-positive step size: the early stop must agree."""
    W, s, grid = inputs(oracle, 40, 256, 43)
    got, want, _ = both(wq, ctx, oracle, W, 64, s, grid, 32, 0.5)
    compare(got, want)
    got, want, _ = both(wq, ctx, oracle, W, 64, s, grid, 5, 1.0)
    compare(got, want)


def test_degenerate_groups(wq, ctx, oracle):
    """All-zero groups, constant groups, one outlier, zero statistics, clip indices beyond the grid."""
    R, C, G = 24, 512, 128
    W, s, grid = inputs(oracle, R, C, 44)
    W[0:4] = 0
    W[4:8] = 0.125
    W[8:12] = 0
    W[8:12, ::128] = 3.0
    W[12:16] = -W[12:16].abs()
    s = s.copy()
    s[128:256] = 0.0
    got, want, _ = both(wq, ctx, oracle, W, G, s, grid, 10, 0.02)
    compare(got, want)
    idx = np.full((4, C // G, R), 200, np.uint8)
    got, want, _ = both(wq, ctx, oracle, W, G, s, grid, 4, 0.02, clip_idx=idx)
    compare(got, want)


def test_strided_matrix_and_ragged_rows(wq, ctx, oracle):
    W, s, grid = inputs(oracle, 33, 768, 45)
    Wd = W.cuda()
    view = Wd[:, 128:640]                                      # ldw = 768, C = 512
    sd, gd = torch.from_numpy(s[128:640].copy()).cuda(), torch.from_numpy(grid).cuda()
    fit = wq.windq_fit_eval(ctx, view, 64, sd, gd)
    got = wq.windq_fit_refine(ctx, view, 64, sd, gd, fit["clip_idx"], 6, 0.03, want_group_err=True)
    want = oracle.fit_refine(W.numpy()[:, 128:640], 64, s[128:640].copy(), grid, fit["clip_idx"].cpu().numpy(), T=6, lr=0.03)
    compare(got, want)


def test_full_size_matrix_sampled_units(wq, ctx, oracle):
    """One 4096 x 4096 matrix in the launch configuration the library uses for it; the oracle checks
    every row of a few units."""
    R, C, G = 4096, 4096, 128
    W, s, grid = inputs(oracle, R, C, 46)
    Wd, sd, gd = W.cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda()
    fit = wq.windq_fit_eval(ctx, Wd, G, sd, gd)
    got = wq.windq_fit_refine(ctx, Wd, G, sd, gd, fit["clip_idx"], 10, 0.01, want_group_err=True)
    torch.cuda.synchronize()
    units = [0, 13, 31]
    cols = np.concatenate([np.arange(u * G, (u + 1) * G) for u in units])
    want = oracle.fit_refine(W.numpy()[:, cols], G, s[cols], grid, fit["clip_idx"][:, units].cpu().numpy(), T=10, lr=0.01)
    sub = dict(scale=got["scale"][:, units], group_err=got["group_err"][:, units], err=got["err"][units])
    compare(sub, want)


def test_argument_checks(wq, ctx):
    W = torch.zeros((8, 128), dtype=torch.float16, device="cuda")
    s = torch.ones(128, device="cuda")
    grid = torch.ones(4, device="cuda")
    idx = torch.zeros((4, 1, 8), dtype=torch.uint8, device="cuda")
    with pytest.raises(Exception):
        wq.windq_fit_refine(ctx, W, 128, s, grid, idx, 33, 0.01)
    with pytest.raises(Exception):
        wq.windq_fit_refine(ctx, W, 128, s, grid, idx, 10, -0.1)
    with pytest.raises(Exception):
        wq.windq_fit_refine(ctx, W, 128, s, grid, idx[:, :, :4], 10, 0.01)
    out = wq.windq_fit_refine(ctx, W, 128, s, grid, idx, 10, 0.01)
    assert (out["err"] == 0).all()


@pytest.mark.parametrize("R,C,G", [(37, 256, 32), (45, 512, 128), (9, 1024, 512)])
def test_plan_applied_with_refined_scales(wq, ctx, oracle, R, C, G):
    """Codes, scales, zero points and fake-quantised weights of a mixed plan that uses the refined scales."""
    W, s, grid = inputs(oracle, R, C, 500 + G)
    Wd, sd, gd = W.cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda()
    U = C // G
    fit = wq.windq_fit_eval(ctx, Wd, G, sd, gd)
    ref = wq.windq_fit_refine(ctx, Wd, G, sd, gd, fit["clip_idx"], 10, 0.03)
    actions = (np.arange(U) % 7).astype(np.uint8)
    ad = torch.from_numpy(actions).cuda()
    eb = wq.windq_effective_bits(ctx, ad, R, G)
    codes = torch.zeros(2 * R * C + 16 * U, dtype=torch.uint8, device="cuda")
    got = wq.windq_apply_plan(ctx, Wd, G, sd, gd, ad, eb["code_offsets"], codes, fit["clip_idx"], scale_in=ref["scale"])
    torch.cuda.synchronize()
    want = oracle.apply_plan(W.numpy(), G, s, grid, actions, fit["clip_idx"].cpu().numpy(), scale_in=ref["scale"].cpu().numpy())
    n = int(want["code_offsets"][U])
    assert np.array_equal(got["codes"][:n].cpu().numpy(), want["codes"])
    assert np.array_equal(got["scales"].cpu().numpy().view(np.uint16), want["scales"])
    assert np.array_equal(got["zeros"].cpu().numpy().view(np.uint16), want["zeros"])
    assert np.array_equal(got["wq"].cpu().numpy().view(np.uint16), want["wq"])
    # the plain call is untouched by the new argument
    plain = wq.windq_apply_plan(ctx, Wd, G, sd, gd, ad, eb["code_offsets"], codes.clone(), fit["clip_idx"])
    want_plain = oracle.apply_plan(W.numpy(), G, s, grid, actions, fit["clip_idx"].cpu().numpy())
    assert np.array_equal(plain["wq"].cpu().numpy().view(np.uint16), want_plain["wq"])


@pytest.mark.parametrize("R,C,G", [(37, 256, 32), (45, 512, 128), (9, 1024, 512), (300, 256, 64)])
def test_protected_refinement_and_packing(wq, ctx, oracle, R, C, G):
    """Salient weights at 3 % taken out of the groups: refined scales and errors, then a mixed plan packed with
    those scales and the INT8 side storage, all against the oracle bit for bit."""
    W, s, grid = inputs(oracle, R, C, 600 + G)
    Wd, sd, gd = W.cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda()
    U = C // G
    sel = wq.windq_salient_select(ctx, Wd, G, sd, 30000)
    fit = wq.windq_fit_eval(ctx, Wd, G, sd, gd, thresh=sel["thresh"])
    got = wq.windq_fit_refine(ctx, Wd, G, sd, gd, fit["clip_idx"], 10, 0.03, want_group_err=True, thresh=sel["thresh"])
    torch.cuda.synchronize()
    thresh = sel["thresh"].cpu().numpy()
    clip_idx = fit["clip_idx"].cpu().numpy()
    want = oracle.fit_refine(W.numpy(), G, s, grid, clip_idx, T=10, lr=0.03, thresh=thresh)
    compare(got, want)
    actions = ((np.arange(U) + 1) % 7).astype(np.uint8)
    ad = torch.from_numpy(actions).cuda()
    eb = wq.windq_effective_bits(ctx, ad, R, G)
    codes = torch.zeros(2 * R * C + 16 * U, dtype=torch.uint8, device="cuda")
    prot_q = torch.zeros(R * C, dtype=torch.int8, device="cuda")
    plan = wq.windq_apply_plan_protected(ctx, Wd, G, sd, gd, ad, eb["code_offsets"], codes, sel["thresh"], prot_q,
                                         fit["clip_idx"], scale_in=got["scale"])
    torch.cuda.synchronize()
    ref = oracle.apply_plan(W.numpy(), G, s, grid, actions, clip_idx, thresh=thresh, scale_in=want["scale"])
    n = int(ref["code_offsets"][U])
    assert np.array_equal(plan["codes"][:n].cpu().numpy(), ref["codes"])
    assert np.array_equal(plan["scales"].cpu().numpy().view(np.uint16), ref["scales"])
    assert np.array_equal(plan["zeros"].cpu().numpy().view(np.uint16), ref["zeros"])
    assert np.array_equal(plan["wq"].cpu().numpy().view(np.uint16), ref["wq"])
    assert np.array_equal(plan["prot_offsets"].cpu().numpy(), ref["prot_offsets"])
    assert np.array_equal(plan["prot_scale"].cpu().numpy().view(np.uint16), ref["prot_scale"])
    assert np.array_equal(plan["prot_q"][:ref["prot_q"].size].cpu().numpy(), ref["prot_q"])


def test_protected_refinement_with_infinite_thresholds_is_the_plain_one(wq, ctx, oracle):
    W, s, grid = inputs(oracle, 64, 512, 47)
    Wd, sd, gd = W.cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda()
    fit = wq.windq_fit_eval(ctx, Wd, 128, sd, gd)
    a = wq.windq_fit_refine(ctx, Wd, 128, sd, gd, fit["clip_idx"], 10, 0.02, want_group_err=True)
    inf = torch.full((4,), float("inf"), device="cuda")
    b = wq.windq_fit_refine(ctx, Wd, 128, sd, gd, fit["clip_idx"], 10, 0.02, want_group_err=True, thresh=inf)
    assert torch.equal(a["scale"].view(torch.int16), b["scale"].view(torch.int16))
    assert torch.equal(a["group_err"].view(torch.int32), b["group_err"].view(torch.int32))
