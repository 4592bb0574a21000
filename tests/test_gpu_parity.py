"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, on the same seeded inputs.

Bars (fixed in advance): clip indices, codes / packed bytes, fp16 scales / zero points, fake-quantised
weights, the counts behind sparsity / outlier_frac and all int64 totals are bit-exact; float outputs
agree within |g - o| <= 1e-4 |o| + 1e-6.  Group errors are compared bit-exactly as well, since both
sides define them as the same sequence of binary32 operations.
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


def guarded(shape, dtype, fill=0xAB):
    """An output tensor inside a larger buffer whose margins must stay untouched."""
    n = int(np.prod(shape))
    item = torch.empty(0, dtype=dtype).element_size()
    pad = 256 // item
    buf = torch.full((n + 2 * pad,), 0, dtype=dtype, device="cuda")
    buf.view(torch.uint8).fill_(fill)
    view = buf[pad:pad + n].view(*shape)

    def intact():
        raw = buf.view(torch.uint8)
        return bool((raw[:256] == fill).all()) and bool((raw[256 + n * item:] == fill).all())
    return view, intact


def make(R, C, seed, dist="student_t", T=96):
    W = ws.weights(R, C, seed, dist)
    X = ws.activations(T, C, seed + 7)
    return W, X


# ------------------------------------------------------------------ act_stats
@pytest.mark.parametrize("T,C", [(512, 4096), (77, 264), (1, 8), (300, 11008)])
def test_act_stats(wq, ctx, oracle, T, C):
    X = ws.activations(T, C, 100 + T)
    want = oracle.act_stats(X.numpy())
    out, intact = guarded((C,), torch.float32)
    wq.windq_act_stats(ctx, X.cuda(), out)
    torch.cuda.synchronize()
    assert intact()
    assert close(out.cpu().numpy(), want).all()


def test_act_stats_strided_rows(wq, ctx, oracle):
    X = ws.activations(64, 512, 5)
    big = torch.zeros((64, 768), dtype=torch.float16, device="cuda")
    big[:, :512] = X.cuda()
    got = wq.windq_act_stats(ctx, big[:, :512])
    assert close(got.cpu().numpy(), oracle.act_stats(X.numpy())).all()


def test_act_stats_batch(wq, ctx, oracle):
    """Several inputs of different shapes in one launch: the oracle's values, the bits of the separate calls,
    nothing written past an output, and the same again on a second call (the arrival
    counters are back at zero)."""
    shapes = [(300, 11008), (77, 264), (1, 8), (512, 4096), (65, 1000), (1100, 28672)]
    Xs = [ws.activations(T, C, 700 + j) for j, (T, C) in enumerate(shapes)]
    tiny = torch.randint(1, 1024, (70, 64), generator=torch.Generator().manual_seed(5), dtype=torch.int16)
    Xs.append((tiny | (tiny << 15)).view(torch.float16))      # subnormal fp16 values of both signs: nothing is flushed
    shapes.append((70, 64))
    Xd = [X.cuda() for X in Xs]
    wide = torch.zeros((65, 1280), dtype=torch.float16, device="cuda")     # a strided view as one of the jobs
    wide[:, :1000] = Xd[4]
    Xd[4] = wide[:, :1000]
    pairs = [guarded((C,), torch.float32) for _, C in shapes]
    for rep in range(2):
        for out, _ in pairs:
            out.fill_(-1.0)
        wq.windq_act_stats_batch(ctx, Xd, [out for out, _ in pairs])
        torch.cuda.synchronize()
        for (out, intact), X, Xg in zip(pairs, Xs, Xd):
            assert intact()
            assert close(out.cpu().numpy(), oracle.act_stats(X.numpy())).all()
            assert torch.equal(out, wq.windq_act_stats(ctx, Xg))
            assert close(wq.windq_act_stats_noalloc(ctx, Xg, torch.empty_like(out)).cpu().numpy(), oracle.act_stats(X.numpy())).all()
    # the subnormal input on its own terms (its statistics are far below the absolute tolerance above)
    assert np.allclose(pairs[-1][0].cpu().numpy(), oracle.act_stats(Xs[-1].numpy()), rtol=1e-5, atol=0.0)
    assert wq.windq_scratch_bytes_act_stats_batch(shapes) == sum(wq.windq_scratch_bytes_act_stats(T, C) for T, C in shapes)
    with pytest.raises(wq.WindqError):
        wq.windq_act_stats_batch(ctx, [Xd[0]] * 17)
    with pytest.raises(wq.WindqError):
        wq.windq_act_stats_batch(ctx, [Xd[0], torch.zeros((4, 12), dtype=torch.float16, device="cuda")])


# ------------------------------------------------------------------ unit_features
@pytest.mark.parametrize("R,C,G", [(300, 512, 128), (64, 256, 32), (1000, 1024, 512), (97, 256, 64), (4096, 512, 256)])
def test_unit_features(wq, ctx, oracle, R, C, G):
    W, X = make(R, C, 200 + G)
    W[::5, ::7] = 0
    s = oracle.act_stats(X.numpy())
    want = oracle.unit_features(W.numpy(), G, s)
    out, intact = guarded((C // G, 8), torch.float32)
    wq.windq_unit_features(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert intact()
    assert (got[:, 3:5] == want[:, 3:5]).all()          # exact counts -> identical ratios
    assert close(got, want).all()


# ------------------------------------------------------------------ fit_eval
def run_fit(wq, ctx, W, G, s, grid):
    R, C = W.shape
    U = C // G
    err, ok1 = guarded((U, 6), torch.float32)
    energy, ok2 = guarded((U,), torch.float32)
    clip_idx, ok3 = guarded((4, U, R), torch.uint8)
    group_err, ok4 = guarded((6, U, R), torch.float32)
    out = wq.windq_fit_eval(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(),
                            want_group_err=True, out=dict(err=err, energy=energy, clip_idx=clip_idx, group_err=group_err))
    torch.cuda.synchronize()
    assert ok1() and ok2() and ok3() and ok4()
    return {k: v.cpu().numpy() for k, v in out.items()}


def check_fit(got, want):
    mism = got["clip_idx"] != want["clip_idx"]
    assert (got["group_err"].view(np.uint32) == want["group_err"].view(np.uint32)).all()
    assert not mism.any()
    assert close(got["err"], want["err"]).all()
    assert close(got["energy"], want["energy"]).all()


@pytest.mark.parametrize("G,R,C,K", [(128, 70, 512, 20), (64, 37, 256, 20), (32, 33, 128, 20), (256, 19, 1024, 20),
                                     (512, 9, 1024, 20), (128, 8, 256, 7), (64, 40, 128, 64), (32, 64, 64, 40),
                                     (128, 1, 128, 1)])
def test_fit_eval_small(wq, ctx, oracle, G, R, C, K):
    W, X = make(R, C, 300 + G + K)
    s = oracle.act_stats(X.numpy())
    grid = ws.clip_grid(K)
    want = oracle.fit_eval(W.numpy(), G, s, grid, threads=8)
    check_fit(run_fit(wq, ctx, W, G, s, grid), want)


def test_fit_eval_degenerate_inputs(wq, ctx, oracle):
    G, R = 128, 24
    W = ws.weights(R, 4 * G, 9, "normal")
    W[:, :G] = 0                                   # all-zero unit
    W[:, G:2 * G] = 0.37                           # constant unit
    W[0, 2 * G:3 * G] = -0.0                       # negative zeros
    W[1, 2 * G:3 * G] = 6.0e-8                     # fp16 subnormals
    s = np.ones(4 * G, np.float32)
    s[3 * G:] = 0                                  # no activation weight at all
    grid = ws.clip_grid(20)
    want = oracle.fit_eval(W.numpy(), G, s, grid)
    check_fit(run_fit(wq, ctx, W, G, s, grid), want)


def test_fit_eval_config1_single_layer(wq, ctx, oracle):
    spec = ws.CONFIGS["cfg1_single_layer"]
    W = ws.weights(4096, 4096, ws.matrix_seed(0, 0, 0), "normal")
    X = ws.activations(spec.T, 4096, ws.matrix_seed(0, 0, 8))
    s = oracle.act_stats(X.numpy())
    grid = ws.clip_grid(20)
    out = wq.windq_fit_eval(ctx, W.cuda(), 128, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(), want_group_err=True)
    got = {k: v.cpu().numpy() for k, v in out.items()}
    # the oracle on every fourth unit (8 of 32 units, 4.2e6 weights)
    for u0 in range(0, 32, 4):
        want = oracle.fit_eval(W.numpy(), 128, s, grid, units=(u0, u0 + 1))
        assert (got["clip_idx"][:, u0] == want["clip_idx"][:, u0]).all()
        assert (got["group_err"][:, u0].view(np.uint32) == want["group_err"][:, u0].view(np.uint32)).all()
        assert close(got["err"][u0], want["err"][u0]).all() and close(got["energy"][u0], want["energy"][u0]).all()


@pytest.mark.parametrize("G", [32, 64, 128, 256, 512])
def test_eight_bit_search_skips_only_losers(wq, ctx, oracle, G):
    """The eight-bit clip search leaves out candidates whose error is bounded below by a single weight's term.  The
    kept index and error must be those of the full search, bit for bit, whatever the order of the grid (the search
    scans it backwards), with repeated ratios (the first of equal errors wins), with more candidates than one table
    holds, with statistics that vanish where the extremes sit (the bound is then zero and rules nothing out) and
    with an outlier that is free to clip (the best ratio is then the narrowest, met last)."""
    R, U = 37, 5
    rng = np.random.default_rng(40 + G)
    W = ws.weights(R, U * G, 41 + G, "student_t")
    W[:, :G] = 0                                                        # every candidate ties at zero error
    W[3, G:2 * G] = 0.25                                                # a constant row
    s = oracle.act_stats(ws.activations(96, U * G, 42 + G).numpy())
    out_col = 3 * G + int(rng.integers(0, G))
    W[:, out_col] = torch.from_numpy(rng.choice([-4.0, 4.0], R).astype(np.float16))   # outliers on a channel ...
    s[out_col] = 0                                                      # ... that no activation ever excites
    s[4 * G:] = 0
    s[4 * G + 5] = 1.0                                                  # one live channel in the last unit
    asc = ws.clip_grid(20)
    grids = {"ascending": asc, "descending": asc[::-1].copy(),
             "shuffled with repeats": rng.permutation(np.concatenate([asc, asc[5:9], asc[-1:]])).astype(np.float32),
             "one": asc[-1:].copy(), "sixty-four": rng.uniform(1.0 / 64, 1.0, 64).astype(np.float32)}
    for name, grid in grids.items():
        want = oracle.fit_eval(W.numpy(), G, s, grid)
        wq.windq_fit_work(ctx, reset=True)
        got = run_fit(wq, ctx, W, G, s, grid)
        evaluated, searched = wq.windq_fit_work(ctx)
        check_fit(got, want)
        assert 0 < evaluated <= searched, name
        assert searched % (4 * len(grid)) == 0, name
    # on weight-like data with the widest range last, most eight-bit candidates are ruled out
    Wl = ws.weights(256, 4 * G, 43 + G, "student_t")
    sl = oracle.act_stats(ws.activations(96, 4 * G, 44 + G).numpy())
    wq.windq_fit_work(ctx, reset=True)
    got = run_fit(wq, ctx, Wl, G, sl, asc)
    evaluated, searched = wq.windq_fit_work(ctx, reset=True)
    check_fit(got, oracle.fit_eval(Wl.numpy(), G, sl, asc, threads=8))
    assert evaluated < 0.95 * searched


def test_selfcheck_finds_no_mismatch(wq, ctx):
    """The fits take 1 / scale by the hardware approximation and one Newton step; for every fp16 value a scale can
    have that must be the IEEE quotient, which the oracle uses."""
    assert wq.windq_selfcheck(ctx) == 0


def test_unit_errors_without_group_errors(wq, ctx, oracle):
    """When no group errors are asked for, the 1.58- and 1-bit unit errors come from the sums of the fit instead of
    a term-by-term pass: tolerance outputs, checked here on ordinary and on degenerate inputs (zero units, constant
    units, statistics that vanish on part of a unit, statistics of very different sizes)."""
    G, R = 128, 40
    W = ws.weights(R, 6 * G, 29, "student_t")
    W[:, :G] = 0
    W[:, G:2 * G] = 0.37
    W[2, 2 * G:3 * G] = -0.0
    s = oracle.act_stats(ws.activations(64, 6 * G, 30).numpy())
    s[3 * G:4 * G] = 0
    s[4 * G:4 * G + 100] = 0
    s[5 * G] *= 1.0e4
    grid = ws.clip_grid(20)
    want = oracle.fit_eval(W.numpy(), G, s, grid, threads=4)
    got = wq.windq_fit_eval(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda())
    torch.cuda.synchronize()
    assert got["group_err"] is None
    assert (got["clip_idx"].cpu().numpy() == want["clip_idx"]).all()
    assert close(got["err"].cpu().numpy(), want["err"]).all()
    assert close(got["energy"].cpu().numpy(), want["energy"]).all()


def test_fit_eval_is_reproducible(wq, ctx):
    W = ws.weights(333, 1024, 77, "student_t").cuda()
    s = torch.rand(1024, device="cuda") + 0.1
    grid = torch.from_numpy(ws.clip_grid(20)).cuda()
    a = wq.windq_fit_eval(ctx, W, 128, s, grid, want_group_err=True)
    b = wq.windq_fit_eval(ctx, W, 128, s, grid, want_group_err=True)
    for k in a:
        assert torch.equal(a[k], b[k])


# ------------------------------------------------------------------ effective_bits
@pytest.mark.parametrize("U,R,G", [(32, 4096, 128), (1, 1, 32), (2500, 37, 64), (86, 4096, 512)])
def test_effective_bits(wq, ctx, oracle, U, R, G):
    rng = np.random.default_rng(U)
    acts = rng.integers(0, 7, U).astype(np.uint8)
    for sb, zb in ((16, 16), (0, 0), (32, 8)):
        want = oracle.effective_bits(acts, R, G, sb, zb)
        got = wq.windq_effective_bits(ctx, torch.from_numpy(acts).cuda(), R, G, sb, zb)
        assert (got["unit_centibits"].cpu().numpy() == want["unit_centibits"]).all()
        assert (got["code_offsets"].cpu().numpy() == want["code_offsets"]).all()
        assert int(got["total_centibits"].item()) == want["total_centibits"]
        assert int(got["total_packed_bytes"].item()) == want["total_packed_bytes"]


def test_effective_bits_flags_bad_action(wq, ctx):
    acts = torch.tensor([1, 2, 9, 3], dtype=torch.uint8, device="cuda")
    got = wq.windq_effective_bits(ctx, acts, 16, 128)
    assert int(got["total_centibits"].item()) == -1 and int(got["total_packed_bytes"].item()) == -1
    assert got["unit_centibits"].cpu().tolist()[2] == -1


# ------------------------------------------------------------------ apply_plan
def run_apply(wq, ctx, W, G, s, grid, acts, clip_idx):
    R, C = W.shape
    U = C // G
    a_d = torch.from_numpy(acts).cuda()
    eb = wq.windq_effective_bits(ctx, a_d, R, G)
    n_codes = int(eb["code_offsets"][-1].item())
    codes, ok1 = guarded((max(n_codes, 1),), torch.uint8)
    scales, ok2 = guarded((U, R), torch.float16)
    zeros, ok3 = guarded((U, R), torch.float16)
    wq_t, ok4 = guarded((R, C), torch.float16)
    out = wq.windq_apply_plan(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(), a_d,
                              eb["code_offsets"], codes, None if clip_idx is None else torch.from_numpy(clip_idx).cuda(),
                              out=dict(scales=scales, zeros=zeros, wq=wq_t))
    torch.cuda.synchronize()
    assert ok1() and ok2() and ok3() and ok4()
    return dict(codes=out["codes"][:n_codes].cpu().numpy(), scales=out["scales"].cpu().view(torch.int16).numpy().view(np.uint16),
                zeros=out["zeros"].cpu().view(torch.int16).numpy().view(np.uint16),
                wq=out["wq"].cpu().view(torch.int16).numpy().view(np.uint16))


@pytest.mark.parametrize("G,R", [(128, 70), (64, 133), (32, 200), (256, 19), (512, 67), (128, 3), (128, 64)])
def test_apply_plan_all_actions(wq, ctx, oracle, G, R):
    C = 8 * G
    W, X = make(R, C, 400 + G + R)
    s = oracle.act_stats(X.numpy())
    grid = ws.clip_grid(20)
    acts = np.array([0, 1, 2, 3, 4, 5, 6, 5], np.uint8)
    fit = oracle.fit_eval(W.numpy(), G, s, grid, threads=8, want_group_err=False)
    want = oracle.apply_plan(W.numpy(), G, s, grid, acts, fit["clip_idx"])
    for clip_idx in (fit["clip_idx"], None):
        got = run_apply(wq, ctx, W, G, s, grid, acts, clip_idx)
        for key in ("codes", "scales", "zeros", "wq"):
            assert got[key].shape == want[key].shape, key
            assert (got[key] == want[key]).all(), key


def test_apply_plan_uses_clip_idx_from_fit_eval(wq, ctx, oracle):
    G, R, C = 128, 96, 1024
    W, X = make(R, C, 500)
    s = oracle.act_stats(X.numpy())
    grid = ws.clip_grid(20)
    fit = wq.windq_fit_eval(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda())
    acts = np.array([4, 3, 2, 1, 4, 4, 3, 2], np.uint8)
    want = oracle.apply_plan(W.numpy(), G, s, grid, acts, None)
    got = run_apply(wq, ctx, W, G, s, grid, acts, fit["clip_idx"].cpu().numpy())
    for key in ("codes", "scales", "zeros", "wq"):
        assert (got[key] == want[key]).all(), key


def test_apply_plan_degenerate_inputs(wq, ctx, oracle):
    G, R = 128, 20
    W = ws.weights(R, 7 * G, 19, "normal")
    W[:, :3 * G] = 0
    W[3, 3 * G:4 * G] = -0.0
    s = np.ones(7 * G, np.float32)
    s[5 * G:] = 0
    grid = ws.clip_grid(20)
    for acts in (np.array([1, 5, 6, 4, 3, 5, 6], np.uint8), np.array([4, 6, 5, 2, 1, 6, 5], np.uint8)):
        want = oracle.apply_plan(W.numpy(), G, s, grid, acts, None)
        got = run_apply(wq, ctx, W, G, s, grid, acts, None)
        for key in ("codes", "scales", "zeros", "wq"):
            assert (got[key] == want[key]).all(), key


# ------------------------------------------------------------------ argument checks (no launch)
def test_argument_errors(wq, ctx):
    W = torch.zeros((16, 256), dtype=torch.float16, device="cuda")
    s = torch.ones(256, device="cuda")
    grid = torch.from_numpy(ws.clip_grid(20)).cuda()
    with pytest.raises(wq.WindqError) as e:
        wq.windq_fit_eval(ctx, W, 100, s, grid)
    assert e.value.status == 4 and "G = 100" in str(e.value)
    with pytest.raises(wq.WindqError) as e:
        wq.windq_fit_eval(ctx, W[:, :192], 128, s, grid)
    assert e.value.status == 2
    with pytest.raises(wq.WindqError) as e:
        wq.windq_fit_eval(ctx, W, 128, s, torch.ones(65, device="cuda"))
    assert e.value.status == 4
    with pytest.raises(wq.WindqError) as e:
        wq.windq_fit_eval(ctx, W[:, 4:132], 128, s, grid)          # 8-byte offset: misaligned
    assert e.value.status == 3
    with pytest.raises(wq.WindqError) as e:
        wq.windq_act_stats(ctx, torch.zeros((4, 12), dtype=torch.float16, device="cuda"))
    assert e.value.status in (2, 3)
    with pytest.raises(wq.WindqError) as e:
        wq.windq_effective_bits(ctx, torch.zeros(4, dtype=torch.uint8, device="cuda"), 16, 128, scale_bits=-1)
    assert e.value.status == 4
    # the context stays usable after errors
    out = wq.windq_fit_eval(ctx, W, 128, s, grid)
    assert float(out["err"].abs().sum()) == 0.0


# ------------------------------------------------------------------ layouts, limits, contexts
def test_strided_weight_matrix(wq, ctx, oracle):
    """W as a column block of a wider matrix (ldw > C): every call reads the same values as from a
    packed copy, and apply_plan writes only inside the block of the fake-quantised output."""
    G, R, C = 128, 50, 512
    W, X = make(R, C, 610)
    s = oracle.act_stats(X.numpy())
    grid = ws.clip_grid(20)
    wide = torch.full((R, C + 256), 7.0, dtype=torch.float16, device="cuda")
    wide[:, 128:128 + C] = W.cuda()
    view = wide[:, 128:128 + C]
    s_d, grid_d = torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda()
    want = oracle.fit_eval(W.numpy(), G, s, grid, threads=8)
    got = wq.windq_fit_eval(ctx, view, G, s_d, grid_d, want_group_err=True)
    check_fit({k: v.cpu().numpy() for k, v in got.items()}, want)
    assert close(wq.windq_unit_features(ctx, view, G, s_d).cpu().numpy(), oracle.unit_features(W.numpy(), G, s)).all()
    acts = np.array([3, 5, 6, 0], np.uint8)
    a_d = torch.from_numpy(acts).cuda()
    eb = wq.windq_effective_bits(ctx, a_d, R, G)
    codes = torch.empty(int(eb["code_offsets"][-1].item()), dtype=torch.uint8, device="cuda")
    wq_wide = torch.full_like(wide, -3.0)
    plan = wq.windq_apply_plan(ctx, view, G, s_d, grid_d, a_d, eb["code_offsets"], codes, got["clip_idx"],
                               out=dict(wq=wq_wide[:, 128:128 + C]))
    o = oracle.apply_plan(W.numpy(), G, s, grid, acts, want["clip_idx"])
    assert (codes.cpu().numpy() == o["codes"]).all()
    assert (plan["wq"].cpu().view(torch.int16).numpy().view(np.uint16) == o["wq"]).all()
    assert bool((wq_wide[:, :128] == -3.0).all()) and bool((wq_wide[:, 128 + C:] == -3.0).all())


def test_empty_inputs_are_refused(wq, ctx):
    grid = torch.from_numpy(ws.clip_grid(20)).cuda()
    s = torch.ones(256, device="cuda")
    empty = torch.zeros((0, 256), dtype=torch.float16, device="cuda")
    for call in (lambda: wq.windq_fit_eval(ctx, empty, 128, s, grid),
                 lambda: wq.windq_unit_features(ctx, empty, 128, s),
                 lambda: wq.windq_act_stats(ctx, empty),
                 lambda: wq.windq_effective_bits(ctx, torch.zeros(0, dtype=torch.uint8, device="cuda"), 16, 128)):
        with pytest.raises(wq.WindqError) as e:
            call()
        assert e.value.status in (1, 2)          # NULL (no storage) or SHAPE


def test_scratch_sizes_and_reserve(wq, oracle):
    c = wq.windq_create(0)
    try:
        R, C, G = 333, 1024, 64
        need = max(wq.windq_scratch_bytes_fit_eval(R, C, G), wq.windq_scratch_bytes_unit_features(R, C, G),
                   wq.windq_scratch_bytes_act_stats(512, C))
        assert need > 0 and wq.windq_scratch_bytes_fit_eval(R, C, 100) == 0
        wq.windq_reserve(c, need)
        W, X = make(R, C, 620)
        s = wq.windq_act_stats(c, X.cuda())
        assert close(s.cpu().numpy(), oracle.act_stats(X.numpy())).all()
        with pytest.raises(wq.WindqError):
            wq.windq_reserve(c, -1)
    finally:
        wq.windq_destroy(c)


def test_two_contexts_on_two_streams(wq, ctx):
    """Contexts own their scratch: calls through different contexts on different streams do not disturb
    each other."""
    other = wq.windq_create(0)
    try:
        W1 = ws.weights(400, 1024, 630, "student_t").cuda()
        W2 = ws.weights(300, 2048, 631, "student_t").cuda()
        s1, s2 = torch.rand(1024, device="cuda") + 0.1, torch.rand(2048, device="cuda") + 0.1
        grid = torch.from_numpy(ws.clip_grid(20)).cuda()
        ref1 = wq.windq_fit_eval(ctx, W1, 128, s1, grid)
        ref2 = wq.windq_fit_eval(ctx, W2, 64, s2, grid)
        f1 = wq.windq_unit_features(ctx, W1, 128, s1).clone()
        torch.cuda.synchronize()
        st1, st2 = torch.cuda.Stream(), torch.cuda.Stream()
        for _ in range(3):
            a = wq.windq_fit_eval(ctx, W1, 128, s1, grid, stream=st1)
            b = wq.windq_fit_eval(other, W2, 64, s2, grid, stream=st2)
            f = wq.windq_unit_features(other, W1, 128, s1, stream=st2)
        torch.cuda.synchronize()
        for k in ("err", "energy", "clip_idx"):
            assert torch.equal(a[k], ref1[k]) and torch.equal(b[k], ref2[k])
        assert torch.equal(f, f1)
    finally:
        wq.windq_destroy(other)


def test_one_context_on_two_streams_ordered_by_events(wq, ctx):
    """Calls on one context share its scratch buffer, so they must not overlap on the GPU.  Two streams that hand
    the context back and forth through events (each call's stream waits for an event recorded after the previous
    call) are ordered, and give the results of a single stream."""
    W1 = ws.weights(400, 1024, 650, "student_t").cuda()
    W2 = ws.weights(300, 2048, 651, "student_t").cuda()
    s1, s2 = torch.rand(1024, device="cuda") + 0.1, torch.rand(2048, device="cuda") + 0.1
    grid = torch.from_numpy(ws.clip_grid(20)).cuda()
    ref1 = wq.windq_fit_eval(ctx, W1, 128, s1, grid)
    ref2 = wq.windq_fit_eval(ctx, W2, 64, s2, grid)
    ref_f = wq.windq_unit_features(ctx, W1, 128, s1).clone()
    torch.cuda.synchronize()
    st = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = []
    prev = None
    for n in range(6):
        cur = st[n % 2]
        if prev is not None:
            cur.wait_event(prev)
        with torch.cuda.stream(cur):
            if n % 3 == 0:
                outs.append(("fit1", wq.windq_fit_eval(ctx, W1, 128, s1, grid, stream=cur)))
            elif n % 3 == 1:
                outs.append(("fit2", wq.windq_fit_eval(ctx, W2, 64, s2, grid, stream=cur)))
            else:
                outs.append(("feat", wq.windq_unit_features(ctx, W1, 128, s1, stream=cur)))
            prev = torch.cuda.Event()
            prev.record(cur)
    torch.cuda.synchronize()
    for name, out in outs:
        if name == "feat":
            assert torch.equal(out, ref_f)
        else:
            ref = ref1 if name == "fit1" else ref2
            for k in ("err", "energy", "clip_idx"):
                assert torch.equal(out[k], ref[k]), (name, k)


def test_apply_plan_leaves_a_unit_with_a_bad_action_code_untouched(wq, ctx, oracle):
    """Action codes live on the device: a code above 6 cannot be refused before the launch.  The unit is skipped
    (its outputs keep what the arrays held), windq_effective_bits flags the plan with totals of -1, and every
    other unit is packed as the oracle packs it."""
    G, R, C = 128, 40, 640
    W, X = make(R, C, 660)
    s = oracle.act_stats(X.numpy())
    grid = ws.clip_grid(20)
    acts = np.array([4, 5, 9, 6, 2], np.uint8)
    bad = 2
    fit = oracle.fit_eval(W.numpy(), G, s, grid, threads=4, want_group_err=False)
    a_d = torch.from_numpy(acts).cuda()
    eb = wq.windq_effective_bits(ctx, a_d, R, G)
    assert int(eb["total_centibits"].item()) == -1 and int(eb["total_packed_bytes"].item()) == -1
    offs = eb["code_offsets"].cpu().numpy()
    assert offs[bad + 1] == offs[bad]                       # the flagged unit has an empty block
    U = C // G
    codes = torch.full((int(offs[-1]),), 0xEE, dtype=torch.uint8, device="cuda")
    canary = dict(scales=torch.full((U, R), 7.0, dtype=torch.float16, device="cuda"),
                  zeros=torch.full((U, R), 7.0, dtype=torch.float16, device="cuda"),
                  wq=torch.full((R, C), 7.0, dtype=torch.float16, device="cuda"))
    plan = wq.windq_apply_plan(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(), a_d,
                               eb["code_offsets"], codes, torch.from_numpy(fit["clip_idx"]).cuda(), out=canary)
    torch.cuda.synchronize()
    assert bool((plan["scales"][bad] == 7.0).all()) and bool((plan["zeros"][bad] == 7.0).all())
    assert bool((plan["wq"][:, bad * G:(bad + 1) * G] == 7.0).all())
    for u in range(U):
        if u == bad:
            continue
        want = oracle.apply_plan(W.numpy()[:, u * G:(u + 1) * G], G, s[u * G:(u + 1) * G], grid, acts[u:u + 1],
                                 fit["clip_idx"][:, u:u + 1])
        assert (codes[offs[u]:offs[u + 1]].cpu().numpy() == want["codes"]).all()
        assert (plan["scales"][u].cpu().view(torch.int16).numpy().view(np.uint16) == want["scales"][0]).all()
        assert (plan["wq"][:, u * G:(u + 1) * G].cpu().contiguous().view(torch.int16).numpy().view(np.uint16) == want["wq"]).all()


def test_fit_eval_largest_grid_and_widest_chunk(wq, ctx, oracle):
    G, R, C, K = 512, 21, 1024, 64
    W, X = make(R, C, 640)
    s = oracle.act_stats(X.numpy())
    grid = ws.clip_grid(K, lo=1.0 / 64.0)
    want = oracle.fit_eval(W.numpy(), G, s, grid, threads=8)
    check_fit(run_fit(wq, ctx, W, G, s, grid), want)
    acts = np.array([4, 2], np.uint8)
    o = oracle.apply_plan(W.numpy(), G, s, grid, acts, None)
    got = run_apply(wq, ctx, W, G, s, grid, acts, None)
    for key in ("codes", "scales", "zeros", "wq"):
        assert (got[key] == o[key]).all(), key


def test_act_stats_near_the_fp16_limit(wq, ctx, oracle):
    X = torch.full((300, 64), 60000.0, dtype=torch.float16)
    X[::2] = -65504.0
    got = wq.windq_act_stats(ctx, X.cuda()).cpu().numpy()
    assert np.isfinite(got).all() and close(got, oracle.act_stats(X.numpy())).all()


# ------------------------------------------------------------------ full size, sampled units
def plan_for_target(wq, ctx, U, R, G, target, seed):
    """A seeded random plan at `target` average bits (the benchmark's recipe): the cost table comes
    from windq_effective_bits itself, the drawing from the shared generator module."""
    all_actions = torch.arange(7, dtype=torch.uint8, device="cuda")
    per_action = wq.windq_effective_bits(ctx, all_actions, R, G)["unit_centibits"].cpu().numpy()
    costs = np.tile(per_action[None, :], (U, 1))
    return ws.random_plan(costs, np.full(U, R * G, np.int64), target, seed)


FULL_SIZE_CASES = [
    # config, matrix index in the block, units sampled per chunk width, plan target (None: uniform random actions)
    ("cfg2_llama7b_block", 6, 2, 2.0),      # down_proj 4096 x 11008, N(0, 0.02), plan at 2.0 bits
    ("cfg3_llama7b_model", 4, 3, None),     # gate_proj 11008 x 4096, Student-t, chunk widths 64 and 128
    ("cfg3_llama7b_model", 0, 2, 1.58),     # q_proj 4096 x 4096, plan at 1.58 bits
    ("cfg4_llama13b_model", 5, 2, 3.0),     # up_proj 13824 x 5120, 40 clip ratios, 4096 tokens
    ("cfg5_llama70b_model", 4, 1, 2.0),     # gate_proj 28672 x 8192
    ("cfg5_llama70b_model", 1, 2, 2.0),     # k_proj 1024 x 8192 (grouped-query attention)
    ("cfg5_llama70b_model", 6, 1, 2.0),     # down_proj 8192 x 28672
    ("llama3_8b_g256", 4, 1, None),         # gate_proj 14336 x 4096 at the paper's chunk sizes 256 and 512
    ("llama3_8b_g256", 2, 2, None),         # v_proj 1024 x 4096 (grouped-query attention)
    ("llama32_1b_g256", 6, 2, 2.0),         # down_proj 2048 x 8192 of the 1B shape, chunk size 256, plan at 2.0 bits
    ("llama32_1b_g256", 1, 1, None),        # k_proj 512 x 2048
]


@pytest.mark.parametrize("config,mi,n_units,target", FULL_SIZE_CASES)
def test_full_size_matrix_sampled_units(wq, ctx, oracle, config, mi, n_units, target):
    """A full-size matrix of one of the five configurations, generated on the device with the
    benchmark's recipe and run in the benchmark's launch shape; the oracle recomputes sampled units
    from the same bits.  Properties that hold at any size are checked on every unit."""
    spec = ws.CONFIGS[config]
    m = spec.block_matrices()[mi]
    W = ws.block_weight(spec, 0, 0, m, device="cuda")
    X = ws.block_input(spec, 0, 0, m.x_id, device="cuda")
    s = wq.windq_act_stats(ctx, X)
    grid = ws.clip_grid(spec.K)
    grid_d = torch.from_numpy(grid).cuda()
    s_h = s.cpu().numpy()
    assert close(s_h, oracle.act_stats(X.cpu().numpy())).all()
    del X
    for G in spec.chunk_widths:
        U = m.C // G
        fit = wq.windq_fit_eval(ctx, W, G, s, grid_d)
        feat = wq.windq_unit_features(ctx, W, G, s).cpu().numpy()
        rng = np.random.default_rng(G)
        if target is None:
            acts = rng.integers(0, 7, U).astype(np.uint8)
        else:
            acts = plan_for_target(wq, ctx, U, m.R, G, target, 17)
        a_d = torch.from_numpy(acts).cuda()
        eb = wq.windq_effective_bits(ctx, a_d, m.R, G)
        o_eb = oracle.effective_bits(acts, m.R, G)
        assert int(eb["total_centibits"].item()) == o_eb["total_centibits"]
        assert int(eb["total_packed_bytes"].item()) == o_eb["total_packed_bytes"]
        assert (eb["code_offsets"].cpu().numpy() == o_eb["code_offsets"]).all()
        if target is not None:
            assert abs(o_eb["total_centibits"] / (100.0 * m.R * m.C) - target) <= 0.005
        codes = torch.empty(int(eb["code_offsets"][-1].item()), dtype=torch.uint8, device="cuda")
        plan = wq.windq_apply_plan(ctx, W, G, s, grid_d, a_d, eb["code_offsets"], codes, fit["clip_idx"])
        offs = eb["code_offsets"].cpu().numpy()
        # any size: every clip index is a grid index; errors are finite and non-negative; skip units
        # come back unchanged
        err = fit["err"].cpu().numpy()
        assert int(fit["clip_idx"].max().item()) < spec.K
        assert np.isfinite(err).all() and (err >= 0).all() and (fit["energy"].cpu().numpy() >= err[:, 5] * 0).all()
        for u in np.flatnonzero(acts == 0)[:2]:
            assert torch.equal(plan["wq"][:, u * G:(u + 1) * G], W[:, u * G:(u + 1) * G])
        for u in rng.choice(U, n_units, replace=False):
            Wu = W[:, u * G:(u + 1) * G].cpu().numpy()
            su = s_h[u * G:(u + 1) * G]
            want = oracle.fit_eval(Wu, G, su, grid, threads=8, want_group_err=False)
            assert (fit["clip_idx"][:, u].cpu().numpy() == want["clip_idx"][:, 0]).all()
            assert close(fit["err"][u].cpu().numpy(), want["err"][0]).all()
            assert close(fit["energy"][u].cpu().numpy(), want["energy"][0]).all()
            wf = oracle.unit_features(Wu, G, su)
            assert (feat[u, 3:5] == wf[0, 3:5]).all() and close(feat[u], wf[0]).all()
            wp = oracle.apply_plan(Wu, G, su, grid, acts[u:u + 1], want["clip_idx"])
            assert (codes[offs[u]:offs[u + 1]].cpu().numpy() == wp["codes"]).all()
            assert (plan["scales"][u].cpu().view(torch.int16).numpy().view(np.uint16) == wp["scales"][0]).all()
            assert (plan["zeros"][u].cpu().view(torch.int16).numpy().view(np.uint16) == wp["zeros"][0]).all()
            assert (plan["wq"][:, u * G:(u + 1) * G].cpu().view(torch.int16).numpy().view(np.uint16) == wp["wq"]).all()
    del W
    torch.cuda.empty_cache()


@pytest.mark.parametrize("R,C,G", [(512, 2048, 256), (512, 2048, 128), (100, 4096, 512), (1000, 512, 32)])
def test_fit_eval_of_a_matrix_smaller_than_the_grid(wq, ctx, oracle, R, C, G):
    """Matrices with fewer items than the grid has warps take the launch shape that hands every item out in
    five parts; clip indices and group errors must be those of the oracle bit for bit, unit sums within tolerance."""
    W = ws.weights(R, C, 77 + R, "student_t")
    X = ws.activations(64, C, 78)
    s = oracle.act_stats(X.numpy())
    grid = ws.clip_grid(20)
    got = wq.windq_fit_eval(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(), want_group_err=True)
    torch.cuda.synchronize()
    units = sorted(set([0, C // G - 1, (C // G) // 2]))
    cols = np.concatenate([np.arange(u * G, (u + 1) * G) for u in units])
    want = oracle.fit_eval(W.numpy()[:, cols], G, s[cols], grid)
    assert np.array_equal(got["clip_idx"][:, units].cpu().numpy(), want["clip_idx"])
    assert np.array_equal(got["group_err"][:, units].cpu().numpy().view(np.uint32), want["group_err"].view(np.uint32))
    assert close(got["err"][units].cpu().numpy(), want["err"]).all()
    assert close(got["energy"][units].cpu().numpy(), want["energy"]).all()


def test_apply_plan_clip_indices_beyond_the_grid_mean_the_last_ratio(wq, ctx, oracle):
    R, C, G, K = 40, 512, 128, 7
    W = ws.weights(R, C, 91, "student_t")
    s = oracle.act_stats(ws.activations(64, C, 92).numpy())
    grid = ws.clip_grid(K)
    U = C // G
    idx = np.random.default_rng(3).integers(0, 256, (4, U, R)).astype(np.uint8)      # most entries are >= K
    actions = np.array([1, 2, 3, 4], np.uint8)
    ad = torch.from_numpy(actions).cuda()
    eb = wq.windq_effective_bits(ctx, ad, R, G)
    codes = torch.zeros(2 * R * C + 16 * U, dtype=torch.uint8, device="cuda")
    got = wq.windq_apply_plan(ctx, W.cuda(), G, torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda(), ad,
                              eb["code_offsets"], codes, torch.from_numpy(idx).cuda())
    torch.cuda.synchronize()
    want = oracle.apply_plan(W.numpy(), G, s, grid, actions, idx)
    clamped = oracle.apply_plan(W.numpy(), G, s, grid, actions, np.minimum(idx, K - 1))
    assert np.array_equal(want["codes"], clamped["codes"]) and np.array_equal(want["wq"], clamped["wq"])
    n = int(want["code_offsets"][U])
    assert np.array_equal(got["codes"][:n].cpu().numpy(), want["codes"])
    assert np.array_equal(got["scales"].cpu().numpy().view(np.uint16), want["scales"])
    assert np.array_equal(got["zeros"].cpu().numpy().view(np.uint16), want["zeros"])
    assert np.array_equal(got["wq"].cpu().numpy().view(np.uint16), want["wq"])


@pytest.mark.parametrize("G,shapes", [(128, [(300, 512), (64, 1024), (1000, 256), (17, 128)]),
                                      (64, [(40, 256), (2048, 2048)]),
                                      (256, [(512, 2048)] * 3 + [(2048, 2048)]),
                                      (32, [(5, 32)])])
def test_fit_eval_batch_equals_the_separate_calls(wq, ctx, oracle, G, shapes):
    """Several matrices in one launch: every output of every job equals that of its own windq_fit_eval call bit
    for bit (clip indices, group errors, and the unit sums, which are added in the same order), and sampled units
    equal the oracle."""
    grid = ws.clip_grid(20)
    gd = torch.from_numpy(grid).cuda()
    Ws = [ws.weights(R, C, 300 + i, "student_t").cuda() for i, (R, C) in enumerate(shapes)]
    ss = [(torch.rand(C, generator=torch.Generator().manual_seed(i)) * 3 + 0.01).cuda() for i, (R, C) in enumerate(shapes)]
    got = wq.windq_fit_eval_batch(ctx, Ws, G, ss, gd, want_group_err=True)
    torch.cuda.synchronize()
    for W, s, out in zip(Ws, ss, got):
        one = wq.windq_fit_eval(ctx, W, G, s, gd, want_group_err=True)
        assert torch.equal(out["clip_idx"], one["clip_idx"])
        assert torch.equal(out["group_err"].view(torch.int32), one["group_err"].view(torch.int32))
        assert torch.equal(out["err"].view(torch.int32), one["err"].view(torch.int32))
        assert torch.equal(out["energy"].view(torch.int32), one["energy"].view(torch.int32))
    W, s, out = Ws[0], ss[0], got[0]
    want = oracle.fit_eval(W.cpu().numpy()[:, :G], G, s.cpu().numpy()[:G], grid)
    assert np.array_equal(out["clip_idx"][:, :1].cpu().numpy(), want["clip_idx"])
    assert close(out["err"][:1].cpu().numpy(), want["err"]).all()


def test_fit_eval_batch_argument_checks(wq, ctx):
    gd = torch.from_numpy(ws.clip_grid(4)).cuda()
    W = torch.zeros((8, 128), dtype=torch.float16, device="cuda")
    s = torch.ones(128, device="cuda")
    with pytest.raises(Exception):
        wq.windq_fit_eval_batch(ctx, [W] * 17, 128, [s] * 17, gd)
    with pytest.raises(Exception):
        wq.windq_fit_eval_batch(ctx, [W, torch.zeros((8, 100), dtype=torch.float16, device="cuda")], 128, [s, s], gd)
    out = wq.windq_fit_eval_batch(ctx, [W], 128, [s], gd)
    assert (out[0]["err"] == 0).all()


@pytest.mark.parametrize("G,shapes", [(128, [(300, 512), (64, 1024), (1000, 256), (17, 128)]),
                                      (64, [(40, 256), (2048, 2048)]),
                                      (256, [(512, 2048)] * 3 + [(2048, 2048)]),
                                      (32, [(5, 32)]),
                                      (128, [(5000, 128), (3, 4096)])])
def test_unit_features_batch_equals_the_separate_calls(wq, ctx, oracle, G, shapes):
    """Several matrices in one pass: the histogram features and those of s equal the separate calls bit for bit,
    the mean within tolerance, and everything equals the oracle within tolerance."""
    Ws = [ws.weights(R, C, 400 + i, "student_t").cuda() for i, (R, C) in enumerate(shapes)]
    for W in Ws:
        W[::7, ::3] = 0
    ss = [(torch.rand(C, generator=torch.Generator().manual_seed(i)) * 3 + 0.01).cuda() for i, (R, C) in enumerate(shapes)]
    got = wq.windq_unit_features_batch(ctx, Ws, G, ss)
    torch.cuda.synchronize()
    for W, s, f in zip(Ws, ss, got):
        one = wq.windq_unit_features(ctx, W, G, s)
        assert torch.equal(f[:, 1:].view(torch.int32), one[:, 1:].view(torch.int32))
        assert close(f[:, 0].cpu().numpy(), one[:, 0].cpu().numpy()).all()
        want = oracle.unit_features(W.cpu().numpy(), G, s.cpu().numpy())
        assert close(f.cpu().numpy(), want).all()


def test_batches_take_strided_matrices_and_preallocated_outputs(wq, ctx):
    """Jobs that are column slices of one wider tensor (ldw > C) and outputs supplied by the caller."""
    G = 128
    big = ws.weights(200, 1024, 510, "student_t").cuda()
    Ws = [big[:, :256], big[:, 256:768], big[:100, 768:]]
    ss = [(torch.rand(W.shape[1], generator=torch.Generator().manual_seed(i)) + 0.01).cuda() for i, W in enumerate(Ws)]
    gd = torch.from_numpy(ws.clip_grid(20)).cuda()
    feats = [torch.full((W.shape[1] // G, 8), -1.0, device="cuda") for W in Ws]
    out_f = wq.windq_unit_features_batch(ctx, Ws, G, ss, feats)
    outs = [dict(err=torch.full((W.shape[1] // G, 6), -1.0, device="cuda")) for W in Ws]
    out_e = wq.windq_fit_eval_batch(ctx, Ws, G, ss, gd, outs=outs, want_energy=False, want_clip_idx=False)
    torch.cuda.synchronize()
    for W, s, f, o, o_given in zip(Ws, ss, out_f, out_e, outs):
        Wc = W.contiguous()
        assert torch.equal(f[:, 1:], wq.windq_unit_features(ctx, Wc, G, s)[:, 1:])
        one = wq.windq_fit_eval(ctx, Wc, G, s, gd)
        assert o["err"].data_ptr() == o_given["err"].data_ptr() and o["energy"] is None and o["clip_idx"] is None
        assert torch.equal(o["err"], one["err"])


def test_effective_bits_batch_equals_the_separate_calls(wq, ctx, oracle):
    rng = np.random.default_rng(8)
    G = 128
    plans = [(rng.integers(0, 7, U).astype(np.uint8), R) for U, R in [(32, 4096), (86, 4096), (1, 3), (1500, 11008), (32, 11008)] * 4]
    plans[3][0][5] = 9                                            # a code that is not an action: totals of -1
    acts = [torch.from_numpy(a).cuda() for a, _ in plans]
    got = wq.windq_effective_bits_batch(ctx, acts, [R for _, R in plans], G, 16, 8)
    torch.cuda.synchronize()
    for (a, R), ad, out in zip(plans, acts, got):
        one = wq.windq_effective_bits(ctx, ad, R, G, 16, 8)
        for key in ("unit_centibits", "code_offsets", "total_centibits", "total_packed_bytes"):
            assert torch.equal(out[key], one[key]), key
    want = oracle.effective_bits(plans[0][0], plans[0][1], G, 16, 8)
    assert int(got[0]["total_centibits"].item()) == int(want["total_centibits"])
    assert np.array_equal(got[0]["code_offsets"].cpu().numpy(), want["code_offsets"])
    assert int(got[3]["total_centibits"].item()) == -1
    with pytest.raises(Exception):
        wq.windq_effective_bits_batch(ctx, acts * 2, [R for _, R in plans] * 2, G)      # 40 jobs


@pytest.mark.parametrize("G,shapes", [(128, [(300, 512), (64, 1024), (17, 128)]), (64, [(40, 256), (1100, 512)]),
                                      (256, [(512, 2048), (33, 256)]), (32, [(5, 32)])])
def test_apply_plan_batch_equals_the_separate_calls(wq, ctx, oracle, G, shapes):
    """Three plans of every matrix in one launch: codes, scales, zero points and fake-quantised weights of every job
    equal those of its own windq_apply_plan call bit for bit, and one job equals the oracle."""
    grid = ws.clip_grid(20)
    gd = torch.from_numpy(grid).cuda()
    rng = np.random.default_rng(G)
    jobs, singles = [], []
    for i, (R, C) in enumerate(shapes):
        W = ws.weights(R, C, 700 + i, "student_t").cuda()
        s = (torch.rand(C, generator=torch.Generator().manual_seed(i)) * 3 + 0.01).cuda()
        U = C // G
        fit = wq.windq_fit_eval(ctx, W, G, s, gd)
        for plan in range(3):
            acts = torch.from_numpy(rng.integers(0, 7, U).astype(np.uint8)).cuda()
            eb = wq.windq_effective_bits(ctx, acts, R, G)
            jobs.append(dict(W=W, s=s, actions=acts, clip_idx=fit["clip_idx"], code_offsets=eb["code_offsets"],
                             codes=torch.zeros(2 * R * C + 16 * U, dtype=torch.uint8, device="cuda")))
            singles.append(wq.windq_apply_plan(ctx, W, G, s, gd, acts, eb["code_offsets"],
                                               torch.zeros(2 * R * C + 16 * U, dtype=torch.uint8, device="cuda"), fit["clip_idx"]))
    got = wq.windq_apply_plan_batch(ctx, jobs, G, gd)
    torch.cuda.synchronize()
    assert len(got) == len(jobs)
    for out, one in zip(got, singles):
        assert torch.equal(out["codes"], one["codes"])
        assert torch.equal(out["scales"].view(torch.int16), one["scales"].view(torch.int16))
        assert torch.equal(out["zeros"].view(torch.int16), one["zeros"].view(torch.int16))
        assert torch.equal(out["wq"].view(torch.int16), one["wq"].view(torch.int16))
    j0 = jobs[1]
    want = oracle.apply_plan(j0["W"].cpu().numpy(), G, j0["s"].cpu().numpy(), grid, j0["actions"].cpu().numpy(),
                             j0["clip_idx"].cpu().numpy())
    n = int(want["code_offsets"][-1])
    assert np.array_equal(got[1]["codes"][:n].cpu().numpy(), want["codes"])
    assert np.array_equal(got[1]["wq"].cpu().numpy().view(np.uint16), want["wq"])


def test_apply_plan_batch_argument_checks(wq, ctx):
    gd = torch.from_numpy(ws.clip_grid(4)).cuda()
    W = torch.zeros((8, 128), dtype=torch.float16, device="cuda")
    s = torch.ones(128, device="cuda")
    acts = torch.zeros(1, dtype=torch.uint8, device="cuda")
    eb = wq.windq_effective_bits(ctx, acts, 8, 128)
    idx = torch.zeros((4, 1, 8), dtype=torch.uint8, device="cuda")
    job = dict(W=W, s=s, actions=acts, clip_idx=idx, code_offsets=eb["code_offsets"],
               codes=torch.zeros(4096, dtype=torch.uint8, device="cuda"), wq=None)
    with pytest.raises(Exception):
        wq.windq_apply_plan_batch(ctx, [job] * 25, 128, gd)
    out = wq.windq_apply_plan_batch(ctx, [job], 128, gd)
    assert out[0]["wq"] is None and (out[0]["codes"][:2048] == 0).all()


@pytest.mark.parametrize("G,shapes", [(128, [(300, 512), (64, 1024), (1000, 256), (17, 128)]),
                                      (64, [(40, 256), (2048, 2048)]),
                                      (256, [(512, 2048)] * 3 + [(2048, 2048)]),
                                      (32, [(5, 32)]),
                                      (128, [(5000, 128), (3, 4096)])])
def test_features_fit_batch_equals_the_two_batched_calls(wq, ctx, oracle, G, shapes):
    """Features and fits in one pass over the weights: fit outputs equal windq_fit_eval_batch bit for bit, the
    histogram features and those of s equal windq_unit_features_batch bit for bit, the mean within tolerance, and
    everything equals the oracle."""
    grid = ws.clip_grid(20)
    gd = torch.from_numpy(grid).cuda()
    Ws = [ws.weights(R, C, 500 + i, "student_t").cuda() for i, (R, C) in enumerate(shapes)]
    for W in Ws:
        W[::7, ::3] = 0
    ss = [(torch.rand(C, generator=torch.Generator().manual_seed(i)) * 3 + 0.01).cuda() for i, (R, C) in enumerate(shapes)]
    feats, fits = wq.windq_features_fit_batch(ctx, Ws, G, ss, gd, want_group_err=True)
    torch.cuda.synchronize()
    ref_fit = wq.windq_fit_eval_batch(ctx, Ws, G, ss, gd, want_group_err=True)
    ref_feat = wq.windq_unit_features_batch(ctx, Ws, G, ss)
    torch.cuda.synchronize()
    for W, s, f, out, rf, rfit in zip(Ws, ss, feats, fits, ref_feat, ref_fit):
        for k in ("clip_idx", "group_err", "err", "energy"):
            assert torch.equal(out[k].view(torch.uint8), rfit[k].view(torch.uint8)), k
        assert torch.equal(f[:, 1:].view(torch.int32), rf[:, 1:].view(torch.int32))
        assert close(f[:, 0].cpu().numpy(), rf[:, 0].cpu().numpy()).all()
        want = oracle.unit_features(W.cpu().numpy(), G, s.cpu().numpy())
        assert (f[:, 3:5].cpu().numpy() == want[:, 3:5]).all() and close(f.cpu().numpy(), want).all()
    # twice in a row: the histograms are cleared by the call
    feats2, _ = wq.windq_features_fit_batch(ctx, Ws, G, ss, gd)
    torch.cuda.synchronize()
    for a, b in zip(feats, feats2):
        assert torch.equal(a[:, 1:], b[:, 1:])


@pytest.mark.parametrize("G,shapes", [(64, [(300, 512), (64, 1024), (1000, 256)]), (128, [(40, 256), (2048, 2048)]),
                                      (32, [(5, 64)]), (256, [(512, 2048), (33, 512)])])
def test_unit_features_at_two_widths_from_one_pass(wq, ctx, oracle, G, shapes):
    """windq_unit_features_batch2: the features at width 2 G come from pairs of the histograms built at width G; both
    sets equal their own windq_unit_features_batch calls (histogram features and those of s bit for bit, the mean
    within tolerance) and the oracle."""
    Ws = [ws.weights(R, C, 600 + i, "student_t").cuda() for i, (R, C) in enumerate(shapes)]
    for W in Ws:
        W[::7, ::3] = 0
    ss = [(torch.rand(C, generator=torch.Generator().manual_seed(i)) * 3 + 0.01).cuda() for i, (R, C) in enumerate(shapes)]
    fine, wide = wq.windq_unit_features_batch(ctx, Ws, G, ss, feats_2G=True)
    torch.cuda.synchronize()
    ref_fine = wq.windq_unit_features_batch(ctx, Ws, G, ss)
    ref_wide = wq.windq_unit_features_batch(ctx, Ws, 2 * G, ss)
    torch.cuda.synchronize()
    for W, s, f, f2, rf, rw in zip(Ws, ss, fine, wide, ref_fine, ref_wide):
        assert torch.equal(f.view(torch.int32), rf.view(torch.int32))
        assert torch.equal(f2[:, 1:].view(torch.int32), rw[:, 1:].view(torch.int32))
        assert close(f2[:, 0].cpu().numpy(), rw[:, 0].cpu().numpy()).all()
        want = oracle.unit_features(W.cpu().numpy(), 2 * G, s.cpu().numpy())
        assert (f2[:, 3:5].cpu().numpy() == want[:, 3:5]).all() and close(f2.cpu().numpy(), want).all()
    # a job may decline the wider units; an odd number of units is refused when any job asks for them
    only_first = [True] + [None] * (len(Ws) - 1)
    f_only, w_only = wq.windq_unit_features_batch(ctx, Ws, G, ss, feats_2G=[torch.empty_like(wide[0])] + only_first[1:])
    torch.cuda.synchronize()
    assert torch.equal(w_only[0], wide[0]) and all(x is None for x in w_only[1:])
    odd = torch.zeros((8, 3 * G), dtype=torch.float16, device="cuda")
    with pytest.raises(wq.WindqError) as e:
        wq.windq_unit_features_batch(ctx, [odd], G, [torch.ones(3 * G, device="cuda")], feats_2G=[torch.zeros((1, 8), device="cuda")])
    assert e.value.status == 2
