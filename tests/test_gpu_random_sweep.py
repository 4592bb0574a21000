"""Randomised parity sweep on the GPU: random shapes, chunk widths, grid sizes, weight and statistic distributions
(zeros, one-sided, ties, sparse, fp16 subnormals, outlier columns, statistics spanning 20 decades) through the whole
chain -- features, fits, plan packing (one plan, and several plans in one pass), the search over the ternary
assignment and packing with its thresholds, salient selection, protected fits, refinement, protected and refined
packing -- against the oracle.  Integer and bit-pattern outputs are compared exactly."""
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


def gen_W(rng, R, C):
    kind = rng.integers(0, 8)
    if kind == 0:
        W = rng.standard_normal((R, C)) * 0.02
    elif kind == 1:
        W = rng.standard_t(3, (R, C)) * 0.02
    elif kind == 2:
        W = rng.standard_normal((R, C)) * 10 ** rng.uniform(-7, 3)
    elif kind == 3:
        W = np.abs(rng.standard_normal((R, C)))                              # one-sided
    elif kind == 4:
        W = -np.abs(rng.standard_normal((R, C))) * 1e-3
    elif kind == 5:
        W = np.round(rng.standard_normal((R, C)) * 3) / 4                    # many ties
    elif kind == 6:
        W = rng.standard_normal((R, C)) * (rng.random((R, C)) < 0.1)         # sparse
    else:
        W = rng.standard_normal((R, C)) * 1e-6                               # fp16 subnormals
    W = W.astype(np.float16)
    if rng.random() < 0.3:
        W[rng.integers(0, R), :] = 0
    if rng.random() < 0.3:
        W[:, rng.integers(0, C)] *= np.float16(50)
    W[~np.isfinite(W)] = 0
    return W


def gen_s(rng, C):
    kind = rng.integers(0, 5)
    if kind == 0:
        s = rng.random(C) * 4 + 0.01
    elif kind == 1:
        s = rng.lognormal(0, 2, C)
    elif kind == 2:
        s = rng.random(C) * (rng.random(C) < 0.5)                            # many zeros
    elif kind == 3:
        s = np.full(C, 1.0)
    else:
        s = rng.random(C) * 10 ** rng.uniform(-12, 8)
    return s.astype(np.float32)


def bits32(a):
    return np.ascontiguousarray(a).view(np.uint32)


def bits16(t):
    return t.cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("seed", range(6))
def test_random_chain(wq, ctx, oracle, seed):
    rng = np.random.default_rng(1000 + seed)
    for it in range(10):
        G = int(rng.choice([32, 64, 128, 256, 512]))
        U = int(rng.integers(1, 5))
        C = G * U
        R = int(rng.integers(1, 140))
        K = int(rng.choice([1, 2, 7, 20, 33, 64]))
        W, s, grid = gen_W(rng, R, C), gen_s(rng, C), ws.clip_grid(K)
        Wd, sd, gd = torch.from_numpy(W).cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda()
        tag = "seed=%d it=%d G=%d U=%d R=%d K=%d" % (seed, it, G, U, R, K)

        assert np.allclose(wq.windq_unit_features(ctx, Wd, G, sd).cpu().numpy(), oracle.unit_features(W, G, s),
                           rtol=1e-4, atol=1e-6), tag
        want = oracle.fit_eval(W, G, s, grid)
        got = wq.windq_fit_eval(ctx, Wd, G, sd, gd, want_group_err=True)
        assert np.array_equal(got["clip_idx"].cpu().numpy(), want["clip_idx"]), tag
        assert np.array_equal(bits32(got["group_err"].cpu().numpy()), bits32(want["group_err"])), tag

        actions = rng.integers(0, 7, U).astype(np.uint8)
        ad = torch.from_numpy(actions).cuda()
        eb = wq.windq_effective_bits(ctx, ad, R, G)
        codes = torch.zeros(2 * R * C + 16 * U, dtype=torch.uint8, device="cuda")
        use_idx = rng.random() < 0.7
        pg = wq.windq_apply_plan(ctx, Wd, G, sd, gd, ad, eb["code_offsets"], codes, got["clip_idx"] if use_idx else None)
        po = oracle.apply_plan(W, G, s, grid, actions, want["clip_idx"] if use_idx else None)
        n = int(po["code_offsets"][U])
        assert np.array_equal(pg["codes"][:n].cpu().numpy(), po["codes"]), tag
        assert np.array_equal(bits16(pg["wq"]), po["wq"]), tag
        assert np.array_equal(bits16(pg["scales"]), po["scales"]) and np.array_equal(bits16(pg["zeros"]), po["zeros"]), tag

        # unit sums without group errors (the 1.58- and 1-bit ones then come from the fit's sums): tolerance outputs
        plain = wq.windq_fit_eval(ctx, Wd, G, sd, gd)
        assert np.array_equal(plain["clip_idx"].cpu().numpy(), want["clip_idx"]), tag
        assert np.allclose(plain["err"].cpu().numpy(), want["err"], rtol=1e-4, atol=1e-6), tag

        # several plans of the matrix in one pass
        n_plans = int(rng.integers(1, 5))
        plans, wants = [], []
        for p in range(n_plans):
            acts_p = rng.integers(0, 7, U).astype(np.uint8)
            ap = torch.from_numpy(acts_p).cuda()
            ebp = wq.windq_effective_bits(ctx, ap, R, G)
            plans.append(dict(actions=ap, code_offsets=ebp["code_offsets"],
                              codes=torch.zeros(2 * R * C + 16 * U, dtype=torch.uint8, device="cuda")))
            wants.append(oracle.apply_plan(W, G, s, grid, acts_p, want["clip_idx"]))
        outs = wq.windq_apply_plan_multi(ctx, Wd, G, sd, gd, got["clip_idx"], plans)
        for out, wp in zip(outs, wants):
            m = int(wp["code_offsets"][U])
            assert np.array_equal(out["codes"][:m].cpu().numpy(), wp["codes"]) and np.array_equal(bits16(out["wq"]), wp["wq"]), tag
            assert np.array_equal(bits16(out["scales"]), wp["scales"]) and np.array_equal(bits16(out["zeros"]), wp["zeros"]), tag

        # search over the ternary assignment, and packing with its thresholds
        Kt = int(rng.choice([1, 3, 9, 64]))
        thr = np.sort(rng.uniform(0.05, 3.0, Kt)).astype(np.float32)
        td = torch.from_numpy(thr).cuda()
        to = oracle.fit_ternary_search(W, G, s, thr)
        tg = wq.windq_fit_ternary_search(ctx, Wd, G, sd, td, want_group_err=True)
        assert np.array_equal(tg["thr_idx"].cpu().numpy(), to["thr_idx"]), tag
        assert np.array_equal(bits16(tg["alpha"]), to["alpha"].view(np.uint16)), tag
        assert np.array_equal(bits32(tg["group_err"].cpu().numpy()), bits32(to["group_err"])), tag
        codes.zero_()
        sgp = wq.windq_apply_plan_searched(ctx, Wd, G, sd, gd, ad, eb["code_offsets"], codes, got["clip_idx"], td, tg["thr_idx"])
        sop = oracle.apply_plan_searched(W, G, s, grid, actions, want["clip_idx"], thr, to["thr_idx"])
        assert np.array_equal(sgp["codes"][:n].cpu().numpy(), sop["codes"]) and np.array_equal(bits16(sgp["wq"]), sop["wq"]), tag
        assert np.array_equal(bits16(sgp["scales"]), sop["scales"]), tag

        rate = int(rng.choice([0, 10000, 30000, 200000, 1000000]))
        so = oracle.salient_select(W, G, s, rate)
        sg = wq.windq_salient_select(ctx, Wd, G, sd, rate)
        assert np.array_equal(bits32(sg["thresh"].cpu().numpy()), bits32(so["thresh"])), tag
        assert np.array_equal(sg["count"].cpu().numpy(), so["count"]) and np.array_equal(sg["mask"].cpu().numpy(), so["mask"]), tag
        fpo = oracle.fit_eval(W, G, s, grid, thresh=so["thresh"])
        fpg = wq.windq_fit_eval(ctx, Wd, G, sd, gd, want_group_err=True, thresh=sg["thresh"])
        assert np.array_equal(fpg["clip_idx"].cpu().numpy(), fpo["clip_idx"]), tag
        assert np.array_equal(bits32(fpg["group_err"].cpu().numpy()), bits32(fpo["group_err"])), tag

        T = int(rng.choice([0, 1, 5, 10, 32]))
        lr = float(rng.choice([0.0, 0.01, 0.05, 0.5, 1.0]))
        ro = oracle.fit_refine(W, G, s, grid, fpo["clip_idx"], T=T, lr=lr, thresh=so["thresh"])
        rg = wq.windq_fit_refine(ctx, Wd, G, sd, gd, fpg["clip_idx"], T, lr, want_group_err=True, thresh=sg["thresh"])
        assert np.array_equal(bits16(rg["scale"]), ro["scale"].view(np.uint16)), tag
        assert np.array_equal(bits32(rg["group_err"].cpu().numpy()), bits32(ro["group_err"])), tag

        prot_q = torch.zeros(R * C, dtype=torch.int8, device="cuda")
        codes.zero_()
        ag = wq.windq_apply_plan_protected(ctx, Wd, G, sd, gd, ad, eb["code_offsets"], codes, sg["thresh"], prot_q,
                                           fpg["clip_idx"], scale_in=rg["scale"])
        ao = oracle.apply_plan(W, G, s, grid, actions, fpo["clip_idx"], thresh=so["thresh"], scale_in=ro["scale"])
        assert np.array_equal(ag["codes"][:n].cpu().numpy(), ao["codes"]) and np.array_equal(bits16(ag["wq"]), ao["wq"]), tag
        assert np.array_equal(ag["prot_offsets"].cpu().numpy(), ao["prot_offsets"]), tag
        assert np.array_equal(bits16(ag["prot_scale"]), ao["prot_scale"]), tag
        assert np.array_equal(ag["prot_q"][:ao["prot_q"].size].cpu().numpy(), ao["prot_q"]), tag
