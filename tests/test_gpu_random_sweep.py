"""Randomised parity sweep on the GPU: random shapes, chunk widths, grid sizes, weight and statistic distributions
(zeros, one-sided, ties, sparse, fp16 subnormals, outlier columns, statistics spanning 20 decades) through the whole
chain -- features, fits, plan packing, salient selection, protected fits, refinement, protected and refined packing --
against the oracle.  Integer and bit-pattern outputs are compared exactly."""
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
