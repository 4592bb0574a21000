"""windq_apply_plan_multi (several plans of one matrix in one pass over its weights) through the C ABI: every plan's
outputs equal those of its own windq_apply_plan call and of the CPU oracle, bit for bit."""
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


def u16(t):
    return t.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("G,R,C,n_plans", [(128, 300, 1024, 3), (64, 133, 512, 4), (32, 200, 256, 2), (256, 19, 2048, 3),
                                           (512, 67, 1024, 4), (128, 3, 896, 1), (128, 1100, 512, 3)])
def test_multi_equals_separate_calls_and_the_oracle(wq, ctx, oracle, G, R, C, n_plans):
    W = ws.weights(R, C, 800 + G + R, "student_t")
    s = oracle.act_stats(ws.activations(96, C, 801 + G).numpy())
    grid = ws.clip_grid(20)
    U = C // G
    Wd, sd, gd = W.cuda(), torch.from_numpy(s).cuda(), torch.from_numpy(grid).cuda()
    fit = wq.windq_fit_eval(ctx, Wd, G, sd, gd)
    rng = np.random.default_rng(G + R)
    plans, singles, acts_np = [], [], []
    for p in range(n_plans):
        acts = rng.integers(0, 7, U).astype(np.uint8)
        if p == 0:
            acts[:7] = np.arange(7)[:min(7, U)] if U >= 7 else acts[:7]
        acts_np.append(acts)
        a_d = torch.from_numpy(acts).cuda()
        eb = wq.windq_effective_bits(ctx, a_d, R, G)
        n = int(eb["code_offsets"][-1].item())
        plans.append(dict(actions=a_d, code_offsets=eb["code_offsets"], codes=torch.full((n,), 0xEE, dtype=torch.uint8, device="cuda")))
        singles.append(wq.windq_apply_plan(ctx, Wd, G, sd, gd, a_d, eb["code_offsets"],
                                           torch.full((n,), 0xDD, dtype=torch.uint8, device="cuda"), fit["clip_idx"]))
    if n_plans > 1:
        plans[-1]["wq"] = None                      # a plan without fake-quantised output
    got = wq.windq_apply_plan_multi(ctx, Wd, G, sd, gd, fit["clip_idx"], plans)
    torch.cuda.synchronize()
    assert len(got) == n_plans
    clip_h = fit["clip_idx"].cpu().numpy()
    for p, (out, one) in enumerate(zip(got, singles)):
        assert torch.equal(out["codes"], one["codes"]), p
        assert torch.equal(out["scales"].view(torch.int16), one["scales"].view(torch.int16)), p
        assert torch.equal(out["zeros"].view(torch.int16), one["zeros"].view(torch.int16)), p
        if out["wq"] is None:
            assert n_plans > 1 and p == n_plans - 1
        else:
            assert torch.equal(out["wq"].view(torch.int16), one["wq"].view(torch.int16)), p
        want = oracle.apply_plan(W.numpy(), G, s, grid, acts_np[p], clip_h)
        assert np.array_equal(out["codes"].cpu().numpy(), want["codes"]), p
        assert np.array_equal(u16(out["scales"]), want["scales"]) and np.array_equal(u16(out["zeros"]), want["zeros"]), p
        if out["wq"] is not None:
            assert np.array_equal(u16(out["wq"]), want["wq"]), p


def test_multi_on_a_full_size_matrix_with_the_benchmark_plans(wq, ctx, oracle):
    """up_proj of the 7B-shaped model with plans at 1.58 / 2.0 / 3.0 bits in one call: equal to three separate calls,
    sampled units equal to the oracle."""
    spec = ws.CONFIGS["cfg3_llama7b_model"]
    m = spec.block_matrices()[5]
    G, U = 128, m.C // 128
    W = ws.block_weight(spec, 0, 0, m, device="cuda")
    s = wq.windq_act_stats(ctx, ws.block_input(spec, 0, 0, m.x_id, device="cuda"))
    grid = ws.clip_grid(spec.K)
    gd = torch.from_numpy(grid).cuda()
    fit = wq.windq_fit_eval(ctx, W, G, s, gd)
    per_action = wq.windq_effective_bits(ctx, torch.arange(7, dtype=torch.uint8, device="cuda"), m.R, G)["unit_centibits"].cpu().numpy()
    costs = np.tile(per_action[None, :], (U, 1))
    plans, singles, acts_np = [], [], []
    for ti, target in enumerate((1.58, 2.0, 3.0)):
        acts = ws.random_plan(costs, np.full(U, m.R * G, np.int64), target, 40 + ti)
        acts_np.append(acts)
        a_d = torch.from_numpy(acts).cuda()
        eb = wq.windq_effective_bits(ctx, a_d, m.R, G)
        n = int(eb["code_offsets"][-1].item())
        plans.append(dict(actions=a_d, code_offsets=eb["code_offsets"], codes=torch.empty(n, dtype=torch.uint8, device="cuda")))
        singles.append(wq.windq_apply_plan(ctx, W, G, s, gd, a_d, eb["code_offsets"], torch.empty(n, dtype=torch.uint8, device="cuda"),
                                           fit["clip_idx"]))
    got = wq.windq_apply_plan_multi(ctx, W, G, s, gd, fit["clip_idx"], plans)
    torch.cuda.synchronize()
    s_h = s.cpu().numpy()
    for p, (out, one) in enumerate(zip(got, singles)):
        for k in ("codes", "scales", "zeros", "wq"):
            assert torch.equal(out[k].view(torch.uint8), one[k].view(torch.uint8)), (p, k)
        offs = plans[p]["code_offsets"].cpu().numpy()
        for u in (0, 17, 31):
            want = oracle.apply_plan(W[:, u * G:(u + 1) * G].cpu().numpy(), G, s_h[u * G:(u + 1) * G], grid, acts_np[p][u:u + 1],
                                     fit["clip_idx"][:, u:u + 1].cpu().numpy())
            assert np.array_equal(out["codes"][offs[u]:offs[u + 1]].cpu().numpy(), want["codes"])
            assert np.array_equal(u16(out["wq"][:, u * G:(u + 1) * G]), want["wq"])


def test_multi_argument_checks(wq, ctx):
    gd = torch.from_numpy(ws.clip_grid(4)).cuda()
    W = torch.zeros((8, 128), dtype=torch.float16, device="cuda")
    s = torch.ones(128, device="cuda")
    acts = torch.zeros(1, dtype=torch.uint8, device="cuda")
    eb = wq.windq_effective_bits(ctx, acts, 8, 128)
    idx = torch.zeros((4, 1, 8), dtype=torch.uint8, device="cuda")

    def plan():
        return dict(actions=acts, code_offsets=eb["code_offsets"], codes=torch.zeros(4096, dtype=torch.uint8, device="cuda"), wq=None)
    with pytest.raises(wq.WindqError) as e:
        wq.windq_apply_plan_multi(ctx, W, 128, s, gd, idx, [plan() for _ in range(5)])
    assert e.value.status == 2
    shared = plan()
    with pytest.raises(wq.WindqError) as e:
        wq.windq_apply_plan_multi(ctx, W, 128, s, gd, idx, [shared, dict(shared)])          # two plans, one codes array
    assert e.value.status == 4
    out = wq.windq_apply_plan_multi(ctx, W, 128, s, gd, idx, [plan(), plan()])
    torch.cuda.synchronize()
    assert out[0]["wq"] is None and bool((out[0]["codes"][:2048] == 0).all())


@pytest.mark.parametrize("G,shapes", [(128, [(300, 1024), (1100, 512)]), (64, [(133, 512), (40, 256)]), (32, [(200, 256)]),
                                      (256, [(19, 2048)]), (512, [(67, 1024)])])
def test_low_bit_parameters_from_the_fit_give_the_same_plans(wq, ctx, oracle, G, shapes):
    """windq_fit_eval_batch can leave the scales (and the 1.58-bit threshold) of its two low-bit fits in a table that
    windq_apply_plan_multi takes in place of forming the sums again: every output equals the call without the table,
    and the table's scales are the oracle's."""
    grid = ws.clip_grid(20)
    gd = torch.from_numpy(grid).cuda()
    Ws = [ws.weights(R, C, 860 + i, "student_t").cuda() for i, (R, C) in enumerate(shapes)]
    for W in Ws:
        W[::5, :G] = 0                              # some all-zero groups (empty support)
    ss = [(torch.rand(C, generator=torch.Generator().manual_seed(i)) * 3).cuda() for i, (R, C) in enumerate(shapes)]
    for s in ss:
        s[G // 2:G] = 0                             # and groups whose support may carry no activation weight
    fits = wq.windq_fit_eval_batch(ctx, Ws, G, ss, gd, want_lowbit=True)
    rng = np.random.default_rng(G)
    for W, s, fit in zip(Ws, ss, fits):
        R, C = W.shape
        U = C // G
        plans_a, plans_b, acts_np = [], [], []
        for p in range(3):
            acts = rng.choice([5, 6, 5, 6, 4, 0, 2], U).astype(np.uint8)
            acts_np.append(acts)
            a_d = torch.from_numpy(acts).cuda()
            eb = wq.windq_effective_bits(ctx, a_d, R, G)
            n = int(eb["code_offsets"][-1].item())
            for plans in (plans_a, plans_b):
                plans.append(dict(actions=a_d, code_offsets=eb["code_offsets"], codes=torch.full((n,), 0xEE, dtype=torch.uint8, device="cuda")))
        with_table = wq.windq_apply_plan_multi(ctx, W, G, s, gd, fit["clip_idx"], plans_a, lowbit=fit["lowbit"])
        without = wq.windq_apply_plan_multi(ctx, W, G, s, gd, fit["clip_idx"], plans_b)
        torch.cuda.synchronize()
        for a, b in zip(with_table, without):
            for k in ("codes", "scales", "zeros", "wq"):
                assert torch.equal(a[k].view(torch.uint8), b[k].view(torch.uint8)), k
        want = oracle.apply_plan(W.cpu().numpy(), G, s.cpu().numpy(), grid, np.full(U, 5, np.uint8), fit["clip_idx"].cpu().numpy())
        assert np.array_equal(u16(fit["lowbit"][0]), want["scales"])
        want = oracle.apply_plan(W.cpu().numpy(), G, s.cpu().numpy(), grid, np.full(U, 6, np.uint8), fit["clip_idx"].cpu().numpy())
        assert np.array_equal(u16(fit["lowbit"][1]), want["scales"])
