"""GPU parity of the heuristic allocator's rule against the CPU oracle: ranking, actions and the
final total are integers and compared exactly, on the same score and count arrays."""
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


def run(wq, ctx, sal, n, g, target, headroom, p=None, sb=0, zb=0):
    dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a).astype(dt)).cuda()
    out = wq.windq_greedy_allocate(ctx, dev(sal, np.float32), dev(n, np.int64), dev(g, np.int64), target, headroom,
                                   None if p is None else dev(p, np.int64), scale_bits=sb, zero_bits=zb)
    torch.cuda.synchronize()
    return out["actions"].cpu().numpy(), out["order"].cpu().numpy(), int(out["total_centibits"].item())


def units(seed, U, ties=True):
    rng = np.random.default_rng(seed)
    G = rng.choice([32, 64, 128, 256], U)
    g = rng.integers(1, 5000, U)
    n = G * g
    p = (n * rng.choice([0.0, 0.02, 0.03, 0.5, 1.0], U, p=[0.2, 0.3, 0.4, 0.05, 0.05])).astype(np.int64)
    sal = rng.random(U).astype(np.float32)
    if ties:
        sal = rng.choice(sal[:max(1, U // 7)], U)
    return sal, n, g, p


def check(wq, ctx, oracle, sal, n, g, target, headroom, p, sb, zb):
    want = oracle.greedy_allocate(sal, n, g, target, headroom, n_protected=p, scale_bits=sb, zero_bits=zb)
    got = run(wq, ctx, sal, n, g, target, headroom, p, sb, zb)
    assert np.array_equal(got[1], want[1]), "ranking"
    assert np.array_equal(got[0], want[0]), "actions"
    assert got[2] == want[2]
    return want


@pytest.mark.parametrize("U", [1, 2, 31, 32, 33, 1023, 1024, 1025, 2049, 5000])
@pytest.mark.parametrize("target,headroom", [(200, 0), (218, 10), (150, 0), (100, 0), (90, 0), (300, 40), (450, 0), (230, 100)])
def test_rule_matches_oracle(wq, ctx, oracle, U, target, headroom):
    sal, n, g, p = units(31 * U + target, U)
    check(wq, ctx, oracle, sal, n, g, target, headroom, p, 16, 8)


def test_every_branch_is_reached(wq, ctx, oracle):
    """The cases above must between them produce every action the rule can give and both sweeps."""
    seen = set()
    for target, headroom in [(200, 0), (218, 10), (150, 0), (100, 0), (300, 40), (230, 100)]:
        sal, n, g, p = units(77 + target, 3000)
        want = check(wq, ctx, oracle, sal, n, g, target, headroom, p, 16, 16)
        seen |= set(want[0].tolist())
    assert seen == {2, 3, 4, 5, 6}


def test_no_protection_array_and_no_parameter_bits(wq, ctx, oracle):
    sal, n, g, _ = units(5, 4000, ties=False)
    check(wq, ctx, oracle, sal, n, g, 210, 15, None, 0, 0)


def test_signed_zeros_negative_and_infinite_scores(wq, ctx, oracle):
    sal = np.array([-1.0, 0.0, -0.0, 2.0, -np.inf, np.inf, 1e-45, -1e-45] * 40, np.float32)
    n = np.full(sal.size, 128 * 7)
    want = check(wq, ctx, oracle, sal, n, n // 128, 180, 0, None, 0, 0)
    assert want[1][:40].tolist() == list(range(5, 320, 8))


def test_model_sized_plan_from_measured_saliency(wq, ctx, oracle):
    """Units of the seven matrices of two 7B-shaped blocks at G = 128 with their measured scores and
    protected counts: the call chain a user of the allocator makes."""
    shapes = [(4096, 4096)] * 4 + [(11008, 4096)] * 2 + [(4096, 11008)]
    G = 128
    sal, n, g, p = [], [], [], []
    for i, (R, C) in enumerate(shapes * 2):
        R = R // 8                                   # fewer rows keep the test short; U per matrix is the full one
        W = ws.weights(R, C, 4000 + i, "student_t").cuda()
        s = torch.rand(C, generator=torch.Generator().manual_seed(i)).cuda() + 0.01
        sal.append(wq.windq_unit_saliency(ctx, W, G, s))
        sel = wq.windq_salient_select(ctx, W, G, s, 30000)
        p.append(sel["count"])
        U = C // G
        n.append(torch.full((U,), R * G, dtype=torch.int64))
        g.append(torch.full((U,), R, dtype=torch.int64))
    sal = torch.cat(sal).cpu().numpy()
    p = torch.cat(p).cpu().numpy()
    n, g = torch.cat(n).numpy(), torch.cat(g).numpy()
    want = check(wq, ctx, oracle, sal, n, g, 200, 10, p, 0, 0)
    N = int(n.sum())
    assert want[2] <= 200 * N
    assert (want[0] >= 5).any() and (want[0] <= 3).any()


def test_bad_counts_give_minus_one(wq, ctx):
    sal = np.ones(10, np.float32)
    n = np.full(10, 64)
    p = np.zeros(10, np.int64)
    p[3] = 65
    assert run(wq, ctx, sal, n, n // 32, 200, 0, p)[2] == -1


def test_argument_checks(wq, ctx):
    sal = torch.ones(4, device="cuda")
    n = torch.full((4,), 64, dtype=torch.int64, device="cuda")
    with pytest.raises(Exception):
        wq.windq_greedy_allocate(ctx, sal, n, n, 1601, 0)
    with pytest.raises(Exception):
        wq.windq_greedy_allocate(ctx, sal, n, n, 200, -1)
    with pytest.raises(Exception):
        wq.windq_greedy_allocate(ctx, sal, n[:3], n, 200, 0)


def test_all_scores_equal_and_two_distinct_scores(wq, ctx, oracle):
    """Every unit in one bucket of the ranking, and all units in the two end buckets."""
    _, n, g, p = units(9, 3000)
    check(wq, ctx, oracle, np.full(3000, 0.25, np.float32), n, g, 190, 5, p, 16, 8)
    sal = np.where(np.arange(3000) % 3 == 0, 1e-30, 3e38).astype(np.float32)
    check(wq, ctx, oracle, sal, n, g, 190, 5, p, 16, 8)


def test_quarter_of_a_million_units(wq, ctx, oracle):
    """More units than any bucket table entry count per bucket assumes: 262,144 units, scores spread over
    six decades with many repeats."""
    U = 262144
    rng = np.random.default_rng(12)
    sal = (10.0 ** rng.uniform(-4, 2, U)).astype(np.float32)
    sal[rng.integers(0, U, U // 10)] = sal[rng.integers(0, U, U // 10)]
    g = rng.integers(1, 64, U)
    n = g * 128
    p = (n * 0.03).astype(np.int64)
    check(wq, ctx, oracle, sal, n, g, 200, 10, p, 16, 16)
