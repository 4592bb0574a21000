"""windq_act_stats_noalloc against windq_act_stats, through the C ABI.

The no-allocation entry point serves hosts that cannot call cudaMalloc when a statistic is needed
(all device memory already handed to their own pool, or a loop that cannot take the device-wide
synchronisation an allocation implies).  Its partial sums live in one array built into the
library, shared by every call and never cleared, so the test makes two calls in a row with
different shapes and data -- the second smaller than the first, so that anything it wrongly picked
up from the first call's leftovers would show -- and compares each with the allocating entry
point.  This file is named to be collected last: a run that stops at the first failure has then
already run every other test.
"""
import pytest
import torch

import windq_synth as ws

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-4, 1e-6


@pytest.fixture(scope="module")
def wq():
    import paper_2605_26660_b200 as wq
    return wq


def test_noalloc_matches_act_stats_on_two_calls_in_a_row(wq, oracle):
    ctx = wq.windq_create(0)
    try:
        for T, C, seed in ((700, 1480, 11), (130, 264, 12)):
            X = ws.activations(T, C, seed)
            Xd = X.cuda()
            want = wq.windq_act_stats(ctx, Xd)
            got = torch.full((C,), float("nan"), dtype=torch.float32, device="cuda")
            wq.windq_act_stats_noalloc(ctx, Xd, got)
            torch.cuda.synchronize()
            assert bool((torch.abs(got - want) <= RTOL * torch.abs(want) + ATOL).all()), (T, C)
            ref = torch.from_numpy(oracle.act_stats(X.numpy())).cuda()      # and against the CPU oracle directly
            assert bool((torch.abs(got - ref) <= RTOL * torch.abs(ref) + ATOL).all()), (T, C)
    finally:
        wq.windq_destroy(ctx)


def test_noalloc_refuses_what_does_not_fit(wq):
    ctx = wq.windq_create(0)
    try:
        T, C = 4096, 28672                       # 64 slices x 28672 channels x 4 bytes = 7.3 MB > 4 MB
        assert wq.windq_scratch_bytes_act_stats(T, C) > wq.NOALLOC_SCRATCH_BYTES
        X = torch.zeros((T, C), dtype=torch.float16, device="cuda")
        out = torch.full((C,), -1.0, dtype=torch.float32, device="cuda")
        with pytest.raises(wq.WindqError) as e:
            wq.windq_act_stats_noalloc(ctx, X, out)
        assert e.value.status == 5 and "built-in array" in str(e.value)
        torch.cuda.synchronize()
        assert bool((out == -1.0).all())         # nothing was launched
    finally:
        wq.windq_destroy(ctx)
