"""The multi-GPU host logic on CPU: two gloo ranks shard the blocks of a model with no data-path
exchange, and the only cross-rank values (plan bits: int64 sum; step time: max) are reduced exactly.
Each rank runs the oracle's bit accounting on its own blocks' plans; the sum over ranks must equal
the single-process total."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _load_sharding():
    # the sharding helpers are plain torch.distributed code; load the file directly so that the
    # CUDA package (which builds and loads the library on import) is not needed on CPU
    import importlib.util
    spec = importlib.util.spec_from_file_location("windq_sharding", os.path.join(ROOT, "paper_2605_26660_b200", "sharding.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


N_BLOCKS, UNITS_PER_BLOCK, R, G = 7, 24, 64, 128


def _block_plan(block):
    rng = np.random.default_rng(1000 + block)
    return rng.integers(0, 7, UNITS_PER_BLOCK).astype(np.uint8)


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        sharding = _load_sharding()
        import oracle
        oracle.build()
        mine = sharding.block_range(N_BLOCKS, rank, world)
        local_cb, local_n = 0, 0
        for b in mine:
            eb = oracle.effective_bits(_block_plan(b), R, G)
            local_cb += int(eb["total_centibits"])
            local_n += UNITS_PER_BLOCK * R * G
        total_cb = sharding.sum_int64(local_cb)
        avg = sharding.average_bits(local_cb, local_n)
        slowest = sharding.max_float(10.0 + rank)
        np.save(os.path.join(out_dir, "rank%d.npy" % rank),
                np.array([total_cb, avg, slowest, len(mine), min(mine, default=-1), max(mine, default=-1)], np.float64))
    finally:
        dist.destroy_process_group()


def test_block_range_is_a_partition():
    sharding = _load_sharding()
    for n in (0, 1, 7, 32, 80):
        for world in (1, 2, 3, 8):
            seen = [b for r in range(world) for b in sharding.block_range(n, r, world)]
            assert seen == list(range(n))
            sizes = [len(sharding.block_range(n, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.block_range(4, 2, 2)


def test_reductions_without_a_process_group():
    sharding = _load_sharding()
    assert sharding.sum_int64(12345678901234) == 12345678901234
    assert sharding.max_float(1.5) == 1.5
    assert sharding.average_bits(2 * 100 * 1000, 1000) == 2.0


def test_two_gloo_ranks_agree_with_one_process(tmp_path, oracle):
    world = 2
    port = _free_port()
    mp.start_processes(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True, start_method="spawn")
    want_cb = sum(int(oracle.effective_bits(_block_plan(b), R, G)["total_centibits"]) for b in range(N_BLOCKS))
    want_avg = want_cb / (100.0 * N_BLOCKS * UNITS_PER_BLOCK * R * G)
    got = [np.load(os.path.join(str(tmp_path), "rank%d.npy" % r)) for r in range(world)]
    for g in got:
        assert int(g[0]) == want_cb                  # exact int64 sum
        assert g[1] == want_avg                      # b_bar = sum B_i / sum n_i over all ranks
        assert g[2] == 10.0 + (world - 1)            # step time = slowest rank
    assert sum(int(g[3]) for g in got) == N_BLOCKS   # every block scored exactly once
    assert int(got[0][5]) + 1 == int(got[1][4])      # contiguous, disjoint ranges


# ---- the allocator's rule over units that live on different ranks ------------------------------------
def _rank_units(rank):
    rng = np.random.default_rng(50 + rank)
    U = 40 + 13 * rank                                   # ranks hold different numbers of units
    g = rng.integers(8, 200, U)
    n = g * rng.choice([32, 64, 128], U)
    p = (n * 0.03).astype(np.int64)
    sal = rng.choice(rng.random(12).astype(np.float32), U)   # equal scores across ranks: ties by global index
    return sal, n, g, p


def _oracle_rule(oracle):
    def rule(sal, n, g, p):
        actions, _, total = oracle.greedy_allocate(sal.numpy(), n.numpy(), g.numpy(), 200, 10, n_protected=p.numpy(),
                                                   scale_bits=16, zero_bits=8)
        return dict(actions=torch.from_numpy(actions), total_centibits=total)
    return rule


def _alloc_worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        sharding = _load_sharding()
        import oracle
        oracle.build()
        sal, n, g, p = (torch.from_numpy(a) for a in _rank_units(rank))
        actions, total = sharding.allocate_across_ranks(_oracle_rule(oracle), sal, n, g, p)
        np.save(os.path.join(out_dir, "alloc%d.npy" % rank), np.concatenate([[total], actions.numpy().astype(np.int64)]))
    finally:
        dist.destroy_process_group()


def test_allocator_rule_over_two_ranks_equals_one_process(tmp_path, oracle):
    world = 2
    mp.start_processes(_alloc_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True, start_method="spawn")
    parts = [_rank_units(r) for r in range(world)]
    sal, n, g, p = (np.concatenate([q[i] for q in parts]) for i in range(4))
    want, _, want_total = oracle.greedy_allocate(sal, n, g, 200, 10, n_protected=p, scale_bits=16, zero_bits=8)
    pos = 0
    for r in range(world):
        got = np.load(os.path.join(str(tmp_path), "alloc%d.npy" % r))
        U = parts[r][0].size
        assert int(got[0]) == want_total
        assert np.array_equal(got[1:], want[pos:pos + U].astype(np.int64))
        pos += U
    assert {2, 3, 4, 5} & set(want.tolist())


def test_gather_units_without_a_process_group():
    sh = _load_sharding()
    a, b = torch.arange(5, dtype=torch.float32), torch.arange(5, dtype=torch.int64)
    (ga, gb), lo, hi = sh.gather_units(a, b)
    assert torch.equal(ga, a) and torch.equal(gb, b) and (lo, hi) == (0, 5)
    with pytest.raises(ValueError):
        sh.gather_units(a, b[:3])


# ---- activation statistics of an input whose tokens are split over the ranks ---------------------------
ACT_T, ACT_C = 96, 256


def _act_input():
    import windq_synth as ws
    return ws.activations(ACT_T, ACT_C, 61).numpy()


def _act_worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        sharding = _load_sharding()
        import oracle
        oracle.build()
        X = _act_input()
        lo, hi = (0, 40) if rank == 0 else (40, ACT_T)           # unequal slices
        s_local = torch.from_numpy(oracle.act_stats(X[lo:hi]))
        s = sharding.combine_act_stats(s_local, hi - lo)
        np.save(os.path.join(out_dir, "act%d.npy" % rank), s.numpy())
    finally:
        dist.destroy_process_group()


def test_token_sharded_act_stats_equal_the_whole_input(tmp_path, oracle):
    world = 2
    mp.start_processes(_act_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True, start_method="spawn")
    want = oracle.act_stats(_act_input())
    got = [np.load(os.path.join(str(tmp_path), "act%d.npy" % r)) for r in range(world)]
    assert np.array_equal(got[0], got[1])                       # every rank holds the same statistic
    assert np.allclose(got[0], want, rtol=1e-6, atol=0)


# ---- the whole path of a small model, its blocks split over two ranks --------------------------------------
def _tiny_spec():
    import windq_synth as ws
    return ws.ModelSpec("tiny", 4, 256, 384, 128, "student_t", 64, 6, (64,))


def _score_blocks(oracle, spec, blocks):
    """The oracle's path over `blocks`: per unit the error table, the energy, the saliency score and the counts the
    allocator needs (units in block order, then matrix order)."""
    import windq_synth as ws
    G = spec.chunk_widths[0]
    grid = ws.clip_grid(spec.K)
    err, energy, sal, nw, ng = [], [], [], [], []
    for b in blocks:
        stats = {i: oracle.act_stats(ws.block_input(spec, 0, b, i).numpy()) for i, _ in spec.block_inputs()}
        for m in spec.block_matrices():
            W = ws.block_weight(spec, 0, b, m).numpy()
            fit = oracle.fit_eval(W, G, stats[m.x_id], grid, want_group_err=False)
            err.append(fit["err"])
            energy.append(fit["energy"])
            sal.append(oracle.unit_saliency(W, G, stats[m.x_id]))
            nw.append(np.full(m.C // G, m.R * G, np.int64))
            ng.append(np.full(m.C // G, m.R, np.int64))
    if not err:
        return (np.zeros((0, 6), np.float32), np.zeros(0, np.float32), np.zeros(0, np.float32), np.zeros(0, np.int64),
                np.zeros(0, np.int64))
    return np.concatenate(err), np.concatenate(energy), np.concatenate(sal), np.concatenate(nw), np.concatenate(ng)


def _tiny_rule(oracle):
    def rule(sal, n, g, p):
        actions, _, total = oracle.greedy_allocate(sal.numpy(), n.numpy(), g.numpy(), 200, 10, scale_bits=16, zero_bits=16)
        return dict(actions=torch.from_numpy(actions), total_centibits=total)
    return rule


def _path_worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        sharding = _load_sharding()
        import oracle
        oracle.build()
        spec = _tiny_spec()
        mine = sharding.block_range(spec.n_blocks, rank, world)
        err, energy, sal, nw, ng = _score_blocks(oracle, spec, mine)
        table = sharding.gather_rows(torch.from_numpy(err))                       # the model's error table on every rank
        actions, total = sharding.allocate_across_ranks(_tiny_rule(oracle), torch.from_numpy(sal), torch.from_numpy(nw),
                                                        torch.from_numpy(ng))
        # bit accounting of this rank's slice of the plan, summed exactly over the ranks
        G = spec.chunk_widths[0]
        local_cb, pos = 0, 0
        for b in mine:
            for m in spec.block_matrices():
                U = m.C // G
                local_cb += int(oracle.effective_bits(actions[pos:pos + U].numpy(), m.R, G)["total_centibits"])
                pos += U
        np.savez(os.path.join(out_dir, "path%d.npz" % rank), table=table.numpy(), actions=actions.numpy(),
                 total=np.int64(total), summed=np.int64(sharding.sum_int64(local_cb)), n_blocks=len(mine))
    finally:
        dist.destroy_process_group()


def test_whole_path_over_two_ranks_equals_one_process(tmp_path, oracle):
    """Strong scaling on the host side: the four blocks of a small model split over two ranks, each rank running the
    path on its blocks only; the gathered error table, the plan of the heuristic allocator and the plan's total bits
    are those of one process over the whole model."""
    world = 2
    mp.start_processes(_path_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True, start_method="spawn")
    spec = _tiny_spec()
    err, energy, sal, nw, ng = _score_blocks(oracle, spec, range(spec.n_blocks))
    want_actions, _, want_total = oracle.greedy_allocate(sal, nw, ng, 200, 10, scale_bits=16, zero_bits=16)
    got = [np.load(os.path.join(str(tmp_path), "path%d.npz" % r)) for r in range(world)]
    pos = 0
    for g in got:
        assert np.array_equal(g["table"].view(np.uint32), err.view(np.uint32))    # same bits: units are independent
        n = g["actions"].size
        assert np.array_equal(g["actions"], want_actions[pos:pos + n])
        pos += n
        assert int(g["total"]) == want_total and int(g["summed"]) == want_total
    assert pos == want_actions.size and sum(int(g["n_blocks"]) for g in got) == spec.n_blocks
