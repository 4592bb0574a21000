#!/usr/bin/env python
"""Benchmark of the WINDQuant scoring path on B200.

    python bench.py --gpus N --steps K --warmup W            # this library (CUDA, C ABI)
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands

A step is one pass of the whole hot path over a LLaMA-7B-shaped model of synthetic weights and
calibration activations (32 decoder blocks; see windq_synth.CONFIGS): per block act_stats of its inputs;
per matrix and chunk width (64, 128) unit_features + fit_eval over every unit; then, at chunk
width 128, effective_bits + apply_plan for three seeded random plans (1.58, 2.0, 3.0 bits).
The metric is unit x bit-width candidate evaluations per second (6 per unit and chunk width).

`value` is measured with the inputs resident in HBM; `e2e` runs the same step from pinned host
memory, host-to-device copies of every weight and activation and device-to-host copies of every
result (error tables, features, packed codes, scales, zero points) inside the timed region.
With N > 1 (torchrun) every rank scores its own replica of the model: weak scaling, no
data-path collective; time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import windq_synth as ws

METRIC = "unit_x_bitwidth_candidate_evals_per_s"
UNIT = "evals/s"
TARGET_BITS = (1.58, 2.0, 3.0)
APPLY_G = 128                    # chunk width the plans are applied at (the first of the workload's widths if it has no 128)
# measured DRAM bytes (read + written) per byte of weights, from the ncu captures summarised under profiles/:
# one 4096 x 4096 matrix per launch (outputs stay in L2), and the seven matrices of a 7B-shaped block per launch
# (mean of the captures at chunk widths 64 and 128)
FIT_TRAFFIC_PER_WEIGHT_BYTE = {False: None, True: (434.4 + 437.0) / 2 / 404.75}   # None: no capture of the kernel as it stands
SEED = 0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="windq", choices=["windq", "reference"])
    ap.add_argument("--workload", default="cfg3_llama7b_model", choices=sorted(ws.CONFIGS))
    ap.add_argument("--blocks", type=int, default=0, help="score only the first B blocks of the model (0 = all)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="with N > 1 ranks: weak = a replica of the model per rank; strong = the blocks of ONE model split over the ranks")
    ap.add_argument("--stream", default="auto", choices=["auto", "yes", "no"],
                    help="keep two blocks on the device and refill them block by block instead of holding the model resident "
                         "(auto: when the model does not fit in half of the free device memory)")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--separate-fits", action="store_true",
                    help="one windq_unit_features and one windq_fit_eval call per matrix instead of one batched call of each per "
                         "block and chunk width")
    ap.add_argument("--fused-features", action="store_true",
                    help="features and fits of a block by one windq_features_fit_batch call (one pass over the weights; "
                         "measured slower than the two batched calls, kept for comparison)")
    ap.add_argument("--separate-plans", action="store_true",
                    help="one windq_apply_plan call per plan instead of one windq_apply_plan_multi call per matrix")
    ap.add_argument("--extras", action="store_true",
                    help="also time the calls beyond the five of a step (protection, refinement, allocator) on block 0")
    return ap.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return dict(hbm_gbs=float(p["hbm_gbs"]), sm_max_mhz=float(p.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=6650.0, sm_max_mhz=1965.0, source="fallback")


# ---------------------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def __enter__(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if not self.path or not os.path.exists(self.path):
            return out
        sm, mx, reasons = [], [], set()
        with open(self.path) as fh:
            for line in fh:
                t = [x.strip() for x in line.split(",")]
                if len(t) < 9:
                    continue
                try:
                    sm.append(float(t[1]))
                    mx.append(float(t[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), t[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if sm:
            busy = [x for x in sm if x > 0.5 * max(mx)] or sm
            out = dict(sm_mhz=float(np.median(busy)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


# ---------------------------------------------------------------------------------------- workload
def matrices_of(spec):
    return [m for m in spec.block_matrices() if m.R > 0 and m.C > 0]


def inputs_of(spec):
    used = {m.x_id for m in matrices_of(spec)}
    return [(i, c) for i, c in spec.block_inputs() if i in used]


def workload_counts(spec, n_blocks):
    mats = matrices_of(spec)
    elems = sum(m.R * m.C for m in mats) * n_blocks
    units = {G: sum(m.C // G for m in mats) * n_blocks for G in spec.chunk_widths}
    return elems, units


def fit_ops_per_element(K):
    """Algorithmic binary32 lane operations per weight element (fma = 1): seven per (bit-width, clip
    ratio) candidate of the four uniform bit-widths, plus about ten once per element."""
    return 28 * K + 10


class DeviceModel:
    """Weights and calibration inputs of this rank's blocks in HBM: all of them resident, or -- streamed -- two block
    slots that are refilled block by block (the synthetic block is regenerated on the device from its seed, which
    stands for the layer-by-layer load of a model larger than the GPU's memory; the refill is not part of the timed
    kernels)."""

    def __init__(self, spec, blocks, seed, streamed=False):
        self.spec, self.blocks, self.seed, self.streamed = spec, list(blocks), seed, streamed
        self.W, self.X = [], []
        self.slot_block = [None, None]
        for b in (self.blocks[:2] if streamed else self.blocks):
            self.W.append([ws.block_weight(spec, seed, b, m, device="cuda") for m in matrices_of(spec)])
            self.X.append({i: ws.block_input(spec, seed, b, i, device="cuda") for i, _ in inputs_of(spec)})
        if streamed:
            self.slot_block = list(self.blocks[:2]) + [None] * (2 - len(self.blocks[:2]))
        torch.cuda.synchronize()

    def block(self, bi):
        """(weights, inputs) of this rank's bi-th block; a streamed model regenerates it into slot bi % 2 first."""
        if not self.streamed:
            return self.W[bi], self.X[bi]
        slot, b = bi % 2, self.blocks[bi]
        if self.slot_block[slot] != b:
            for dst, m in zip(self.W[slot], matrices_of(self.spec)):
                dst.copy_(ws.block_weight(self.spec, self.seed, b, m, device="cuda"))
            for i in self.X[slot]:
                self.X[slot][i].copy_(ws.block_input(self.spec, self.seed, b, i, device="cuda"))
            self.slot_block[slot] = b
        return self.W[slot], self.X[slot]


def make_plans(wq, ctx, spec, n_blocks, G):
    """Seeded random plans for the three target bit-widths; returns {target: [[actions per matrix] per block]}."""
    mats = matrices_of(spec)
    costs, nw = [], []
    all_actions = torch.arange(7, dtype=torch.uint8, device="cuda")
    per_R = {}
    for m in mats:
        if m.R not in per_R:
            per_R[m.R] = wq.windq_effective_bits(ctx, all_actions, m.R, G)["unit_centibits"].cpu().numpy()
    for _ in range(n_blocks):
        for m in mats:
            U = m.C // G
            costs.append(np.tile(per_R[m.R][None, :], (U, 1)))
            nw.append(np.full(U, m.R * G, np.int64))
    costs, nw = np.concatenate(costs), np.concatenate(nw)
    plans = {}
    for ti, target in enumerate(TARGET_BITS):
        flat = ws.random_plan(costs, nw, target, SEED * 7919 + ti)
        per_block, pos = [], 0
        for _ in range(n_blocks):
            row = []
            for m in mats:
                U = m.C // G
                row.append(torch.from_numpy(flat[pos:pos + U].copy()).cuda())
                pos += U
            per_block.append(row)
        plans[target] = per_block
    return plans


class Buffers:
    """Output tensors sized for the largest matrix, reused for every matrix (a consumer would keep
    what it needs); nothing is allocated inside a step.  Every output that the e2e leg copies to the
    host exists `ring` times and the calls write them in turn, so that a device-to-host copy on another
    stream can still be reading one result while the next one is produced."""

    RINGED = ("feat", "err", "energy", "totals", "codes", "scales", "zeros")

    def __init__(self, spec, ring=1):
        mats = matrices_of(spec)
        Gmin = min(spec.chunk_widths)
        maxU = max(m.C // Gmin for m in mats)
        maxRC = max(m.R * m.C for m in mats)
        maxUR = max((m.C // Gmin) * m.R for m in mats)
        dev = "cuda"
        self.ring = ring
        self.s = {i: torch.empty(c, dtype=torch.float32, device=dev) for i, c in inputs_of(spec)}
        self.clip_idx = torch.empty(4 * maxUR, dtype=torch.uint8, device=dev)
        self.unit_cb = torch.empty(maxU, dtype=torch.int64, device=dev)
        self.offsets = torch.empty(maxU + 1, dtype=torch.int64, device=dev)
        self.wq = torch.empty(maxRC, dtype=torch.float16, device=dev)
        self.wq_multi = [self.wq] + [torch.empty(maxRC, dtype=torch.float16, device=dev) for _ in TARGET_BITS[1:]]
        shapes = dict(feat=(maxU * 8, torch.float32), err=(maxU * 6, torch.float32), energy=(maxU, torch.float32),
                      totals=(2 * len(TARGET_BITS), torch.int64), codes=(2 * maxRC + 16 * maxU, torch.uint8),
                      scales=(maxUR, torch.float16), zeros=(maxUR, torch.float16))
        # one set of fit outputs per matrix of a block, for the batched fit (all matrices of a block in one call)
        for mi, m in enumerate(mats):
            shapes["feat%d" % mi] = ((m.C // Gmin) * 8, torch.float32)
            shapes["featw%d" % mi] = ((m.C // Gmin) * 8, torch.float32)
            shapes["totals%d" % mi] = (2 * len(TARGET_BITS), torch.int64)
            shapes["err%d" % mi] = ((m.C // Gmin) * 6, torch.float32)
            shapes["energy%d" % mi] = (m.C // Gmin, torch.float32)
        self.clip_idx_m = [torch.empty(4 * (m.C // Gmin) * m.R, dtype=torch.uint8, device=dev) for m in mats]
        self.lowbit_m = [torch.empty(3 * (m.C // Gmin) * m.R, dtype=torch.float16, device=dev) for m in mats]
        self.offsets_m = [[torch.empty(m.C // Gmin + 1, dtype=torch.int64, device=dev) for _ in TARGET_BITS] for m in mats]
        self.rings = {k: [torch.zeros(n, dtype=dt, device=dev) for _ in range(ring)] for k, (n, dt) in shapes.items()}
        self.turn = {k: 0 for k in shapes}
        self.pending = {}          # (name, slot) -> event of the copy that still reads that slot
        self.last = {}             # name -> slot handed out last

    def take(self, name):
        """The tensor the next call writes `name` into; waits (on the current stream) for a copy that still reads it."""
        slot = self.turn[name] % self.ring
        self.turn[name] += 1
        ev = self.pending.pop((name, slot), None)
        if ev is not None:
            torch.cuda.current_stream().wait_event(ev)
        self.last[name] = slot
        return self.rings[name][slot]

    @property
    def totals(self):
        """The totals written last (those of the block's last matrix when a block is accounted in one launch)."""
        name = "totals%d" % (len(self.clip_idx_m) - 1) if BATCH_FITS else "totals"
        return self.rings[name][self.last.get(name, 0)]


class FitTimer:
    """CUDA events around every windq_fit_eval call of the timed steps (on the launching stream)."""

    def __init__(self):
        self.pairs = []

    def start(self):
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        return e

    def stop(self, e0):
        e1 = torch.cuda.Event(enable_timing=True)
        e1.record()
        self.pairs.append((e0, e1))

    def total_ms(self):
        return sum(a.elapsed_time(b) for a, b in self.pairs)


BATCH_FITS = True      # one windq_fit_eval_batch call per block and chunk width (False: one windq_fit_eval per matrix)
MULTI_APPLY = True     # the plans of a matrix packed by one windq_apply_plan_multi call (False: one windq_apply_plan per plan)
FUSED_FEATURES = False # features and fits of a block by one windq_features_fit_batch call


def jobs_slot(buf, name, ti):
    """Ring slot that plan ti of the matrix just packed wrote `name` into (the last len(TARGET_BITS) slots handed out)."""
    return (buf.turn[name] - len(TARGET_BITS) + ti) % buf.ring


def apply_plans(wq, ctx, spec, m, mi, W, s, G, clip_idx, plans_b, buf, grid_d, sink, accounted=None, lowbit=None):
    """The three plans of one matrix: bit accounting (unless `accounted` = (totals, [code offsets per plan]) holds
    it already), then packing.  Returns the number of kernels launched."""
    U, launches = m.C // G, 0
    totals = accounted[0] if accounted else buf.take("totals")
    if accounted and MULTI_APPLY:
        # one pass over the matrix for all plans (windq_apply_plan_multi): every weight is read once
        jobs = []
        for ti, target in enumerate(TARGET_BITS):
            jobs.append(dict(actions=plans_b[target][mi], code_offsets=accounted[1][ti], codes=buf.take("codes"),
                             scales=buf.take("scales")[:U * m.R].view(U, m.R), zeros=buf.take("zeros")[:U * m.R].view(U, m.R),
                             wq=buf.wq_multi[ti][:m.R * m.C].view(m.R, m.C)))
        outs = wq.windq_apply_plan_multi(ctx, W, G, s, grid_d, clip_idx, jobs, lowbit=lowbit)
        if sink:
            for ti, target in enumerate(TARGET_BITS):
                sink("codes", (outs[ti]["codes"], plans_b[target][mi], m.R, G), slot=jobs_slot(buf, "codes", ti))
                sink("scales", outs[ti]["scales"], slot=jobs_slot(buf, "scales", ti))
                sink("zeros", outs[ti]["zeros"], slot=jobs_slot(buf, "zeros", ti))
            sink("totals%d" % mi, totals)
        return 1
    for ti, target in enumerate(TARGET_BITS):
        acts = plans_b[target][mi]
        if accounted:
            eb = dict(code_offsets=accounted[1][ti])
            launches -= 1
        else:
            eb = wq.windq_effective_bits(ctx, acts, m.R, G, out=dict(
                unit_centibits=buf.unit_cb[:U], code_offsets=buf.offsets[:U + 1],
                total_centibits=totals[2 * ti:2 * ti + 1], total_packed_bytes=totals[2 * ti + 1:2 * ti + 2]))
        plan = wq.windq_apply_plan(ctx, W, G, s, grid_d, acts, eb["code_offsets"], buf.take("codes"), clip_idx,
                                   out=dict(scales=buf.take("scales")[:U * m.R].view(U, m.R),
                                            zeros=buf.take("zeros")[:U * m.R].view(U, m.R),
                                            wq=buf.wq[:m.R * m.C].view(m.R, m.C)))
        launches += 2
        if sink:
            sink("codes", (plan["codes"], acts, m.R, G))
            sink("scales", plan["scales"])
            sink("zeros", plan["zeros"])
    if sink:
        sink("totals%d" % mi if accounted else "totals", totals)
    return launches


def score_block(wq, ctx, spec, Wb, Xb, plans_b, buf, grid_d, timer=None, sink=None):
    """The whole hot path for one block.  Returns the number of kernels launched.  `sink(name, tensor)`
    receives every result (the e2e leg copies them to the host)."""
    launches = 0
    mats = matrices_of(spec)
    ids = sorted(Xb)
    wq.windq_act_stats_batch(ctx, [Xb[i] for i in ids], [buf.s[i] for i in ids])
    launches += 1
    if BATCH_FITS:
        # chunk widths G and 2 G: the features of both come out of one pass at G (windq_unit_features_batch2)
        nested = (not FUSED_FEATURES and len(spec.chunk_widths) == 2 and spec.chunk_widths[1] == 2 * spec.chunk_widths[0]
                  and all(m.C % spec.chunk_widths[1] == 0 for m in mats))
        wide_feats = None
        for G in spec.chunk_widths:
            stats = [buf.s[m.x_id] for m in mats]
            if nested and G == spec.chunk_widths[1]:
                feats = wide_feats
            else:
                feats = [buf.take("feat%d" % mi)[:(m.C // G) * 8].view(m.C // G, 8) for mi, m in enumerate(mats)]
            if nested and G == spec.chunk_widths[0]:
                wide_feats = [buf.take("featw%d" % mi)[:(m.C // (2 * G)) * 8].view(m.C // (2 * G), 8) for mi, m in enumerate(mats)]
                wq.windq_unit_features_batch(ctx, Wb, G, stats, feats, feats_2G=wide_feats)
                launches += 3
            elif not FUSED_FEATURES and not nested:
                wq.windq_unit_features_batch(ctx, Wb, G, stats, feats)
                launches += 2
            outs = [dict(err=buf.take("err%d" % mi)[:(m.C // G) * 6].view(m.C // G, 6),
                         energy=buf.take("energy%d" % mi)[:m.C // G],
                         clip_idx=buf.clip_idx_m[mi][:4 * (m.C // G) * m.R].view(4, m.C // G, m.R),
                         lowbit=buf.lowbit_m[mi][:3 * (m.C // G) * m.R].view(3, m.C // G, m.R) if (MULTI_APPLY and G == APPLY_G) else None)
                    for mi, m in enumerate(mats)]
            e0 = timer.start() if timer else None
            if FUSED_FEATURES:
                wq.windq_features_fit_batch(ctx, Wb, G, stats, grid_d, feats=feats, outs=outs)
                launches += 1
            else:
                wq.windq_fit_eval_batch(ctx, Wb, G, stats, grid_d, outs=outs)
            if timer:
                timer.stop(e0)
            launches += 2
            if sink:
                for mi in range(len(mats)):
                    sink("featw%d" % mi if (nested and G == spec.chunk_widths[1]) else "feat%d" % mi, feats[mi])
            if sink:
                for mi in range(len(mats)):
                    sink("err%d" % mi, outs[mi]["err"])
                    sink("energy%d" % mi, outs[mi]["energy"])
            if G == APPLY_G and plans_b:
                # the bit accounting of the block's 21 (matrix, plan) pairs in one launch
                totals = [buf.take("totals%d" % mi) for mi in range(len(mats))]
                offs = [[buf.offsets_m[mi][ti][:m.C // G + 1] for ti in range(len(TARGET_BITS))] for mi, m in enumerate(mats)]
                wq.windq_effective_bits_batch(
                    ctx, [plans_b[target][mi] for mi in range(len(mats)) for target in TARGET_BITS],
                    [m.R for m in mats for _ in TARGET_BITS], G,
                    outs=[dict(unit_centibits=None, code_offsets=offs[mi][ti], total_centibits=totals[mi][2 * ti:2 * ti + 1],
                               total_packed_bytes=totals[mi][2 * ti + 1:2 * ti + 2])
                          for mi in range(len(mats)) for ti in range(len(TARGET_BITS))])
                launches += 1
                for mi, m in enumerate(mats):
                    launches += apply_plans(wq, ctx, spec, m, mi, Wb[mi], buf.s[m.x_id], G, outs[mi]["clip_idx"], plans_b, buf,
                                            grid_d, sink, accounted=(totals[mi], offs[mi]), lowbit=outs[mi]["lowbit"])
        return launches
    for mi, m in enumerate(mats):
        W, s = Wb[mi], buf.s[m.x_id]
        for G in spec.chunk_widths:
            U = m.C // G
            feat = buf.take("feat")[:U * 8].view(U, 8)
            wq.windq_unit_features(ctx, W, G, s, feat)
            launches += 2
            out = dict(err=buf.take("err")[:U * 6].view(U, 6), energy=buf.take("energy")[:U],
                       clip_idx=buf.clip_idx[:4 * U * m.R].view(4, U, m.R))
            e0 = timer.start() if timer else None
            wq.windq_fit_eval(ctx, W, G, s, grid_d, out=out)
            if timer:
                timer.stop(e0)
            launches += 2
            if sink:
                sink("feat", feat)
                sink("err", out["err"])
                sink("energy", out["energy"])
            if G == APPLY_G and plans_b:
                launches += apply_plans(wq, ctx, spec, m, mi, W, s, G, out["clip_idx"], plans_b, buf, grid_d, sink)
    return launches


def packed_code_bytes(actions_np, R, G):
    per = np.array([2 * G, G, G // 2, 3 * G // 8, G // 4, (G + 4) // 5, G // 8], np.int64)
    return int(((R * per[actions_np] + 15) // 16 * 16).sum())


# ---------------------------------------------------------------------------------------- legs
def run_device_leg(wq, ctx, spec, model, plans, plan_index, buf, grid_d, steps, warmup, rank, sync):
    """Times `steps` steps with everything the kernels read resident in HBM.  A resident model is timed by one pair of
    events around all steps; a streamed one by a pair of events around every block's kernels (the refill of the block
    slots in between is not counted), summed."""
    block_pairs = []

    def step(timer=None, timed=False):
        n = 0
        for bi in range(len(model.blocks)):
            Wb, Xb = model.block(bi)
            if timed and model.streamed:
                e0 = torch.cuda.Event(enable_timing=True)
                e0.record()
            n += score_block(wq, ctx, spec, Wb, Xb, {t: plans[t][plan_index[bi]] for t in plans}, buf, grid_d, timer)
            if timed and model.streamed:
                e1 = torch.cuda.Event(enable_timing=True)
                e1.record()
                block_pairs.append((e0, e1))
        return n

    for _ in range(warmup):
        step()
    timer = FitTimer()
    sync()
    with ClockSampler(rank) as clocks:
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        launches = 0
        for _ in range(steps):
            launches += step(timer, timed=True)
        t1.record()
        sync()
    ms = sum(a.elapsed_time(b) for a, b in block_pairs) if model.streamed else t0.elapsed_time(t1)
    return ms, launches, timer.total_ms(), clocks.summary()


def run_e2e_leg(wq, ctx, spec, model, plans, plan_index, plans_np, buf, grid_d, steps, warmup, sync):
    """Same step from pinned host memory: two device-side block slots, copies on a second stream
    overlapped with the previous block's kernels; every result copied back to pinned host memory.
    As many distinct blocks as a third of the free host memory holds (at most 24 for a streamed model) are kept in
    pinned memory and used in turn: every step still copies every block's bytes from the host."""
    mats = matrices_of(spec)
    nb = len(model.blocks)
    need = sum(m.R * m.C for m in mats) * 2 + sum(spec.T * c for _, c in inputs_of(spec)) * 2
    import psutil
    avail = psutil.virtual_memory().available
    host_blocks = max(1, min(nb, int(avail // (3 * need)), 24 if model.streamed else nb))
    hostW, hostX = [], []
    for bi in range(host_blocks):
        Wb, Xb = model.block(bi)
        hostW.append([w.cpu().pin_memory() for w in Wb])
        hostX.append({i: x.cpu().pin_memory() for i, x in Xb.items()})
    slots = []
    for _ in range(2):
        slots.append(dict(W=[torch.empty_like(w) for w in model.W[0]], X={i: torch.empty_like(x) for i, x in model.X[0].items()},
                          ready=torch.cuda.Event(), free=torch.cuda.Event()))
    copy_stream = torch.cuda.Stream()
    main = torch.cuda.current_stream()
    # pinned result buffers (sized for the largest matrix); results leave on a third stream, so that the
    # kernels of the next matrix do not queue behind the copies of this one
    out_stream = torch.cuda.Stream()
    host_out = {}

    def host_buf(name, n, dtype):
        key = (name, dtype)
        if key not in host_out or host_out[key].numel() < n:
            host_out[key] = torch.empty(n, dtype=dtype).pin_memory()
        return host_out[key][:n]

    d2h = [0]

    def sink(name, t, slot=None):
        if name == "codes":
            codes, acts, R, G = t
            src = codes[:sink.code_bytes[(id(acts))]]
        else:
            src = t.reshape(-1)
        produced = torch.cuda.Event()
        produced.record(main)
        out_stream.wait_event(produced)
        with torch.cuda.stream(out_stream):
            host_buf(name, src.numel(), src.dtype).copy_(src, non_blocking=True)
            copied = torch.cuda.Event()
            copied.record(out_stream)
        # the call that writes this slot next waits for the copy
        buf.pending[(name, buf.last[name] if slot is None else slot)] = copied
        d2h[0] += src.numel() * src.element_size()

    sink.code_bytes = {}
    for target in plans:
        for bi in range(len(plans[target])):
            for mi, m in enumerate(mats):
                sink.code_bytes[id(plans[target][bi][mi])] = packed_code_bytes(plans_np[target][bi][mi], m.R, APPLY_G)
    # make sure the largest pinned result buffers exist before timing
    maxRC = max(m.R * m.C for m in mats)
    host_buf("codes", 2 * maxRC, torch.uint8)
    h2d_per_step = need * nb

    def step():
        n = 0
        for bi in range(nb):
            slot = slots[bi % 2]
            hb = bi % host_blocks
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(slot["free"])
                for dst, src in zip(slot["W"], hostW[hb]):
                    dst.copy_(src, non_blocking=True)
                for i in slot["X"]:
                    slot["X"][i].copy_(hostX[hb][i], non_blocking=True)
                slot["ready"].record(copy_stream)
            main.wait_event(slot["ready"])
            n += score_block(wq, ctx, spec, slot["W"], slot["X"], {t: plans[t][plan_index[bi]] for t in plans}, buf, grid_d, None, sink)
            slot["free"].record(main)
        return n

    for s in slots:
        s["free"].record(main)
    for _ in range(min(warmup, 1)):
        step()
    sync()
    d2h[0] = 0
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    wall0 = time.perf_counter()
    t0.record()
    for _ in range(steps):
        step()
    main.wait_stream(out_stream)      # the step is over when the last result is on the host
    t1.record()
    sync()
    wall = (time.perf_counter() - wall0) * 1e3
    ms = max(t0.elapsed_time(t1), 0.0)
    return ms, wall, h2d_per_step, d2h[0] // max(steps, 1), host_blocks


ORACLE_SAMPLE_MATRICES = 5     # block 0: q, k, v, o and gate projections (about 55 % of a block's weights)


def run_extras(wq, ctx, spec, model, buf, grid_d, reps=3):
    """Times, on the matrices of this rank's first block at the plan chunk width, the calls that are not part
    of a step: saliency score, salient-weight selection at 3 %, the protected fit, the step-size refinement
    (10 steps), packing with protection, and the heuristic allocator's rule over the units of the whole model.
    Returns {name: milliseconds per block} (the allocator: per call)."""
    G, mats = APPLY_G, matrices_of(spec)
    Wb, Xb = model.W[0], model.X[0]
    for i, X in Xb.items():
        wq.windq_act_stats(ctx, X, buf.s[i])
    need = max(max(wq.windq_scratch_bytes_salient_select(m.R, m.C, G), wq.windq_scratch_bytes_fit_eval_protected(m.R, m.C, G),
                   wq.windq_scratch_bytes_apply_plan_protected(m.R, m.C, G), wq.windq_scratch_bytes_fit_refine(m.R, m.C, G))
               for m in mats)
    n_units_model = sum(m.C // G for m in mats) * spec.n_blocks
    wq.windq_reserve(ctx, max(need, wq.windq_scratch_bytes_greedy_allocate(n_units_model)))
    times = {}

    def timed(name, fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = fn()
        e1.record()
        torch.cuda.synchronize()
        times.setdefault(name, []).append(e0.elapsed_time(e1))
        return out

    sal_all, cnt_all, n_all, g_all = [], [], [], []
    for rep in range(reps + 1):
        for mi, m in enumerate(mats):
            W, s, U = Wb[mi], buf.s[m.x_id], m.C // G
            sal = timed("unit_saliency", lambda: wq.windq_unit_saliency(ctx, W, G, s))
            sel = timed("salient_select", lambda: wq.windq_salient_select(ctx, W, G, s, 30000, want_mask=False))
            fit = timed("fit_eval_protected", lambda: wq.windq_fit_eval(ctx, W, G, s, grid_d, thresh=sel["thresh"]))
            plain = wq.windq_fit_eval(ctx, W, G, s, grid_d)
            timed("fit_refine", lambda: wq.windq_fit_refine(ctx, W, G, s, grid_d, plain["clip_idx"], 10, 0.01))
            acts = torch.full((U,), 4, dtype=torch.uint8, device="cuda")
            eb = wq.windq_effective_bits(ctx, acts, m.R, G)
            prot_q = torch.empty(int(0.04 * m.R * m.C) + 1024, dtype=torch.int8, device="cuda")
            timed("apply_plan_protected", lambda: wq.windq_apply_plan_protected(
                ctx, W, G, s, grid_d, acts, eb["code_offsets"], buf.take("codes"), sel["thresh"], prot_q, fit["clip_idx"]))
            if rep == 0:
                sal_all.append(sal)
                cnt_all.append(sel["count"])
                n_all.append(torch.full((U,), m.R * G, dtype=torch.int64, device="cuda"))
                g_all.append(torch.full((U,), m.R, dtype=torch.int64, device="cuda"))
    n_rep = spec.n_blocks
    sal_m, cnt_m = torch.cat(sal_all).repeat(n_rep), torch.cat(cnt_all).repeat(n_rep)
    n_m, g_m = torch.cat(n_all).repeat(n_rep), torch.cat(g_all).repeat(n_rep)
    sal_m = (sal_m * (1.0 + 0.001 * torch.arange(sal_m.numel(), device="cuda") / sal_m.numel())).contiguous()
    for rep in range(reps + 1):
        timed("greedy_allocate", lambda: wq.windq_greedy_allocate(ctx, sal_m, n_m, g_m, 200, 10, cnt_m, scale_bits=16, zero_bits=16))
    out = {}
    for name, ts in times.items():
        per_rep = len(ts) // (reps + 1)
        kept = ts[per_rep:]                                   # the first repetition is the warm-up
        out[name + "_ms"] = sum(kept) / reps
    out["chunk_width"] = G
    out["allocator_units"] = int(sal_m.numel())
    out["note"] = "per block (7 matrices), except greedy_allocate: one call over the model's units"
    return out


def oracle_sample(spec, seed, threads, n_matrices=ORACLE_SAMPLE_MATRICES):
    """The CPU oracle on a bounded sample of the workload: the whole hot path for the first n_matrices matrices of
    block 0 -- their calibration statistics, and per matrix unit_features + fit_eval at every chunk width and the
    three plans at APPLY_G.  With threads > 1 every call runs the oracle's single-threaded routine over disjoint
    unit (or channel) ranges on that many threads; the routine itself is never changed for this.
    Returns (seconds, unit x bit-width evaluations, description)."""
    import oracle
    mats = matrices_of(spec)[:n_matrices]
    Ws = [ws.block_weight(spec, seed, 0, m).numpy() for m in mats]
    Xs = {i: ws.block_input(spec, seed, 0, i).numpy() for i in sorted({m.x_id for m in mats})}
    grid = ws.clip_grid(spec.K)
    rng = np.random.default_rng(seed)
    t0 = time.perf_counter()
    stats = {i: _over_ranges(threads, X.shape[1], lambda a, b, X=X: oracle.act_stats(np.ascontiguousarray(X[:, a:b])), np.concatenate)
             for i, X in Xs.items()}
    evals = 0
    for m, W in zip(mats, Ws):
        s = stats[m.x_id]
        for G in spec.chunk_widths:
            U = m.C // G
            _over_ranges(threads, U, lambda a, b: oracle.unit_features(np.ascontiguousarray(W[:, a * G:b * G]), G, s[a * G:b * G]))
            fit = oracle.fit_eval(W, G, s, grid, threads=threads, want_group_err=False)
            evals += 6 * U
            if G == APPLY_G:
                for ti, _ in enumerate(TARGET_BITS):
                    acts = rng.choice(7, size=U, p=np.array(ws.ACTION_MIX) / sum(ws.ACTION_MIX)).astype(np.uint8)
                    oracle.effective_bits(acts, m.R, G)
                    _over_ranges(threads, U, lambda a, b: oracle.apply_plan(
                        np.ascontiguousarray(W[:, a * G:b * G]), G, s[a * G:b * G], grid, acts[a:b],
                        np.ascontiguousarray(fit["clip_idx"][:, a:b])))
    dt = time.perf_counter() - t0
    desc = "block 0 of %d, matrices %s (%.1f M weights), T=%d: act_stats, unit_features + fit_eval at G=%s, 3 plans applied at G=%d" % (
        spec.n_blocks, "/".join(m.name for m in mats), sum(m.R * m.C for m in mats) / 1e6, spec.T,
        "/".join(map(str, spec.chunk_widths)), APPLY_G)
    return dt, evals, desc


def _over_ranges(threads, n, fn, combine=None):
    """fn(a, b) over disjoint ranges of [0, n) on `threads` threads (one call when threads <= 1)."""
    if threads <= 1 or n <= 1:
        return fn(0, n)
    from concurrent.futures import ThreadPoolExecutor
    bounds = np.linspace(0, n, min(threads, n) + 1).astype(int)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        parts = list(ex.map(lambda ab: fn(int(ab[0]), int(ab[1])), [ab for ab in zip(bounds[:-1], bounds[1:]) if ab[1] > ab[0]]))
    return combine(parts) if combine else None


def cpu_baseline(spec, seed):
    """The oracle, as it stands, on this machine's host cores: on all of them over the five-matrix sample, and on ONE core
    over the first matrix of the sample."""
    threads = os.cpu_count() or 1
    dt, ev, desc = oracle_sample(spec, seed, threads)
    dt1, ev1, desc1 = oracle_sample(spec, seed, 1, n_matrices=1)
    return dict(value=ev / dt, unit=UNIT, cores=threads, kind="oracle", sample=desc, seconds=dt,
                one_core=dict(value=ev1 / dt1, unit=UNIT, cores=1, sample=desc1, seconds=dt1))


def reference_main(args, spec):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = os.cpu_count() or 1
    for _ in range(min(args.warmup, 1)):
        oracle_sample(spec, SEED, threads)
    tot_t, tot_e, desc = 0.0, 0, ""
    for _ in range(args.steps):
        dt, ev, desc = oracle_sample(spec, SEED, threads)
        tot_t += dt
        tot_e += ev
    value = tot_e / tot_t
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1e3 * tot_t / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f32",
                data="synthetic", config=dict(workload=spec.name, sample=desc),
                cpu_baseline=dict(value=value, unit=UNIT, cores=threads, kind="oracle", sample=desc),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line))


def main():
    global APPLY_G, BATCH_FITS, MULTI_APPLY, FUSED_FEATURES
    args = parse_args()
    spec = ws.CONFIGS[args.workload]
    if APPLY_G not in spec.chunk_widths:
        APPLY_G = spec.chunk_widths[0]
    if args.impl == "reference":
        return reference_main(args, spec)
    BATCH_FITS = not args.separate_fits
    MULTI_APPLY = BATCH_FITS and not args.separate_plans
    FUSED_FEATURES = BATCH_FITS and args.fused_features

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the windq library has no CPU path")
    torch.cuda.set_device(local_rank)
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    import paper_2605_26660_b200 as wq
    from paper_2605_26660_b200 import sharding

    def sync():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    peaks = load_peaks()
    ctx = wq.windq_create(local_rank)
    n_blocks = args.blocks if args.blocks > 0 else spec.n_blocks
    strong = args.scaling == "strong" and world > 1
    if strong:
        # the blocks of ONE model split over the ranks; block b keeps its plans
        blocks = sharding.block_range(n_blocks, rank, world)
        plan_index = list(blocks)
    else:
        # weak scaling: rank r scores its own replica (global blocks r * n_blocks ...), every replica under the same plans
        blocks = sharding.block_range(n_blocks * world, rank, world)
        plan_index = list(range(n_blocks))
    block_bytes = 2 * sum(m.R * m.C for m in matrices_of(spec)) + 2 * spec.T * sum(c for _, c in inputs_of(spec))
    free_bytes = torch.cuda.mem_get_info(local_rank)[0]
    streamed = args.stream == "yes" or (args.stream == "auto" and block_bytes * len(blocks) > 0.5 * free_bytes)
    model = DeviceModel(spec, blocks, SEED, streamed=streamed)
    buf = Buffers(spec, ring=len(TARGET_BITS) if MULTI_APPLY else 1)      # the plans of a matrix are packed together: an output set each
    grid_d = torch.from_numpy(ws.clip_grid(spec.K)).cuda()
    plans = make_plans(wq, ctx, spec, n_blocks, APPLY_G) if APPLY_G in spec.chunk_widths else {}
    plans_np = {t: [[a.cpu().numpy() for a in row] for row in plans[t]] for t in plans}
    mats = matrices_of(spec)
    scratch = max(max(wq.windq_scratch_bytes_fit_eval(m.R, m.C, G), wq.windq_scratch_bytes_unit_features(m.R, m.C, G))
                  for m in mats for G in spec.chunk_widths)
    if BATCH_FITS:
        scratch = max(scratch, max(sum(wq.windq_scratch_bytes_fit_eval(m.R, m.C, G) for m in mats) for G in spec.chunk_widths),
                      2 * max(sum(wq.windq_scratch_bytes_unit_features(m.R, m.C, G) for m in mats) for G in spec.chunk_widths))
    if FUSED_FEATURES:
        scratch = max(scratch, wq.windq_scratch_bytes_features_fit_batch(model.W[0], min(spec.chunk_widths)))
    wq.windq_reserve(ctx, scratch)

    elems, units = workload_counts(spec, n_blocks)                  # of one model
    evals_per_step = 6 * sum(units.values())
    job_evals = evals_per_step if strong else world * evals_per_step   # what all ranks together score in a step
    elems_rank, _ = workload_counts(spec, len(blocks))               # what this rank's fits read
    wq.windq_fit_work(ctx, reset=True)
    ms, launches, fit_ms, clocks = run_device_leg(wq, ctx, spec, model, plans, plan_index, buf, grid_d, args.steps, args.warmup,
                                                  local_rank, sync)
    evaluated, searched = wq.windq_fit_work(ctx, reset=True)      # clip candidates the fits evaluated in full / all of them
    ms = sharding.max_float(ms)
    value = job_evals * args.steps / (ms * 1e-3)

    # plan totals (control path): exact int64 sums over ranks
    total_cb = sharding.sum_int64(int(buf.totals[2 * (len(TARGET_BITS) - 1)].item())) if plans else 0
    torch.cuda.synchronize()

    n_fit = max(1, len(spec.chunk_widths) * (1 if BATCH_FITS else len(mats)) * len(blocks) * args.steps)
    fit_elem = elems_rank * len(spec.chunk_widths) * args.steps
    ops = fit_ops_per_element(spec.K)
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    alu_peak = sm_count * 128 * peaks["sm_max_mhz"] * 1e6 / 1e12          # T lane-ops/s, fma = 1
    achieved = fit_elem * ops / (fit_ms * 1e-3) / 1e12
    hbm_time = 2.0 * fit_elem / (peaks["hbm_gbs"] * 1e9)
    alu_time = fit_elem * ops / (alu_peak * 1e12)
    # DRAM traffic of fit_eval_kernel per launch: dram__bytes_read + dram__bytes_write of an ncu capture of the same
    # launch shape (profiles/fit_eval_kernel_batch_cfg3_block_K20.txt: 436 MB against 404.75 MB of weights for a block
    # per launch; one matrix per launch has no capture of the present kernel: null), scaled to this run's average
    # launch by the weights a launch reads (traffic is proportional to them: one pass, no re-reads)
    per_byte = FIT_TRAFFIC_PER_WEIGHT_BYTE[BATCH_FITS]
    traffic = None if per_byte is None else per_byte * 2.0 * fit_elem / n_fit
    roofline = dict(bound="alu" if alu_time >= hbm_time else "hbm", kernel="fit_eval_kernel", achieved=achieved, peak=alu_peak,
                    unit="T fp32 lane-ops/s (fma = 1)", frac=achieved / alu_peak, traffic=traffic, traffic_unit="bytes per launch",
                    launches=n_fit, avg_launch_ms=fit_ms / n_fit, ops_per_element=ops,
                    weight_gbs=2.0 * fit_elem / (fit_ms * 1e-3) / 1e9, hbm_frac=hbm_time / (fit_ms * 1e-3),
                    elem_cand_per_s=fit_elem * (4 * spec.K + 2) / (fit_ms * 1e-3),
                    peak_source="%d SMs x 128 lanes x %.0f MHz (%s)" % (sm_count, peaks["sm_max_mhz"], peaks["source"]))
    # `frac` credits the search with all its candidates (the count the method defines).  The eight-bit search skips
    # candidates that provably cannot win; what the kernel executed is the evaluated share of the 28 K operations,
    # the ten once per weight, and the bound of the eight-bit candidates (seven operations on two of a lane's 32 weights)
    share = evaluated / max(1, searched)
    ops_executed = 28 * spec.K * share + 10 + 7 * spec.K / 16.0
    roofline["executed"] = dict(candidates_evaluated_share=share, ops_per_element=ops_executed,
                                frac=fit_elem * ops_executed / (fit_ms * 1e-3) / 1e12 / alu_peak)

    e2e = None
    if not args.no_e2e:
        del buf
        # with the batched fit the 21 plan applications of a block run back to back: give every one of them its own
        # output slot (and three more), so that packing never waits for a device-to-host copy and the copies of one
        # block overlap the fits of the next
        ebuf = Buffers(spec, ring=3 * len(mats) + 3 if BATCH_FITS else 3)
        e_steps = max(1, min(args.steps, 5))
        e_ms, e_wall, h2d, d2h, host_blocks = run_e2e_leg(wq, ctx, spec, model, plans, plan_index, plans_np, ebuf, grid_d,
                                                          e_steps, args.warmup, sync)
        e_ms = sharding.max_float(max(e_ms, e_wall))
        e2e = dict(value=job_evals * e_steps / (e_ms * 1e-3), unit=UNIT, h2d_bytes_per_step=h2d,
                   d2h_bytes_per_step=d2h, steps=e_steps, ms_per_step=e_ms / e_steps,
                   host_blocks_resident=host_blocks)

    extras = None
    if args.extras and rank == 0:
        extras = run_extras(wq, ctx, spec, model, Buffers(spec), grid_d)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(spec, SEED)

    if rank == 0:
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=ms / args.steps, higher_is_better=True, scaling="strong" if strong else "weak", vs_baseline=None,
                    dtype="f32", data="synthetic",
                    config=dict(workload=spec.name, blocks=n_blocks, elements_per_chunk_width=elems, units=units, K=spec.K,
                                chunk_widths=list(spec.chunk_widths), plan_targets=list(TARGET_BITS), apply_chunk_width=APPLY_G,
                                tokens=spec.T, weights=spec.dist,
                                parallelism="the blocks of one model split over the GPUs" if strong else "replica per GPU",
                                residency="two block slots refilled block by block (the model does not fit); only the kernels "
                                          "of a block are timed" if streamed else "all blocks resident in HBM",
                                features="one pass per block for both chunk widths (windq_unit_features_batch2)"
                                if (not FUSED_FEATURES and BATCH_FITS and len(spec.chunk_widths) == 2 and spec.chunk_widths[1] == 2 * spec.chunk_widths[0])
                                else "one pass per block and chunk width",
                                fits="one windq_features_fit_batch call per block and chunk width" if FUSED_FEATURES
                                else "one windq_unit_features_batch and one windq_fit_eval_batch call per block and chunk width" if BATCH_FITS
                                else "one windq_unit_features and one windq_fit_eval call per matrix",
                                plans="the %d plans of a matrix packed by one windq_apply_plan_multi call" % len(TARGET_BITS) if MULTI_APPLY
                                else "one windq_apply_plan call per matrix and plan",
                                l2="every step streams %.1f GB of inputs, far above the 126 MB L2" % (
                                    (2 * elems + 2 * spec.T * sum(c for _, c in inputs_of(spec)) * n_blocks) / 1e9)),
                    clocks=clocks, e2e=e2e, gpu_launches=launches, roofline=roofline, cpu_baseline=cpu,
                    fit_eval_ms_per_step=fit_ms / args.steps, plan_total_centibits_last=total_cb)
        if extras:
            line["extras"] = extras
        print(json.dumps(line))
    wq.windq_destroy(ctx)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
