"""Seeded synthetic inputs for the WINDQuant scoring path.

Stand-ins for the pretrained LLaMA linear weights and the calibration
activations of the paper's experiments ("Experiment Settings"), which are not
available: same shapes, heavy-tailed / outlier-channel structure, fp16.  This
module serves both the CPU oracle and the CUDA library and therefore holds no
arithmetic of the method itself: no statistics, no quantizer, no bit
accounting.  Everything is a pure function of (seed, shape).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch

# Action codes in the order of the paper's action set (Eq. 3): index -> nominal bits.
ACTION_NAMES = ("skip16", "8", "4", "3", "2", "1.58", "1")
# Learned action mix of the 8B run (appendix pie chart): 39.15 % 1-bit, 36.54 % 1.58-bit,
# 15.65 % 2-bit, 8.65 % ">= 3-bit or skip".  The split of that remainder is a choice made here.
ACTION_MIX = (0.005, 0.0065, 0.025, 0.05, 0.1565, 0.3654, 0.3915)


def matrix_seed(seed: int, block: int, matrix_id: int) -> int:
    return seed * 1000003 + block * 16 + matrix_id


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def clip_grid(K: int, lo: float = 0.5, hi: float = 1.0) -> np.ndarray:
    """K clip ratios, endpoints included, computed in double and rounded to fp32."""
    if K == 1:
        return np.array([hi], np.float32)
    return np.array([lo + (hi - lo) * k / (K - 1) for k in range(K)], np.float64).astype(np.float32)


def weights(R: int, C: int, seed: int, dist: str = "normal", device="cpu", std: float = 0.02,
            outlier_frac: float = 0.001, outlier_gain: float = 20.0) -> torch.Tensor:
    """fp16 [R, C] weight matrix.

    dist = "normal": N(0, std^2).  dist = "student_t": Student-t with 4 degrees of
    freedom rescaled to standard deviation std (t4 has variance 2).  A seeded
    choice of round(outlier_frac * C) input columns is multiplied by outlier_gain.
    """
    g = _gen(seed, device)
    z = torch.randn((R, C), generator=g, device=device, dtype=torch.float32)
    if dist == "student_t":
        # chi-square with 4 dof = -2 ln(U1 U2); t = z * sqrt(4 / chi2)
        u = torch.rand((R, C), generator=g, device=device, dtype=torch.float32).clamp_min_(1e-12)
        u.mul_(torch.rand((R, C), generator=g, device=device, dtype=torch.float32).clamp_min_(1e-12))
        u.log_().mul_(-0.5)                       # chi2 / 4
        z.mul_(u.rsqrt_()).mul_(std / math.sqrt(2.0))
        del u
    elif dist == "normal":
        z.mul_(std)
    else:
        raise ValueError(dist)
    n_out = int(round(outlier_frac * C))
    if n_out > 0:
        cols = torch.randperm(C, generator=g, device=device)[:n_out]
        z[:, cols] *= outlier_gain
    return z.to(torch.float16)


def activations(T: int, C: int, seed: int, device="cpu", n_hot: int = 8, hot_gain: float = 50.0) -> torch.Tensor:
    """fp16 [T, C] calibration activations: x_tj = g_j * N(0,1), g_j ~ lognormal(0,1),
    with n_hot seeded channels multiplied by hot_gain."""
    g = _gen(seed, device)
    gain = torch.randn((C,), generator=g, device=device, dtype=torch.float32).exp_()
    hot = torch.randperm(C, generator=g, device=device)[:n_hot]
    gain[hot] *= hot_gain
    x = torch.randn((T, C), generator=g, device=device, dtype=torch.float32)
    x.mul_(gain.unsqueeze(0))
    return x.clamp_(-60000.0, 60000.0).to(torch.float16)


@dataclass(frozen=True)
class MatrixSpec:
    name: str
    R: int          # out features
    C: int          # in features
    x_id: int       # which calibration input of the block feeds it
    matrix_id: int


@dataclass(frozen=True)
class ModelSpec:
    name: str
    n_blocks: int
    hidden: int
    inter: int
    kv: int
    dist: str
    T: int
    K: int
    chunk_widths: tuple
    only: tuple = ()        # names of the block's matrices that exist (empty = all seven)

    def block_matrices(self):
        h, i, kv = self.hidden, self.inter, self.kv
        all_seven = (
            MatrixSpec("q_proj", h, h, 0, 0), MatrixSpec("k_proj", kv, h, 0, 1),
            MatrixSpec("v_proj", kv, h, 0, 2), MatrixSpec("o_proj", h, h, 1, 3),
            MatrixSpec("gate_proj", i, h, 2, 4), MatrixSpec("up_proj", i, h, 2, 5),
            MatrixSpec("down_proj", h, i, 3, 6),
        )
        return tuple(m for m in all_seven if not self.only or m.name in self.only)

    def block_inputs(self):
        """(x_id, channels) of the calibration inputs of a block (four when all seven matrices exist)."""
        used = {m.x_id for m in self.block_matrices()}
        return tuple(ic for ic in ((0, self.hidden), (1, self.hidden), (2, self.hidden), (3, self.inter)) if ic[0] in used)

    def elements_per_block(self) -> int:
        return sum(m.R * m.C for m in self.block_matrices())


# The five benchmark configurations (LLaMA-1/2-style shapes), and the shape the paper itself reports its
# unit count on ("Episode complexity": LLaMA-3.1-8B, chunk size 256, 32 x 7 x 16 = 3584 units), with its
# ablated chunk size 512 beside it.
CONFIGS = {
    "cfg1_single_layer": ModelSpec("cfg1_single_layer", 1, 4096, 0, 4096, "normal", 512, 20, (128,), only=("q_proj",)),
    "cfg2_llama7b_block": ModelSpec("cfg2_llama7b_block", 1, 4096, 11008, 4096, "normal", 2048, 20, (128,)),
    "cfg3_llama7b_model": ModelSpec("cfg3_llama7b_model", 32, 4096, 11008, 4096, "student_t", 2048, 20, (64, 128)),
    "cfg4_llama13b_model": ModelSpec("cfg4_llama13b_model", 40, 5120, 13824, 5120, "student_t", 4096, 40, (128,)),
    "llama3_8b_g256": ModelSpec("llama3_8b_g256", 32, 4096, 14336, 1024, "student_t", 2048, 20, (256, 512)),
    "llama32_1b_g256": ModelSpec("llama32_1b_g256", 16, 2048, 8192, 512, "student_t", 2048, 20, (256,)),
    "cfg5_llama70b_model": ModelSpec("cfg5_llama70b_model", 80, 8192, 28672, 1024, "student_t", 2048, 20, (128,)),
}


def block_weight(spec: ModelSpec, seed: int, block: int, m: MatrixSpec, device="cpu") -> torch.Tensor:
    return weights(m.R, m.C, matrix_seed(seed, block, m.matrix_id), spec.dist, device)


def block_input(spec: ModelSpec, seed: int, block: int, x_id: int, device="cpu") -> torch.Tensor:
    C = dict(spec.block_inputs())[x_id]
    return activations(spec.T, C, matrix_seed(seed, block, 8 + x_id), device)


def random_plan(cost_table: np.ndarray, n_weights: np.ndarray, target_bits: float, seed: int,
                tol: float = 0.005, max_steps: int = 2_000_000) -> np.ndarray:
    """A seeded random plan whose average cost is within tol of target_bits.

    cost_table[i, a] is the storage cost (centibits) of unit i under action a and
    n_weights[i] its weight count; both come from the caller's bit accounting, so
    that this generator only draws, indexes and sums.  Actions are drawn i.i.d.
    from ACTION_MIX; then a seeded random unit is moved one level down (fewer
    bits) while the plan is over target, one level up while it is under.
    """
    rng = np.random.default_rng(seed)
    n = cost_table.shape[0]
    actions = rng.choice(7, size=n, p=np.array(ACTION_MIX) / sum(ACTION_MIX)).astype(np.uint8)
    idx = np.arange(n)
    total = int(cost_table[idx, actions].sum())
    denom = 100.0 * float(n_weights.sum())
    for _ in range(max_steps):
        avg = total / denom
        if abs(avg - target_bits) <= tol:
            return actions
        i = int(rng.integers(n))
        a = int(actions[i])
        b = min(a + 1, 6) if avg > target_bits else max(a - 1, 0)
        if b != a:
            total += int(cost_table[i, b]) - int(cost_table[i, a])
            actions[i] = b
    raise RuntimeError("random_plan did not reach the target")
