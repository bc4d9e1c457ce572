"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle.

This module holds no arithmetic of the method: it only draws the arrays that
both the CUDA path and the oracle are fed (weights W, codebook table c, upstream
gradient g) and names the workload shapes.  The real Llama-3.2-1B weights and the
paper's incoherence pre-processing are not available offline; the paper treats
pre-processed rows as approximately iid Gaussian (Section 3.1), so N(0,1) draws of
the same shapes stand in for them.

Every array is float32, generated once on the host with numpy's PCG64
``default_rng(seed)``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

BLOCK_N = 256  # weights per trellis block in the Llama-shaped workloads


def codebook(Lb: int, seed: int = 0, V: int = 1) -> np.ndarray:
    """Emission table c[s], s in [0, 2^Lb): iid N(0,1), float32; [2^Lb, V] when a state emits V numbers."""
    shape = (1 << Lb,) if V == 1 else (1 << Lb, V)
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def gaussian(shape, seed: int) -> np.ndarray:
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def student_t(shape, seed: int, nu: float = 4.0) -> np.ndarray:
    """Heavy-tailed weights rescaled to unit variance (Var[t_nu] = nu/(nu-2))."""
    x = np.random.default_rng(seed).standard_t(nu, size=shape)
    return (x / np.sqrt(nu / (nu - 2.0))).astype(np.float32)


@dataclass
class Workload:
    """One named synthetic workload: a list of weight matrices cut row-major into blocks of n."""
    name: str
    Lb: int
    k: int
    n: int
    T: float
    matrices: List[Tuple[str, Tuple[int, int]]]
    w_seed: int = 1
    g_seed: int = 2
    c_seed: int = 0
    dist: str = "normal"
    extra_T: Tuple[float, ...] = field(default_factory=tuple)
    V: int = 1                 # numbers emitted per state and step (a step consumes V weights, k*V bits)

    @property
    def S(self) -> int:
        return 1 << self.Lb

    @property
    def K(self) -> int:
        return 1 << (self.k * self.V)

    @property
    def steps(self) -> int:
        return self.n // self.V

    def num_blocks(self) -> int:
        return sum(r * c // self.n for _, (r, c) in self.matrices)

    def edges_per_sweep(self) -> int:
        """Trellis-edge updates of one sweep: blocks * steps * states * branches."""
        return self.num_blocks() * self.steps * self.S * self.K

    def codebook(self) -> np.ndarray:
        return codebook(self.Lb, self.c_seed, self.V)

    def weights(self, idx: int = 0) -> np.ndarray:
        """Matrix `idx` as [num_blocks, n] (row-major split of each row into blocks of n)."""
        _, (r, c) = self.matrices[idx]
        seed = self.w_seed + idx
        x = student_t((r, c), seed) if self.dist == "student_t" else gaussian((r, c), seed)
        return x.reshape(-1, self.n)

    def upstream(self, idx: int = 0, step: int = 0) -> np.ndarray:
        _, (r, c) = self.matrices[idx]
        return gaussian((r, c), self.g_seed + idx + 7919 * step).reshape(-1, self.n)


def tiny() -> Workload:
    # 64 independent blocks of 64 weights, S = 256, four branches per state
    return Workload("tiny", Lb=8, k=2, n=64, T=0.5, matrices=[("blocks", (64, 64))],
                    w_seed=1, g_seed=2)


def brute() -> Workload:
    # small enough to enumerate all S*K^(n-1) = 16384 paths
    return Workload("brute", Lb=4, k=2, n=6, T=0.5, matrices=[("blocks", (4, 6))],
                    w_seed=11, g_seed=12)


def mid() -> Workload:
    return Workload("mid", Lb=12, k=2, n=BLOCK_N, T=0.1, matrices=[("w", (1024, 1024))],
                    w_seed=2001, g_seed=2501, extra_T=(1.0, 0.1, 0.01, 1e-4))


def q_proj() -> Workload:
    return Workload("llama32_1b_q_proj", Lb=16, k=2, n=BLOCK_N, T=0.1,
                    matrices=[("q_proj", (2048, 2048))], w_seed=3001, g_seed=3501)


def decoder_layer() -> Workload:
    mats = [("q_proj", (2048, 2048)), ("k_proj", (512, 2048)), ("v_proj", (512, 2048)),
            ("o_proj", (2048, 2048)), ("gate_proj", (8192, 2048)), ("up_proj", (8192, 2048)),
            ("down_proj", (2048, 8192))]
    return Workload("llama32_1b_decoder_layer", Lb=16, k=2, n=BLOCK_N, T=0.3, matrices=mats,
                    w_seed=4001, g_seed=4501)


def gate_k3() -> Workload:
    return Workload("gate_student_t_3bpw", Lb=16, k=3, n=BLOCK_N, T=0.01,
                    matrices=[("gate_proj", (8192, 2048))], w_seed=5001, g_seed=5501,
                    dist="student_t", extra_T=(0.01, 0.001))


def qtip_v2() -> Workload:
    # the paper's own trellis configuration (16 state bits, 2 bits per weight, 2 weights per step:
    # 128 steps per 256-weight block, 16 predecessors per state) on the q_proj shape
    return Workload("llama32_1b_q_proj_v2", Lb=16, k=2, n=BLOCK_N, T=0.1,
                    matrices=[("q_proj", (2048, 2048))], w_seed=6001, g_seed=6501, V=2)


def sample_blocks(num_blocks: int, count: int, seed: int = 99) -> np.ndarray:
    """Seeded block indices that always include the first and the last block."""
    count = min(count, num_blocks)
    rng = np.random.default_rng(seed)
    pick = set([0, num_blocks - 1]) if num_blocks > 1 else {0}
    while len(pick) < count:
        pick.add(int(rng.integers(0, num_blocks)))
    return np.array(sorted(pick), dtype=np.int64)
