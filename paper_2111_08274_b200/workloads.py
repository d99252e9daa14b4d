"""Seeded synthetic workloads for the HADFL round: configuration tables and input draws only.

This module holds none of the method's arithmetic.  It names the five workloads (device count,
flat parameter-vector size, local-step pattern, number of devices selected per round, round
count and optimiser constants) and draws the per-round inputs that are free parameters of a
run: the step count of each device and the seed handed to the selection call.  Both the CUDA
path and the CPU checker take their inputs from here, so that they see identical ones.

The flat vectors stand in for the CNNs of the paper's evaluation (ResNet-18 and VGG-16 on
CIFAR-10): same sizes, values N(0, 0.05^2) generated on each side from the run's seed.
"""
from dataclasses import dataclass, field, replace
from typing import List, Optional, Tuple

import numpy as np

BASE_SEED = 0x48414446  # "HADF"


@dataclass(frozen=True)
class Workload:
    name: str
    n_devices: int
    n_params: int
    k: int
    rounds: int
    steps_rule: str                     # "fixed" or "uniform"
    steps_fixed: Tuple[int, ...] = ()   # per-device step counts when steps_rule == "fixed"
    steps_lo: int = 1
    steps_hi: int = 1
    lr: float = 0.01
    momentum: float = 0.9
    weight_decay: float = 5e-4
    grad_std: float = 1e-3
    init_std: float = 0.05
    version_scale: float = 1.0
    weight_mode: int = 0
    dtype: int = 0                      # 0 fp32 storage, 1 bf16 storage of w
    m_dtype: int = 0                    # 0 fp32 storage of the momentum, 1 bf16 (with bf16 w only)
    rounding: int = 0                   # bf16 stores of the local update: 0 nearest even, 1 stochastic
    seed: int = BASE_SEED
    sync_every: int = 0                 # >0: every that many rounds the aggregate is also sent to the unselected devices
    sync_beta: float = 1.0              # weight of the received model on those rounds: 1 overwrite, <1 mix

    def steps_for_round(self, r: int) -> np.ndarray:
        """Step count of every device in round r (int32[n_devices])."""
        if self.steps_rule == "fixed":
            return np.asarray(self.steps_fixed, dtype=np.int32)
        rng = np.random.default_rng([self.seed & 0xFFFFFFFF, 0x57E95, r])
        return rng.integers(self.steps_lo, self.steps_hi + 1, size=self.n_devices).astype(np.int32)

    def select_seed(self) -> int:
        """Seed passed to every selection call of the run (the round index separates rounds)."""
        return (self.seed * 0x9E3779B97F4A7C15 + 0x53454C) & 0xFFFFFFFFFFFFFFFF

    def device_ids(self) -> np.ndarray:
        return np.arange(self.n_devices, dtype=np.int32)


def c1() -> Workload:
    # 4 devices with the paper's style of power ratios, 2 of 4 selected per round, lr 0.01.
    return Workload("c1", 4, 100_000, 2, 10, "fixed", (1, 2, 3, 4), grad_std=1e-2,
                    seed=BASE_SEED + 1)


def c2() -> Workload:
    # ResNet-18-sized vector, heterogeneity ratio 8x: steps uniform in [1, 8], drawn every round.
    return Workload("c2", 8, 11_173_962, 4, 50, "uniform", steps_lo=1, steps_hi=8,
                    seed=BASE_SEED + 2)


def c3() -> Workload:
    # VGG-16-sized vector, power ratios {1,1,2,2,4,4,8,8} twice; versions counted in rounds of
    # the fastest device (scale 1/8); every 10th round the aggregate reaches all devices.
    return Workload("c3", 16, 14_728_266, 4, 100, "fixed", (1, 1, 2, 2, 4, 4, 8, 8) * 2,
                    version_scale=1.0 / 8.0, seed=BASE_SEED + 3, sync_every=10)


def c4(k: int = 8) -> Workload:
    # ResNet-50-sized vector, wide aggregation: k in {2, 8, 16}.
    steps = tuple(1 + (i % 4) for i in range(32))
    return Workload("c4_k%d" % k, 32, 23_520_842, k, 20, "fixed", steps, seed=BASE_SEED + 4)


def c5(log2_p: int, dtype: int = 0, hetero: bool = False) -> Workload:
    # bandwidth sweep: N = 16, k = 4, P = 2^16 .. 2^27, fp32 or bf16 storage.
    steps = (1, 1, 2, 2, 4, 4, 8, 8) * 2 if hetero else (1,) * 16
    name = "c5_p%d_%s%s" % (log2_p, "bf16" if dtype else "fp32", "_het" if hetero else "")
    return Workload(name, 16, 1 << log2_p, 4, 200, "fixed", steps, dtype=dtype,
                    seed=BASE_SEED + 5)


def shrink(w: Workload, n_params: int, rounds: Optional[int] = None) -> Workload:
    """The same workload on a shorter vector / fewer rounds (for checks that must finish fast)."""
    return replace(w, n_params=n_params, rounds=w.rounds if rounds is None else rounds)


def by_name(name: str) -> Workload:
    """c1, c2, c3, c4_k{2,8,16}, c5_p{16..27}_{fp32,bf16}[_het]."""
    table = {"c1": c1, "c2": c2, "c3": c3}
    if name in table:
        return table[name]()
    if name.startswith("c4"):
        return c4(int(name.split("k")[-1])) if "k" in name else c4()
    if name.startswith("c5_p"):
        parts = name.split("_")
        if len(parts) >= 3 and parts[2] in ("fp32", "bf16"):
            return c5(int(parts[1][1:]), dtype=1 if parts[2] == "bf16" else 0,
                      hetero=len(parts) > 3 and parts[3] == "het")
    raise KeyError(name)


def random_rows(n_rows: int, n_params: int, seed: int, std: float = 0.05) -> np.ndarray:
    """Arbitrary fp32 test rows [n_rows, n_params] (for kernel-level checks on given data)."""
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((n_rows, n_params)) * std).astype(np.float32)


def sample_groups(n_params: int, n_random: int, edge: int, seed: int, around=(), halo: int = 64) -> np.ndarray:
    """Sorted, distinct 4-column group indices: the first and last `edge` groups of the vector,
    `n_random` groups drawn uniformly from the rest, and the `halo` groups on either side of every
    group index listed in `around` (e.g. where one pass of a grid ends and the next begins)."""
    n_groups = (n_params + 3) // 4
    if n_groups <= 2 * edge + n_random:
        return np.arange(n_groups, dtype=np.uint32)
    rng = np.random.default_rng(seed)
    mid = rng.choice(np.arange(edge, n_groups - edge), size=n_random, replace=False)
    parts = [np.arange(edge), mid, np.arange(n_groups - edge, n_groups)]
    for g in around:
        parts.append(np.arange(max(0, int(g) - halo), min(n_groups, int(g) + halo)))
    return np.unique(np.concatenate(parts)).astype(np.uint32)


def pass_boundaries(n_params: int, threads_per_pass, cols_per_thread: int = 8):
    """Group indices at which a grid of `threads_per_pass` threads, each holding `cols_per_thread`
    columns, starts a new pass over a vector of n_params columns - for every entry of
    threads_per_pass.  Only used to aim column samples at those seams."""
    out = []
    for t in threads_per_pass:
        step = int(t) * cols_per_thread // 4
        out.extend(range(step, (n_params + 3) // 4, step))
    return out
