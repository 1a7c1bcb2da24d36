"""Seeded synthetic inputs for the HAC / sHAC workloads.

This module only draws random numbers.  It holds none of the method's
arithmetic (no pruning, no quantization, no coding), so that the CPU oracle and
the CUDA library can both be fed from it without sharing any part of the
method.  Every array is float32, C-contiguous and a pure function of
(config, item).

The five workloads mirror the shapes, sparsities and numbers of shared values
used in the paper's comparison of the compressed formats (Sect. V-C: the fully
connected matrices of VGG19, pruned 60-99 %, weight sharing with k = 32 / 256,
dense input vectors), with Gaussian "He-init" matrices standing in for the
trained weights, which are not available.
"""
from __future__ import annotations

import dataclasses
import numpy as np

QUANT_NONE = 0
QUANT_KMEANS = 1
QUANT_UNIFORM = 2
QUANT_GRID = 3
QUANT_PWS = 4


@dataclasses.dataclass(frozen=True)
class Workload:
    """One layer shape plus the build hyper-parameters used on it."""
    config: int            # 1..5, numbering of the benchmark configurations
    name: str
    n: int                 # rows of W   (inputs of the layer)
    m: int                 # columns of W (outputs of the layer)
    sparsity: float        # target fraction of zeros after pruning
    k: int                 # number of shared values for the non-null weights
    quantizer: int         # QUANT_KMEANS or QUANT_UNIFORM
    formats: tuple         # subset of ("hac", "shac")
    batches: tuple         # batch sizes the product is run at
    x_dist: str            # "uniform_pm1" | "relu_normal" | "uniform_01"
    kmeans_iters: int = 20
    item: int = 0          # sub-item (sweep cell) inside the configuration

    @property
    def seed(self) -> int:
        return 1000 * self.config + self.item


def he_std(n: int) -> float:
    """Standard deviation sqrt(2 / fan_in) of the He initialisation."""
    return float(np.sqrt(2.0 / n))


def weights(wl: Workload) -> np.ndarray:
    """W (n x m) float32 ~ N(0, sqrt(2/n)), row-major."""
    rng = np.random.default_rng(wl.seed)
    w = rng.standard_normal((wl.n, wl.m), dtype=np.float32)
    w *= np.float32(he_std(wl.n))
    return np.ascontiguousarray(w)


def inputs(wl: Workload, batch: int, salt: int = 0) -> np.ndarray:
    """X (batch x n) float32, one input vector per row."""
    rng = np.random.default_rng([wl.seed, 7919, batch, salt])
    if wl.x_dist == "uniform_pm1":
        x = rng.random((batch, wl.n), dtype=np.float32) * np.float32(2.0) - np.float32(1.0)
    elif wl.x_dist == "uniform_01":
        x = rng.random((batch, wl.n), dtype=np.float32)
    elif wl.x_dist == "relu_normal":
        x = np.maximum(rng.standard_normal((batch, wl.n), dtype=np.float32), np.float32(0.0))
    else:
        raise ValueError(wl.x_dist)
    return np.ascontiguousarray(x.astype(np.float32))


# ---- the five benchmark configurations --------------------------------------

CFG1_TINY_SHAC = Workload(1, "tiny_shac_256x128", 256, 128, 0.90, 32, QUANT_KMEANS,
                          ("shac",), (1,), "uniform_pm1")
CFG2_DENSE_HAC = Workload(2, "dense_hac_4096x4096_k256", 4096, 4096, 0.0, 256, QUANT_UNIFORM,
                          ("hac",), (1, 64), "uniform_pm1")
CFG3_FC_SHAC = Workload(3, "fc_shac_25088x4096_p96_k32", 25088, 4096, 0.96, 32, QUANT_KMEANS,
                        ("shac",), (1, 16, 128), "relu_normal")
CFG4_CONV = Workload(4, "conv3x3_512_im2col_4608x512_p60_k64", 4608, 512, 0.60, 64, QUANT_KMEANS,
                     ("shac", "hac"), (6272,), "relu_normal")

SWEEP_SPARSITY = (0.0, 0.50, 0.80, 0.90, 0.95, 0.99)
SWEEP_K = (2, 8, 32, 256, 1024)


def sweep_cells(n: int = 4096, m: int = 4096):
    """Configuration 5: sparsity x k grid on one He-init layer (same W for all cells)."""
    cells = []
    for si, s in enumerate(SWEEP_SPARSITY):
        for ki, k in enumerate(SWEEP_K):
            cells.append(Workload(5, f"sweep_{n}x{m}_p{int(round(s * 100))}_k{k}", n, m, s, k,
                                  QUANT_KMEANS, ("hac", "shac"), (1, 32), "uniform_pm1",
                                  item=0))
    return cells


def paper_shaped_cells():
    """The three fully connected shapes of the paper's format comparison (Sect. V-C)."""
    cells = []
    for (n, m) in ((512, 4096), (4096, 4096), (4096, 10)):
        for p in (0.60, 0.90, 0.99):
            for k in (32, 256):
                cells.append(Workload(6, f"paper_{n}x{m}_p{int(p * 100)}_k{k}", n, m, p, k,
                                      QUANT_KMEANS, ("hac", "shac"), (8,), "uniform_01",
                                      item=n + m))
    return cells


def scaled(wl: Workload, n: int, m: int, batches=None) -> Workload:
    """Same recipe on a smaller shape (used by fast tests)."""
    return dataclasses.replace(wl, n=n, m=m, name=f"{wl.name}_as_{n}x{m}",
                               batches=tuple(batches) if batches is not None else wl.batches)


ALL_MAIN = (CFG1_TINY_SHAC, CFG2_DENSE_HAC, CFG3_FC_SHAC, CFG4_CONV)
