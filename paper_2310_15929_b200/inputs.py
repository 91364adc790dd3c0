"""Seeded synthetic inputs for the E-Sparse hot path.

This module only draws random tensors.  It holds none of the method's
arithmetic (no norm, entropy, metric, shuffle, selection or product), so the
CPU oracle and the CUDA path can both be fed the *same bytes* from here
without sharing any code of the method itself.

The five workloads mirror public LLaMA / OPT layer dimensions.  They stand in
for the trained checkpoints and the C4 calibration text that the paper used
(Section "Experiments", calibration on 128 sequences), which are not
available offline; only shapes and the "a few channels carry outliers"
structure (Section "Observations") are reproduced.

Every tensor is drawn in fp64 from a counter-based Philox stream, cast to fp16
once (round-to-nearest-even), and returned as a numpy float16 array.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Tuple

import numpy as np

SEED_BASE = 231015929 * 1000

# tensor ids inside one (config, layer) seed namespace
_T_WEIGHT, _T_CALIB, _T_OUTLIER, _T_GEMM_X = 0, 1, 2, 3


@dataclass(frozen=True)
class Workload:
    """One synthetic layer family."""
    index: int
    name: str
    linears: Dict[str, Tuple[int, int]]      # name -> (No, C)  (out features, in channels)
    calib_tokens: int                        # T
    weight_sigma: float
    heavy_tail_rows: bool                    # Student-t(nu=4) row scales
    outlier_fraction: float                  # fraction of channels that are outliers
    outlier_count: int                       # used instead of the fraction when > 0
    outlier_scale: float
    gemm_tokens: Tuple[int, ...]             # the M values of the workload


def _llama(hidden: int, ffn: int) -> Dict[str, Tuple[int, int]]:
    return {
        "q": (hidden, hidden), "k": (hidden, hidden), "v": (hidden, hidden), "o": (hidden, hidden),
        "gate": (ffn, hidden), "up": (ffn, hidden), "down": (hidden, ffn),
    }


def _opt(hidden: int, ffn: int) -> Dict[str, Tuple[int, int]]:
    return {
        "q": (hidden, hidden), "k": (hidden, hidden), "v": (hidden, hidden), "o": (hidden, hidden),
        "fc1": (ffn, hidden), "fc2": (hidden, ffn),
    }


WORKLOADS = (
    Workload(0, "single-512", {"fc": (512, 512)}, 128, 0.02, False, 0.0, 8, 20.0, (128,)),
    Workload(1, "llama-7b-layer", _llama(4096, 11008), 16 * 2048, 0.02, True, 0.01, 0, 30.0, (1, 16, 128, 2048)),
    Workload(2, "llama-13b-layer", _llama(5120, 13824), 16 * 2048, 0.02, True, 0.01, 0, 30.0, (1, 4, 16, 64)),
    Workload(3, "llama-65b-layer", _llama(8192, 22016), 16 * 2048, 0.02, True, 0.01, 0, 30.0, (2048, 4096, 8192)),
    Workload(4, "opt-66b-layer", _opt(9216, 36864), 16 * 2048, 0.015, False, 0.005, 0, 60.0, (1, 32, 512, 4096)),
)


def _rng(workload: int, layer: int, tensor: int, extra: int = 0) -> np.random.Generator:
    seed = SEED_BASE + 100 * workload + 10 * layer + tensor
    return np.random.Generator(np.random.Philox(key=[seed, extra]))


def _to_f16(a: np.ndarray) -> np.ndarray:
    return a.astype(np.float16)


def layer_index(wl: Workload, linear: str) -> int:
    return list(wl.linears).index(linear)


def outlier_channels(wl: Workload, linear: str, C: int | None = None) -> np.ndarray:
    """Sorted indices of the outlier input channels of one linear."""
    if C is None:
        C = wl.linears[linear][1]
    n = wl.outlier_count if wl.outlier_count > 0 else int(round(wl.outlier_fraction * C))
    n = min(n, C)
    g = _rng(wl.index, layer_index(wl, linear), _T_OUTLIER)
    return np.sort(g.choice(C, size=n, replace=False))


def make_weight(wl: Workload, linear: str, No: int | None = None, C: int | None = None) -> np.ndarray:
    """W [No, C] fp16.  Optional No/C shrink the layer (same distribution, for quick tests)."""
    no_full, c_full = wl.linears[linear]
    No = no_full if No is None else No
    C = c_full if C is None else C
    li = layer_index(wl, linear)
    g = _rng(wl.index, li, _T_WEIGHT)
    out = np.empty((No, C), dtype=np.float16)
    if wl.heavy_tail_rows:
        chi2 = _rng(wl.index, li, _T_WEIGHT, 1).chisquare(4.0, size=No)
        row_scale = np.sqrt(4.0 / chi2)
    else:
        row_scale = np.ones(No)
    step = max(1, (1 << 22) // max(C, 1))
    for r0 in range(0, No, step):
        r1 = min(No, r0 + step)
        blk = g.standard_normal((r1 - r0, C)) * (wl.weight_sigma * row_scale[r0:r1, None])
        out[r0:r1] = _to_f16(blk)
    return out


def _activations(wl: Workload, linear: str, tokens: int, C: int, tensor: int, extra: int) -> np.ndarray:
    li = layer_index(wl, linear)
    g = _rng(wl.index, li, tensor, extra)
    scale = np.ones(C)
    scale[outlier_channels(wl, linear, C)] = wl.outlier_scale
    out = np.empty((tokens, C), dtype=np.float16)
    step = max(1, (1 << 22) // max(C, 1))
    for r0 in range(0, tokens, step):
        r1 = min(tokens, r0 + step)
        out[r0:r1] = _to_f16(g.standard_normal((r1 - r0, C)) * scale[None, :])
    return out


def make_calibration(wl: Workload, linear: str, T: int | None = None, C: int | None = None) -> np.ndarray:
    """Calibration activations Xcal [T, C] fp16."""
    T = wl.calib_tokens if T is None else T
    C = wl.linears[linear][1] if C is None else C
    return _activations(wl, linear, T, C, _T_CALIB, 0)


def make_gemm_x(wl: Workload, linear: str, M: int, C: int | None = None) -> np.ndarray:
    """GEMM activations X [M, C] fp16: a fresh draw with the same outlier channels."""
    C = wl.linears[linear][1] if C is None else C
    return _activations(wl, linear, M, C, _T_GEMM_X, M)


def distinct_shapes(wl: Workload):
    """(No, C) -> first linear name having that shape, in layer order."""
    seen = {}
    for name, shape in wl.linears.items():
        seen.setdefault(shape, name)
    return seen
