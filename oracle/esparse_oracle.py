"""CPU oracle for the E-Sparse hot path -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

A plain, slow, fp64 restatement of what the path computes, written from the
paper's definitions.  It shares no code with the CUDA library and never calls
it; only the tests, the smoke check and the benchmark's CPU-baseline leg may
import it.

Steps (paper section / equation each one follows):

* ``channel_norm``      amplitude AM_c = ||X_c||_2                      (Eq. 2)
* ``channel_entropy``   information richness IR_c = -sum_k p_k log p_k   (Eq. 1, K = 100 bins)
* ``channel_score``     s_c = IR_c + alpha * AM_c                       (bracket of Eq. 3)
* ``metric``            xi[j,c] = |W[j,c]| * s_c                        (Eq. 3)
* ``global_naive_shuffle``  sort channels by the mean of xi, deal neighbours
  into different groups of M                                           (Section "Channel Shuffle", Fig. 3a)
* ``local_block_shuffle``   greedy best-improvement swaps inside blocks of 256 (Algorithm 1, Eq. 5)
* ``select_compress``   keep the 2 largest xi of every 4 consecutive permuted
  channels; emit kept values + 2-bit positions                         (Sections "Introduction"/"Sparse-GEMM", step (1))
* ``product``           Y = X P W_s^T with fp64 accumulation            (Eq. 4's layer product)

Readings of points the paper leaves open (alpha, bin range, log base, dealing
geometry, tie-breaks, exact row sums) are stated at each function.

Parity with the authors' own implementation is unpinned: the paper prints no
number that depends on these readings and can be reproduced without its models
and datasets.  Internal correctness is pinned by the CPU tests (closed forms,
invariants, brute force).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from typing import Optional, Tuple

import numpy as np

BINS = 100          # K in Eq. 1
LBS_BLOCK = 256     # m in the local block shuffle
NEAR_TIE_REL = 1e-6
_FIXED_SCALE = 2.0 ** -24   # every finite fp16 magnitude is an integer multiple of this

_HERE = os.path.dirname(os.path.abspath(__file__))
_LBS_SRC = os.path.join(_HERE, "lbs_oracle.c")
_LBS_SO = os.path.join(_HERE, "_lbs_oracle.so")
_lbs_lib = None


# ----------------------------------------------------------------------------- build / load the C part
def build_c(force: bool = False) -> str:
    """Compile the block-shuffle oracle (plain C, no FMA contraction)."""
    if force or not os.path.exists(_LBS_SO) or os.path.getmtime(_LBS_SO) < os.path.getmtime(_LBS_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-o", _LBS_SO, _LBS_SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LBS_SO


def _lib():
    global _lbs_lib
    if _lbs_lib is None:
        lib = ctypes.CDLL(build_c())
        lib.lbs_oracle_run.restype = ctypes.c_longlong
        lib.lbs_oracle_run.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_long, ctypes.c_void_p,
                                       ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_void_p, ctypes.c_void_p]
        lib.lbs_oracle_objective.restype = ctypes.c_double
        lib.lbs_oracle_objective.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_long,
                                             ctypes.c_void_p, ctypes.c_void_p]
        lib.lbs_oracle_group_value.restype = ctypes.c_double
        lib.lbs_oracle_group_value.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_long, ctypes.c_void_p,
                                               ctypes.c_void_p]
        _lbs_lib = lib
    return _lbs_lib


def oracle_threads() -> int:
    """Threads the C part uses (OpenMP default = cores available to the process)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


# ----------------------------------------------------------------------------- O1 norm
def channel_norm(xcal: np.ndarray) -> np.ndarray:
    """Eq. 2: AM_c = sqrt(sum_t x_tc^2).  Plain L2 norm, no division by T; fp64 accumulation."""
    x = np.asarray(xcal).astype(np.float64)
    return np.sqrt((x * x).sum(axis=0))


# ----------------------------------------------------------------------------- O2 entropy
def channel_histogram(xcal: np.ndarray, bins: int = BINS, global_range: bool = False) -> np.ndarray:
    """Counts n[c,k] of Eq. 1's bins.

    global_range=True is the other reading of "divide it into K bins": one range [lo, hi] for the whole layer
    (minimum and maximum over all channels) instead of each channel's own.

    Reading: the K bins are equal-width on the channel's own range [lo_c, hi_c],
    left-closed, the maximum falls in the last bin; raw signed values are binned.
    A constant channel has no range; its counts are all put in bin 0.
    bin(x) = min(K-1, floor((x - lo) * K / (hi - lo))) evaluated in fp64, which is the
    exact bin for fp16 inputs (numerator exact, quotient correctly rounded).
    """
    xcal = np.asarray(xcal)
    T, C = xcal.shape
    counts = np.zeros((C, bins), dtype=np.int64)
    for c0 in range(0, C, 1024):                      # column chunks only bound the temporaries
        x = xcal[:, c0:c0 + 1024].astype(np.float64)
        w = x.shape[1]
        lo = x.min(axis=0)
        hi = x.max(axis=0)
        if global_range:
            lo = np.full(w, float(xcal.min()))
            hi = np.full(w, float(xcal.max()))
        rng = hi - lo
        safe = np.where(rng > 0, rng, 1.0)
        idx = np.floor(((x - lo[None, :]) * float(bins)) / safe[None, :])
        idx = np.minimum(idx, bins - 1).astype(np.int64)
        idx[:, rng == 0] = 0
        flat = idx + np.arange(w, dtype=np.int64)[None, :] * bins
        counts[c0:c0 + w] = np.bincount(flat.ravel(), minlength=w * bins).reshape(w, bins)
    return counts


def entropy_from_counts(counts: np.ndarray, T: int) -> np.ndarray:
    """Eq. 1 with natural log; empty bins contribute 0; bins summed in index order."""
    C, K = counts.shape
    ir = np.zeros(C, dtype=np.float64)
    for k in range(K):
        n = counts[:, k].astype(np.float64)
        p = n / float(T)
        term = np.where(n > 0, p * np.log(np.where(n > 0, p, 1.0)), 0.0)
        ir = ir - term
    return ir


def channel_entropy(xcal: np.ndarray, bins: int = BINS, global_range: bool = False) -> np.ndarray:
    x = np.asarray(xcal)
    return entropy_from_counts(channel_histogram(x, bins, global_range), x.shape[0])


# ----------------------------------------------------------------------------- O3 score / metric
def channel_score(ir: np.ndarray, am: np.ndarray, alpha: float,
                  use_entropy: bool = True, use_norm: bool = True) -> np.ndarray:
    """s_c = IR_c + alpha * AM_c (bracket of Eq. 3).  alpha is the caller's: the paper never sets it.
    use_entropy=False gives the norm-only baseline of the ablation table; use_norm=False drops the norm."""
    s = np.zeros_like(np.asarray(am, dtype=np.float64))
    if use_entropy:
        s = s + np.asarray(ir, dtype=np.float64)
    if use_norm:
        s = s + float(alpha) * np.asarray(am, dtype=np.float64)
    return s


def metric(W: np.ndarray, s: np.ndarray) -> np.ndarray:
    """Eq. 3: xi[j,c] = |W[j,c]| * s_c, one fp64 multiply per element."""
    return np.abs(np.asarray(W).astype(np.float64)) * np.asarray(s, dtype=np.float64)[None, :]


def abs_fixed(W: np.ndarray) -> np.ndarray:
    """|W| as exact integers in units of 2^-24 (every finite fp16 is such a multiple)."""
    a = np.abs(np.asarray(W).astype(np.float64)) * (2.0 ** 24)
    out = a.astype(np.int64)
    assert np.array_equal(out.astype(np.float64), a)
    return out


# ----------------------------------------------------------------------------- O4 global naive shuffle
def channel_mean_metric(W: np.ndarray, s: np.ndarray) -> np.ndarray:
    """Mean of xi over the No rows of each channel: (s_c * sum_j |W[j,c]|) / No.
    The column sum of |W| is taken exactly (integers of 2^-24), so it does not depend on row order."""
    No = W.shape[0]
    colsum = np.zeros(W.shape[1], dtype=np.int64)
    step = max(1, (1 << 24) // max(W.shape[1], 1))     # row blocks only bound the temporaries: integer sums are exact
    for r0 in range(0, No, step):
        colsum += abs_fixed(W[r0:r0 + step]).sum(axis=0)
    a = colsum.astype(np.float64) * _FIXED_SCALE
    return (np.asarray(s, dtype=np.float64) * a) / float(No)


def global_naive_shuffle(mean: np.ndarray, m_group: int = 4) -> Tuple[np.ndarray, int]:
    """Sort channels by mean metric, descending (ties: lower channel index first), then deal them so
    that channels adjacent in rank land in different groups: with G = C / M groups, the channel of
    rank r goes to group r mod G, slot r div G, i.e. position (r mod G) * M + r div G.
    Returns (theta0, near-tie count) where theta0[p] = original channel placed at position p."""
    mean = np.asarray(mean, dtype=np.float64)
    C = mean.shape[0]
    assert C % m_group == 0
    G = C // m_group
    order = np.argsort(-mean, kind="stable")          # stable => lower index first among equals
    theta0 = np.empty(C, dtype=np.int32)
    r = np.arange(C)
    theta0[(r % G) * m_group + r // G] = order
    sm = mean[order]
    gap = sm[:-1] - sm[1:]
    near = int(np.count_nonzero(gap < NEAR_TIE_REL * np.abs(sm[:-1])))
    return theta0, near


# ----------------------------------------------------------------------------- O5 local block shuffle
def _as_u16(W: np.ndarray) -> np.ndarray:
    W = np.ascontiguousarray(np.asarray(W, dtype=np.float16))
    return W.view(np.uint16)


def objective(W: np.ndarray, s: np.ndarray, theta: np.ndarray) -> float:
    """Eq. 5: total retained metric under the channel order theta (2 of every 4)."""
    w = _as_u16(W)
    s = np.ascontiguousarray(s, dtype=np.float64)
    th = np.ascontiguousarray(theta, dtype=np.int32)
    return float(_lib().lbs_oracle_objective(w.ctypes.data, w.shape[0], w.shape[1], w.shape[1],
                                             s.ctypes.data, th.ctypes.data))


def group_value(W: np.ndarray, s: np.ndarray, channels) -> float:
    w = _as_u16(W)
    s = np.ascontiguousarray(s, dtype=np.float64)
    ch = np.ascontiguousarray(channels, dtype=np.int32)
    return float(_lib().lbs_oracle_group_value(w.ctypes.data, w.shape[0], w.shape[1], s.ctypes.data, ch.ctypes.data))


@dataclass
class LbsInfo:
    swaps_total: int = 0
    swaps_per_block: np.ndarray = field(default_factory=lambda: np.zeros(0, dtype=np.int64))
    near_tie_swaps: int = 0


def local_block_shuffle(W: np.ndarray, s: np.ndarray, theta0: np.ndarray, block: int = LBS_BLOCK,
                        max_swaps: int = 0, incremental: bool = True) -> Tuple[np.ndarray, LbsInfo]:
    """Algorithm 1, lines 3-14.  Blocks of `block` positions (the last one may be shorter).  In each
    block: over all position pairs i<j in different groups, gain = retained sum of the two groups
    after exchanging the channels - before; take the largest (ties: smallest (i,j)); apply it if > 0,
    else stop.  max_swaps > 0 caps the swaps per block."""
    w = _as_u16(W)
    s = np.ascontiguousarray(s, dtype=np.float64)
    theta = np.ascontiguousarray(theta0, dtype=np.int32).copy()
    C = w.shape[1]
    nblocks = (C + block - 1) // block
    per_block = np.zeros(nblocks, dtype=np.int64)
    near = ctypes.c_longlong(0)
    total = _lib().lbs_oracle_run(w.ctypes.data, w.shape[0], C, C, s.ctypes.data, theta.ctypes.data,
                                  int(block), int(max_swaps), 1 if incremental else 0,
                                  per_block.ctypes.data, ctypes.addressof(near))
    if total < 0:
        raise ValueError("bad shapes for local_block_shuffle")
    return theta, LbsInfo(int(total), per_block, int(near.value))


# ----------------------------------------------------------------------------- O6 select + compress
LEGAL_NIBBLES = (0x4, 0x8, 0xC, 0x9, 0xD, 0xE)   # idx0 | idx1 << 2 with idx0 < idx1


def select_compress(W: np.ndarray, s: np.ndarray, theta: np.ndarray):
    """Per row and per group of 4 consecutive permuted channels: rank the 4 candidates by xi descending
    (ties: lower position first), keep the first 2, let idx0 < idx1 be their positions.
    vals[j,2g+e] = W[j, theta[4g+idx_e]] (bit copies); nibble = idx0 | idx1<<2; meta[j, g//2] holds group
    g in its low (g even) or high (g odd) nibble.
    Returns (vals f16 [No,C/2], meta u8 [No,C/8], near_tie bool [No,C/4])."""
    W = np.asarray(W, dtype=np.float16)
    No, C = W.shape
    assert C % 8 == 0
    G = C // 4
    theta = np.asarray(theta, dtype=np.int64)
    Wp = W[:, theta]
    xi = (np.abs(Wp.astype(np.float64)) * np.asarray(s, dtype=np.float64)[theta][None, :]).reshape(No, G, 4)
    rank = np.argsort(-xi, axis=2, kind="stable")
    keep = np.sort(rank[:, :, :2], axis=2)
    idx0, idx1 = keep[:, :, 0], keep[:, :, 1]
    Wg = Wp.reshape(No, G, 4)
    vals = np.empty((No, G, 2), dtype=np.float16)
    vals[:, :, 0] = np.take_along_axis(Wg, idx0[:, :, None], axis=2)[:, :, 0]
    vals[:, :, 1] = np.take_along_axis(Wg, idx1[:, :, None], axis=2)[:, :, 0]
    nib = (idx0 | (idx1 << 2)).astype(np.uint8)
    meta = (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8)
    xs = np.take_along_axis(xi, rank, axis=2)
    near = (xs[:, :, 1] - xs[:, :, 2]) < NEAR_TIE_REL * xs[:, :, 1]
    return vals.reshape(No, C // 2), meta, near


def select_compress_nm(W: np.ndarray, s: np.ndarray, theta: np.ndarray, n_keep: int = 4, m_group: int = 8):
    """General N:M selection (the paper's 4:8 rows of Table 1; "prune N values out of M consecutive values in the
    channel dimension"): per row and per group of M consecutive permuted channels keep the n_keep largest xi (ties: lower
    position first).  There is no tensor-core form for 4:8, so the compressed form is plain: vals[j, g*n_keep + e] =
    the kept weights of group g in position order (bit copies), mask[j, g*M/8 + b] = bit p%8 set iff position p = 8b + p%8
    of the group is kept.  Returns (vals f16 [No, C*n_keep/M], mask u8 [No, C/8], near_tie bool [No, C/M]) where a
    near-tie is a relative gap < 1e-6 between the last kept and the first dropped metric."""
    W = np.asarray(W, dtype=np.float16)
    No, C = W.shape
    assert m_group % 8 == 0 and C % m_group == 0 and 0 < n_keep < m_group
    G = C // m_group
    theta = np.asarray(theta, dtype=np.int64)
    Wp = W[:, theta]
    xi = (np.abs(Wp.astype(np.float64)) * np.asarray(s, dtype=np.float64)[theta][None, :]).reshape(No, G, m_group)
    rank = np.argsort(-xi, axis=2, kind="stable")
    keep = np.sort(rank[:, :, :n_keep], axis=2)
    Wg = Wp.reshape(No, G, m_group)
    vals = np.take_along_axis(Wg, keep, axis=2)
    kept = np.zeros((No, G, m_group), dtype=bool)
    np.put_along_axis(kept, keep, True, axis=2)
    mask = np.packbits(kept.reshape(No, C), axis=1, bitorder="little")
    xs = np.take_along_axis(xi, rank, axis=2)
    near = (xs[:, :, n_keep - 1] - xs[:, :, n_keep]) < NEAR_TIE_REL * xs[:, :, n_keep - 1]
    return vals.reshape(No, G * n_keep), mask, near


def unpack_meta(meta: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """meta u8 [No, C/8] -> (idx0, idx1) int arrays [No, C/4]."""
    meta = np.asarray(meta, dtype=np.uint8)
    No = meta.shape[0]
    nib = np.empty((No, meta.shape[1] * 2), dtype=np.uint8)
    nib[:, 0::2] = meta & 0xF
    nib[:, 1::2] = meta >> 4
    return (nib & 3).astype(np.int64), (nib >> 2).astype(np.int64)


def decompress_permuted(vals: np.ndarray, meta: np.ndarray) -> np.ndarray:
    """Dense [No, C] matrix in PERMUTED channel order, zeros where pruned."""
    vals = np.asarray(vals, dtype=np.float16)
    No, half = vals.shape
    G = half // 2
    idx0, idx1 = unpack_meta(meta)
    out = np.zeros((No, G, 4), dtype=np.float16)
    v = vals.reshape(No, G, 2)
    np.put_along_axis(out, idx0[:, :, None], v[:, :, 0:1], axis=2)
    np.put_along_axis(out, idx1[:, :, None], v[:, :, 1:2], axis=2)
    return out.reshape(No, G * 4)


def decompress(vals: np.ndarray, meta: np.ndarray, theta: np.ndarray) -> np.ndarray:
    """Dense [No, C] matrix in ORIGINAL channel order: column theta[p] receives permuted column p."""
    wp = decompress_permuted(vals, meta)
    out = np.zeros_like(wp)
    out[:, np.asarray(theta, dtype=np.int64)] = wp
    return out


# ----------------------------------------------------------------------------- O7 product
def product(X: np.ndarray, vals: np.ndarray, meta: np.ndarray, theta: Optional[np.ndarray]) -> np.ndarray:
    """Y[t,j] = sum_p Ws[j,p] * X[t, theta[p]] in fp64 (inputs widened exactly), Ws = permuted pruned weight.
    theta None = identity."""
    X = np.asarray(X, dtype=np.float16).astype(np.float64)
    wp = decompress_permuted(vals, meta).astype(np.float64)
    if theta is not None:
        X = X[:, np.asarray(theta, dtype=np.int64)]
    return X @ wp.T


def product_entries(X: np.ndarray, vals: np.ndarray, meta: np.ndarray, theta: Optional[np.ndarray],
                    rows: np.ndarray, cols: np.ndarray) -> np.ndarray:
    """The block Y[rows][:, cols] of `product`, computed without forming the whole output."""
    rows = np.asarray(rows, dtype=np.int64)
    cols = np.asarray(cols, dtype=np.int64)
    return product(np.asarray(X)[rows], np.asarray(vals)[cols], np.asarray(meta)[cols], theta)


def layer_output(Y: np.ndarray, bias: Optional[np.ndarray] = None, relu: bool = False) -> np.ndarray:
    """What a linear layer hands on: the product plus a per-feature bias (the same for every token), then ReLU.
    The paper times the bare product (Table 5); OPT's linears carry a bias and its first feed-forward linear a ReLU."""
    out = np.asarray(Y, dtype=np.float64).copy()
    if bias is not None:
        b = np.asarray(bias).astype(np.float64)
        assert b.shape == (out.shape[1],)
        for t in range(out.shape[0]):
            out[t, :] = out[t, :] + b
    if relu:
        out[out < 0.0] = 0.0
    return out


# ----------------------------------------------------------------------------- whole producer
@dataclass
class PruneResult:
    norm: np.ndarray
    entropy: np.ndarray
    score: np.ndarray
    mean: np.ndarray
    theta0: np.ndarray
    theta: np.ndarray
    vals: np.ndarray
    meta: np.ndarray
    near_tie_groups: np.ndarray
    near_tie_sort: int
    lbs: LbsInfo
    obj_identity: float
    obj_after_gns: float
    obj_after_lbs: float


def metric_prune(W: np.ndarray, xcal: np.ndarray, alpha: float, *, bins: int = BINS,
                 use_entropy: bool = True, use_norm: bool = True, use_gns: bool = True, use_lbs: bool = True,
                 lbs_block: int = LBS_BLOCK, lbs_max_swaps: int = 0, score: Optional[np.ndarray] = None,
                 objectives: bool = True, global_bin_range: bool = False) -> PruneResult:
    """norm -> entropy -> score -> global shuffle -> block shuffle -> 2:4 selection -> compression."""
    W = np.asarray(W, dtype=np.float16)
    C = W.shape[1]
    # (with a supplied score the calibration activations are optional: the statistics are then not formed)
    am = channel_norm(xcal) if xcal is not None else None
    ir = channel_entropy(xcal, bins, global_bin_range) if xcal is not None else None
    s = channel_score(ir, am, alpha, use_entropy, use_norm) if score is None else np.asarray(score, np.float64)
    mean = channel_mean_metric(W, s)
    ident = np.arange(C, dtype=np.int32)
    if use_gns:
        theta0, near_sort = global_naive_shuffle(mean)
    else:
        theta0, near_sort = ident.copy(), 0
    if use_lbs:
        theta, info = local_block_shuffle(W, s, theta0, lbs_block, lbs_max_swaps)
    else:
        theta, info = theta0.copy(), LbsInfo()
    vals, meta, near = select_compress(W, s, theta)
    o_id = objective(W, s, ident) if objectives else float("nan")
    o_g = objective(W, s, theta0) if objectives else float("nan")
    o_l = objective(W, s, theta) if objectives else float("nan")
    return PruneResult(am, ir, s, mean, theta0, theta, vals, meta, near, near_sort, info, o_id, o_g, o_l)
