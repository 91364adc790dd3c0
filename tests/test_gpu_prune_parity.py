"""GPU parity of esp_metric_prune against the CPU oracle, through the C ABI.

Bars: integer outputs (histogram counts, permutation, metadata, kept values as bit patterns, swap and near-tie counts)
bit-exact; fp64 channel statistics within 1e-12 relative (the GPU adds the same exact squares in a different order and
uses a different log implementation).

Everything after the score is integer or exactly rounded fp64 work, so it is compared without any tolerance and without
any excuse: the GPU's score is first held to the oracle's at 1e-12, then the oracle is run on the GPU's OWN score and the
permutation, metadata, kept values, swap count, the three near-tie counts and the three objectives must all be identical.
"""
import math

import numpy as np
import pytest

from oracle import esparse_oracle as orc
from paper_2310_15929_b200 import inputs

pytestmark = pytest.mark.gpu

STAT_RTOL = 1e-12


def layer(seed, No, C, T, outliers=3):
    g = np.random.default_rng(seed)
    W = (g.standard_normal((No, C)) * 0.02).astype(np.float16)
    X = g.standard_normal((T, C))
    X[:, g.choice(C, outliers, replace=False)] *= 25
    return W, X.astype(np.float16)


def assert_identical_to_oracle(g, ref, check_stats=True):
    """Every discrete output and every exactly-rounded fp64 output of one esp_metric_prune call against the oracle's
    result for the same score: no tolerance, no excuse."""
    vals, meta, perm = g.host()
    assert np.array_equal(perm, ref.theta)
    assert np.array_equal(meta, ref.meta)
    assert np.array_equal(vals.view(np.uint16), ref.vals.view(np.uint16))
    if check_stats:
        assert g.stats.near_tie_groups == int(ref.near_tie_groups.sum())
        assert g.stats.near_tie_sort == ref.near_tie_sort
        assert g.stats.near_tie_swaps == ref.lbs.near_tie_swaps
        assert g.stats.lbs_swaps_total == ref.lbs.swaps_total
        assert g.stats.obj_identity == ref.obj_identity           # same exact sums, same order of additions
        assert g.stats.obj_after_gns == ref.obj_after_gns
        assert g.stats.obj_after_lbs == ref.obj_after_lbs


def assert_statistics(g, X, alpha, **score_kw):
    """AM_c, IR_c, s_c of the GPU against the oracle's at the statistics bar; returns the GPU's score."""
    am, ir = orc.channel_norm(X), orc.channel_entropy(X, global_range=bool(score_kw.pop("global_range", False)))
    s = orc.channel_score(ir, am, alpha, **score_kw)
    assert np.allclose(g.norm.cpu().numpy(), am, rtol=STAT_RTOL, atol=0)
    assert np.allclose(g.entropy.cpu().numpy(), ir, rtol=STAT_RTOL, atol=1e-14)
    gs = g.score.cpu().numpy()
    assert np.allclose(gs, s, rtol=STAT_RTOL, atol=1e-14)
    return gs


@pytest.mark.parametrize("No,C,T", [(512, 512, 128), (200, 264, 333), (96, 1024, 77)])
def test_channel_statistics(No, C, T):
    from tests.gpu_util import GpuPrune
    W, X = layer(100 + C, No, C, T)
    X[:, 5] = 3.0                                              # a constant channel: entropy exactly 0
    X[: T // 2, 6] = -1.0; X[T // 2:, 6] = 1.0                 # two values
    alpha = 1.0 / math.sqrt(T)
    g = GpuPrune(W, X, alpha, use_lbs=0)
    assert_statistics(g, X, alpha)
    assert g.entropy[5].item() == 0.0
    if T % 2 == 0:
        assert abs(g.entropy[6].item() - math.log(2)) < 1e-14


@pytest.mark.parametrize("No,C,T,block", [(512, 512, 128, 256), (200, 264, 90, 256), (130, 520, 64, 128), (64, 64, 50, 16)])
def test_shuffle_select_compress_bit_exact_given_oracle_scores(No, C, T, block):
    """With the oracle's s_c handed in, everything downstream must be identical bit for bit."""
    from tests.gpu_util import GpuPrune
    W, X = layer(200 + C, No, C, T)
    alpha = 1.0 / math.sqrt(T)
    ref = orc.metric_prune(W, X, alpha, lbs_block=block)
    g = GpuPrune(W, None, alpha, score=ref.score, lbs_block=block)
    assert_identical_to_oracle(g, ref)
    assert ref.lbs.swaps_total > 0


@pytest.mark.parametrize("No,C,block,cap", [(1100, 520, 256, 0), (1024, 256, 256, 12), (2100, 264, 256, 6)])
def test_block_shuffle_tall_weights_bit_exact(No, C, block, cap):
    """From 769 rows on the table kernels read a candidate's column four 16-byte loads ahead and finish with a ragged
    tail: padded row counts of 1280 (one unrolled pass + a tail), 1024 (no tail) and 2304 (two passes + a tail), with a
    ragged last block of channels."""
    from tests.gpu_util import GpuPrune
    g0 = np.random.default_rng(7000 + No)
    W = (g0.standard_normal((No, C)) * 0.02 * np.sqrt(4.0 / g0.chisquare(4.0, size=(No, 1)))).astype(np.float16)
    s = 1.0 + 3.0 * g0.random(C)
    ref = orc.metric_prune(W, None, 1.0, score=s, lbs_block=block, lbs_max_swaps=cap)
    g = GpuPrune(W, None, 1.0, score=s, lbs_block=block, lbs_max_swaps=cap)
    assert_identical_to_oracle(g, ref)
    assert ref.lbs.swaps_total > 0


def test_llama7b_q_projection_full_size_block_shuffle():
    """Workload 1's q projection whole (4096 x 4096, 16 shuffle blocks, Student-t rows): global shuffle, block shuffle
    capped at 4 swaps per block on both sides (the oracle's table alone is 4.3e9 row evaluations), selection and
    compression, all bit-exact given the same score."""
    from tests.gpu_util import GpuPrune
    wl = inputs.WORKLOADS[1]
    W = inputs.make_weight(wl, "q")
    s = 1.0 + 3.0 * np.random.default_rng(11).random(W.shape[1])
    ref = orc.metric_prune(W, None, 1.0, score=s, lbs_max_swaps=4)
    g = GpuPrune(W, None, 1.0, score=s, lbs_max_swaps=4)
    assert_identical_to_oracle(g, ref)
    assert ref.lbs.swaps_total == 4 * 16


@pytest.mark.parametrize("wl_index,lin", [(3, "gate"), (4, "fc1")])
def test_block_shuffle_all_rows_of_the_widest_layers(wl_index, lin):
    """All 22016 / 36864 output rows of the widest LLaMA-65B / OPT-66B linears on one block of 256 input channels
    (the per-row record of the table kernels then fills most of shared memory), two swaps, bit-exact."""
    from tests.gpu_util import GpuPrune
    wl = inputs.WORKLOADS[wl_index]
    W = inputs.make_weight(wl, lin, C=256)
    s = 1.0 + 3.0 * np.random.default_rng(12 + wl_index).random(256)
    ref = orc.metric_prune(W, None, 1.0, score=s, lbs_max_swaps=2)
    g = GpuPrune(W, None, 1.0, score=s, lbs_max_swaps=2)
    assert_identical_to_oracle(g, ref)
    assert ref.lbs.swaps_total == 2


@pytest.mark.parametrize("toggles", [dict(use_gns=0, use_lbs=0), dict(use_gns=1, use_lbs=0), dict(use_gns=0, use_lbs=1),
                                     dict(use_entropy=0), dict(use_norm=0), dict(lbs_max_swaps=5)])
def test_ablation_toggles(toggles):
    from tests.gpu_util import GpuPrune
    W, X = layer(300, 128, 256, 100)
    alpha = 0.25
    kw = dict(use_entropy=True, use_norm=True, use_gns=True, use_lbs=True, lbs_max_swaps=0)
    kw.update({k: (bool(v) if k.startswith("use") else v) for k, v in toggles.items()})
    g = GpuPrune(W, X, alpha, **toggles)
    gs = assert_statistics(g, X, alpha, use_entropy=kw["use_entropy"], use_norm=kw["use_norm"])
    ref = orc.metric_prune(W, X, alpha, score=gs, **kw)       # the oracle on the GPU's own score
    assert_identical_to_oracle(g, ref)
    if not kw["use_lbs"]:
        assert g.stats.lbs_swaps_total == 0 and g.stats.obj_after_lbs == g.stats.obj_after_gns
    if not kw["use_gns"]:                                     # the block shuffle then starts from the identity order
        assert g.stats.near_tie_sort == 0 and g.stats.obj_after_gns == g.stats.obj_identity


def test_config0_end_to_end():
    """Workload 0: 512x512 layer, 128 calibration tokens, 8 outlier channels x20, both values of alpha."""
    from tests.gpu_util import GpuPrune
    wl = inputs.WORKLOADS[0]
    W, X = inputs.make_weight(wl, "fc"), inputs.make_calibration(wl, "fc")
    for alpha in (1.0, 1.0 / math.sqrt(X.shape[0])):
        g = GpuPrune(W, X, alpha)
        gs = assert_statistics(g, X, alpha)
        ref = orc.metric_prune(W, X, alpha, score=gs)
        assert_identical_to_oracle(g, ref)
        assert g.stats.obj_after_lbs >= g.stats.obj_after_gns > 0.0
        # run-to-run determinism
        g2 = GpuPrune(W, X, alpha)
        for a, c in zip(g.host(), g2.host()):
            assert np.array_equal(a.view(np.uint8), c.view(np.uint8))


def test_llama7b_shaped_slice():
    """Config 1 distributions (Student-t rows, 1 % outlier channels x30) on a reduced q-projection:
    all 4096 input channels (16 shuffle blocks), 256 output rows, 2048 calibration tokens."""
    from tests.gpu_util import GpuPrune
    wl = inputs.WORKLOADS[1]
    W = inputs.make_weight(wl, "q", No=256)
    X = inputs.make_calibration(wl, "q", T=2048)
    alpha = 1.0 / math.sqrt(X.shape[0])
    g = GpuPrune(W, X, alpha, lbs_max_swaps=24)
    gs = assert_statistics(g, X, alpha)
    ref = orc.metric_prune(W, X, alpha, score=gs, lbs_max_swaps=24)
    assert_identical_to_oracle(g, ref)


def test_decompress_and_pack_roundtrip():
    import torch
    from paper_2310_15929_b200 import binding as b
    from tests.gpu_util import GpuPrune, DEV
    W, X = layer(400, 136, 264, 60)
    ref = orc.metric_prune(W, X, 0.3)
    g = GpuPrune(W, None, 0.3, score=ref.score)
    out = torch.empty(136, 264, dtype=torch.float16, device=DEV)
    b.esp_decompress(g.vals, g.meta, g.perm, 136, 264, out)
    assert np.array_equal(out.cpu().numpy().view(np.uint16), orc.decompress(ref.vals, ref.meta, ref.theta).view(np.uint16))
    # the packed copy holds exactly the kept values (as a multiset per tile) plus legal metadata
    packed = g.packed.cpu().numpy().reshape(2, 3, 18432)
    tile = packed[0, 0, :16384].view(np.float16).reshape(128, 64)
    unsw = np.empty_like(tile)
    for r in range(128):
        for q in range(8):
            unsw[r, q * 8:(q + 1) * 8] = tile[r, (q ^ (r & 7)) * 8:(q ^ (r & 7)) * 8 + 8]
    assert np.array_equal(unsw.view(np.uint16), ref.vals[:128, :64].view(np.uint16))
    nibbles = packed[:, :, 16384:]
    assert set(np.unique(nibbles & 0xF).tolist()) | set(np.unique(nibbles >> 4).tolist()) <= set(orc.LEGAL_NIBBLES)


@pytest.mark.parametrize("No,C,T", [(96, 256, 200), (200, 1024, 130)])
def test_four_of_eight_pattern(No, C, T):
    """4:8 (Table 1's second pattern): statistics, score, global shuffle in groups of 8, 4-of-8 selection and compression
    against the oracle run on the GPU's own score, bit-exact; the library refuses what 4:8 has no form for."""
    from paper_2310_15929_b200 import binding as b
    from tests.gpu_util import GpuPrune
    W, X = layer(70 + C, No, C, T)
    alpha = 1.0 / math.sqrt(T)
    gp = GpuPrune(W, X, alpha, stats=True, pack=False, n_keep=4, m_group=8, use_lbs=0)
    gs = assert_statistics(gp, X, alpha)
    theta0, near_sort = orc.global_naive_shuffle(orc.channel_mean_metric(W, gs), m_group=8)
    vals_ref, mask_ref, near = orc.select_compress_nm(W, gs, theta0, 4, 8)
    vals, mask, perm = gp.host()
    assert np.array_equal(perm, theta0)
    assert np.array_equal(mask, mask_ref)
    assert np.array_equal(vals.view(np.uint16), vals_ref.view(np.uint16))
    assert gp.stats.near_tie_groups == int(near.sum())
    assert gp.stats.near_tie_sort == near_sort
    with pytest.raises(b.EsparseError) as e:
        GpuPrune(W, X, alpha, stats=False, pack=False, n_keep=4, m_group=8, use_lbs=1)
    assert e.value.status == b.ESP_ERR_UNSUPPORTED
    with pytest.raises(b.EsparseError) as e:
        GpuPrune(W, X, alpha, stats=False, pack=True, n_keep=4, m_group=8, use_lbs=0)
    assert e.value.status == b.ESP_ERR_UNSUPPORTED


@pytest.mark.parametrize("C,splits", [(264, (100, 37, 256, 3)), (1024, (77,)), (512, (1, 1, 700, 5000))])
def test_streaming_calibration_equals_one_shot(C, splits):
    """Chunked statistics (two passes over the chunks) against the oracle on the concatenation: counts bit-exact,
    norm / entropy / score to the statistics bar; then the streamed score drives the same pruning decisions."""
    from tests.gpu_util import GpuPrune, calibrate_in_chunks
    T = sum(splits)
    W, X = layer(900 + C, 128, C, T)
    X[:, 5] = 3.0
    X[-1, 7] = 1000.0                                           # the range of channel 7 is set by the last chunk
    alpha = 1.0 / math.sqrt(T)
    chunks, r = [], 0
    for n in splits:
        chunks.append(X[r: r + n]); r += n
    norm, ent, score, counts, score_d = calibrate_in_chunks(chunks, alpha)
    assert np.array_equal(counts, orc.channel_histogram(X))
    assert counts.sum(axis=1).tolist() == [T] * C
    am, ir = orc.channel_norm(X), orc.channel_entropy(X)
    assert np.allclose(norm, am, rtol=STAT_RTOL, atol=0)
    assert np.allclose(ent, ir, rtol=STAT_RTOL, atol=1e-14)
    assert np.allclose(score, orc.channel_score(ir, am, alpha), rtol=STAT_RTOL, atol=0)
    assert ent[5] == 0.0
    # ablation switches reach the streamed score too
    _, _, s_norm_only, _, _ = calibrate_in_chunks(chunks, alpha, use_entropy=0)
    assert np.allclose(s_norm_only, alpha * am, rtol=STAT_RTOL, atol=0)
    # the streamed score feeds the pruner without the calibration matrix
    ref = orc.metric_prune(W, None, alpha, use_lbs=False, score=score)
    g = GpuPrune(W, None, alpha, score=score, use_lbs=0)
    assert_identical_to_oracle(g, ref)


@pytest.mark.parametrize("No,C,T", [(128, 264, 333), (96, 1024, 200)])
def test_global_bin_range_variant(No, C, T):
    """Layer-wide bin range (the other reading of Eq. 1): entropy and score to the statistics bar, everything downstream
    identical to the oracle on the GPU's own score, and different from the per-channel reading on this input."""
    from tests.gpu_util import GpuPrune
    W, X = layer(300 + C, No, C, T)
    X[:, 9] = (X[:, 9].astype(np.float32) / 64).astype(np.float16)          # a narrow channel
    alpha = 1.0 / math.sqrt(T)
    g = GpuPrune(W, X, alpha, use_lbs=0, global_bin_range=1)
    gs = assert_statistics(g, X, alpha, global_range=True)
    assert g.entropy[9].item() < 0.5 * orc.channel_entropy(X)[9]
    ref = orc.metric_prune(W, X, alpha, use_lbs=False, global_bin_range=True, score=gs)
    assert_identical_to_oracle(g, ref)


# --------------------------------------------------------------------------- full width: workloads 2, 3, 4
@pytest.mark.parametrize("wl_index,lin", [(2, "q"), (2, "down"), (3, "down"), (4, "fc2")])
def test_channel_statistics_full_width_full_calibration(wl_index, lin):
    """Norm, entropy and score over all C input channels and all 16 x 2048 calibration tokens of the LLaMA-13B, LLaMA-65B
    and OPT-66B shaped layers (C = 5120, 13824, 22016, 36864).  The GPU processes the whole [T, C] matrix, once through
    esp_metric_prune and once as two uneven chunks through the streaming-calibration calls; the oracle, whose statistics
    are per channel, is applied to a seeded sample of channels: all outlier channels, the channels at the kernels' 64- and
    256-wide boundaries, and random ones.  Counts bit-exact, fp64 statistics to 1e-12."""
    import torch
    from tests.gpu_util import GpuPrune, calibrate_in_chunks, DEV
    wl = inputs.WORKLOADS[wl_index]
    C = wl.linears[lin][1]
    X = inputs.make_calibration(wl, lin)
    T = X.shape[0]
    assert T == 16 * 2048
    g0 = np.random.default_rng(500 + wl_index)
    out = inputs.outlier_channels(wl, lin)
    cols = np.unique(np.concatenate([out[:64], g0.choice(C, 160, replace=False),
                                     [0, 63, 64, 255, 256, C - 257, C - 256, C - 65, C - 64, C - 1]]))
    Xs = np.ascontiguousarray(X[:, cols])
    am, cnt = orc.channel_norm(Xs), orc.channel_histogram(Xs)
    ir = orc.entropy_from_counts(cnt, T)
    alpha = 1.0 / math.sqrt(T)
    s = orc.channel_score(ir, am, alpha)
    # one-shot path (what the benchmark's producer runs); the weight is a thin slice, the statistics do not read it
    W = inputs.make_weight(wl, lin, No=128)
    g = GpuPrune(W, X, alpha, use_lbs=0, stats=False, pack=False)
    assert np.allclose(g.norm.cpu().numpy()[cols], am, rtol=STAT_RTOL, atol=0)
    assert np.allclose(g.entropy.cpu().numpy()[cols], ir, rtol=STAT_RTOL, atol=1e-14)
    assert np.allclose(g.score.cpu().numpy()[cols], s, rtol=STAT_RTOL, atol=0)
    del g
    torch.cuda.empty_cache()
    # streaming path: exposes the counts themselves
    cut = 20000
    norm, ent, score, counts, _ = calibrate_in_chunks([X[:cut], X[cut:]], alpha)
    assert np.array_equal(counts[cols], cnt)
    assert counts.sum(axis=1).tolist() == [T] * C
    assert np.allclose(norm[cols], am, rtol=STAT_RTOL, atol=0)
    assert np.allclose(ent[cols], ir, rtol=STAT_RTOL, atol=1e-14)
    assert np.allclose(score[cols], s, rtol=STAT_RTOL, atol=0)
