"""Full-size parity on the LLaMA-13B, LLaMA-65B and OPT-66B shaped layers (the 7B layer is covered in
test_gpu_spgemm_parity.py), in the launch configuration bench.py times: channel-major X, default plan.

The oracle cannot form these products whole, so it is applied to what it can compute one by one: the global shuffle of
all input channels (whole permutation, bit-exact), the 2-of-4 selection and compression of a seeded sample of feature rows
(bit-exact against the GPU's rows of `vals` and `meta`, which the GPU produced for the whole weight from the same scores),
and the product on sampled token rows x those feature rows plus the rows and columns at tile boundaries.
"""
import numpy as np
import pytest

from oracle import esparse_oracle as orc
from paper_2310_15929_b200 import inputs

pytestmark = pytest.mark.gpu

CASES = [
    # workload, linear, token counts
    (2, "q", (1, 4, 16, 64)), (2, "gate", (1, 64)), (2, "down", (4, 64)),
    (3, "q", (2048, 8192)), (3, "gate", (2048,)), (3, "down", (4096,)),
    (4, "q", (1, 32, 512, 4096)), (4, "fc1", (32, 4096)), (4, "fc2", (1, 512)),
]


@pytest.mark.parametrize("wl_index,lin,tokens", CASES)
def test_full_size_layer_sampled(wl_index, lin, tokens):
    from tests.gpu_util import GpuPrune, spgemm
    from tests.test_gpu_spgemm_parity import check, ref_entries
    wl = inputs.WORKLOADS[wl_index]
    N, K = wl.linears[lin]
    g = np.random.default_rng(1000 * wl_index + N + K)
    W = inputs.make_weight(wl, lin)
    s = 1.0 + g.random(K)
    # global shuffle over all K input channels on the GPU (no block shuffle: the oracle's table for these widths takes
    # hours) against the oracle's: the whole permutation and the near-tie count of the sort, bit-exact
    theta, near_sort = orc.global_naive_shuffle(orc.channel_mean_metric(W, s))
    gp = GpuPrune(W, None, 1.0, score=s, stats=True, use_lbs=0)
    assert np.array_equal(gp.perm.cpu().numpy(), theta)
    assert gp.stats.near_tie_sort == near_sort

    cols = np.unique(np.concatenate([g.choice(N, 40, replace=False), [0, 127, 128, 255, 256, 511, 512, N - 1]]))
    vals_ref, meta_ref, near = orc.select_compress(W[cols], s, theta)
    del W
    vals_gpu = gp.vals[cols].cpu().numpy()
    meta_gpu = gp.meta[cols].cpu().numpy()
    assert np.array_equal(meta_gpu, meta_ref)
    assert np.array_equal(vals_gpu.view(np.uint16), vals_ref.view(np.uint16))

    for M in tokens:
        X = inputs.make_gemm_x(wl, lin, M)
        Y = spgemm(X, gp.packed, theta, N, channel_major=True)
        rows = np.unique(np.concatenate([g.choice(M, min(M, 6), replace=False),
                                         [0, M - 1, min(M - 1, 119), min(M - 1, 120), min(M - 1, 239), min(M - 1, 240)]]))
        Yref = ref_entries(X, vals_gpu, meta_gpu, theta, rows, np.arange(len(cols)))
        check(Y[np.ix_(rows, cols)], Yref)
        del X, Y
