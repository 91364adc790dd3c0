"""esp_spgemm_static: the product for callers that cannot allocate device memory.

A host engine that owns all of HBM through its own pool and runs operators from a hook with no workspace
argument -- or a serving thread that must stay clear of cudaMalloc because it can stall the device --
gets the same product from esp_spgemm_static, whose scratch (the transposed copy of X and, beyond 256 tokens, the
operand images of X with their flags) is a fixed 8 MiB array inside the library.  This file checks, through the C ABI, that it returns what esp_spgemm returns on two calls in
a row (the second call reuses the array with other sizes, so stale contents of the first must not leak), that it
agrees with the CPU oracle, and that sizes beyond the array are refused before anything is launched.

Collected last on purpose (file name): a failure here cannot hide a failure elsewhere in a -x run.
"""
import numpy as np
import pytest

from paper_2310_15929_b200 import binding as b

A = 0x10000   # fake 16-byte-aligned address: the size check must come before any use of the pointers


def test_sizes_beyond_the_built_in_scratch_are_refused():
    K = 4096
    m_ok = b.ESP_STATIC_SCRATCH_BYTES // (K * 2)            # 1024 tokens fill the array exactly
    too_big = b.esp_spgemm_static_raw(A, m_ok + 1, K, K, A, None, 512, A, 512, b.ESP_OUT_F16, None)
    assert too_big == b.ESP_ERR_STATIC_LIMIT
    assert "esp_spgemm_static" in b.esp_status_string(too_big)
    assert b.esp_spgemm_static_raw(A, 16, K, K, A, None, 512, A, 100, b.ESP_OUT_F16, None) == b.ESP_ERR_SHAPE
    assert b.esp_spgemm_static_raw(None, 16, K, K, A, None, 512, A, 512, b.ESP_OUT_F16, None) == b.ESP_ERR_INVALID_ARG


@pytest.mark.gpu
def test_static_scratch_matches_workspace_path_twice_in_a_row():
    import torch
    from oracle import esparse_oracle as orc
    from tests.gpu_util import pack_on_gpu
    from tests.test_gpu_spgemm_parity import check, pruned, ref_product

    dev = torch.device("cuda:0")
    g = np.random.default_rng(42)
    # (N, K, M, output type, kernel the sizes plan onto).  First a mid-sized call (fills 160 token columns of the array
    # with the transposed copy), then a decode-sized one that reuses the same bytes with a different row pitch, then the
    # first again.  Then sizes beyond 256 tokens, where the array carries the operand images of X, their ready flags, the
    # inverted permutation and the per-tile counters of the tiling pass: the second such call finds the first one's flags
    # and counters still in the array, a smaller call in between overwrites part of them.
    cases = [(384, 1024, 150, torch.float16, b.ESP_KERNEL_STREAM), (384, 1024, 5, torch.float32, b.ESP_KERNEL_STREAM),
             (384, 1024, 150, torch.float16, b.ESP_KERNEL_STREAM),
             (640, 1024, 300, torch.float16, b.ESP_KERNEL_PAIR_TILED), (640, 1024, 300, torch.float16, b.ESP_KERNEL_PAIR_TILED),
             (640, 1024, 40, torch.float16, b.ESP_KERNEL_STREAM), (640, 1024, 300, torch.float32, b.ESP_KERNEL_PAIR_TILED),
             (640, 1024, 520, torch.float16, b.ESP_KERNEL_PAIR_TILED)]
    weights = {}
    for N, K, M, dtype, kernel in cases:
        if (N, K) not in weights:
            vals, meta, theta = pruned(41 + N, N, K)
            weights[(N, K)] = (vals, meta, theta, pack_on_gpu(vals, meta), torch.from_numpy(theta).to(dev))
        vals, meta, theta, packed, th = weights[(N, K)]
        X = g.standard_normal((M, K)).astype(np.float16)
        Xd = torch.from_numpy(X).to(dev)
        o = b.esp_gemm_opts_default()
        o.out_dtype = b.ESP_OUT_F32 if dtype == torch.float32 else b.ESP_OUT_F16
        assert b.esp_spgemm_plan(M, N, K, o, True)["kernel"] == kernel
        ws = torch.empty(b.esp_spgemm_workspace_bytes(M, N, K, o), dtype=torch.uint8, device=dev)
        assert ws.numel() <= b.ESP_STATIC_SCRATCH_BYTES         # the built-in array offers at least what this call's plan uses
        Y_ws = torch.full((M, N), float("nan"), dtype=dtype, device=dev)
        Y_st = torch.full((M, N), float("nan"), dtype=dtype, device=dev)
        b.esp_spgemm(Xd, packed, th, Y_ws, o, ws)
        torch.cuda.synchronize()
        # nothing may be allocated by the call: neither through torch's pool nor behind its back (the driver's own count of
        # free bytes on the device sees a cudaMalloc from inside the library, torch's counter would not)
        pool_before = torch.cuda.memory_allocated(dev)
        free_before, _ = torch.cuda.mem_get_info(dev)
        b.esp_spgemm_static(Xd, packed, th, Y_st)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info(dev)
        assert torch.cuda.memory_allocated(dev) == pool_before
        assert free_after == free_before
        assert b.esp_last_device_status() == b.ESP_OK
        # same kernels, same order of accumulation: the two entry points agree to the bit ...
        assert torch.equal(Y_ws, Y_st)
        # ... and with the oracle within the GEMM tolerances used everywhere else
        check(Y_st.cpu().numpy(), ref_product(X, vals, meta, theta), dtype == torch.float32)


def test_python_wrapper_reports_the_status_code():
    """The wrapper raises the library's error type carrying the status (checked on the host: nothing is launched)."""
    class FakeTensor:
        def __init__(self, shape, stride0):
            self.shape, self._stride0 = shape, stride0

        def stride(self, i):
            return self._stride0

        def data_ptr(self):
            return A
    K = 4096
    M = b.ESP_STATIC_SCRATCH_BYTES // (K * 2) + 1
    import torch
    Y = FakeTensor((M, 512), 512)
    Y.dtype = torch.float16
    with pytest.raises(b.EsparseError) as e:
        b.esp_spgemm_static(FakeTensor((M, K), K), FakeTensor((1,), 1), None, Y, stream=0)
    assert e.value.status == b.ESP_ERR_STATIC_LIMIT
