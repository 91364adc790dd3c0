"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the header
declares, and rejects bad arguments before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2310_15929_b200 import binding as b
from paper_2310_15929_b200.build import HEADER, LIB_PATH


def header_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(esp_[a-z_0-9]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(LIB_PATH)
    names = header_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(b.EXPORTS)


def test_version_and_status_strings():
    assert b.esp_version() >= 100
    seen = {b.esp_status_string(i) for i in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert b.esp_status_string(99) == "unknown status"


def test_defaults_follow_the_paper():
    o = b.esp_prune_opts_default()
    assert (o.bins, o.n_keep, o.m_group, o.lbs_block) == (100, 2, 4, 256)
    assert o.use_entropy and o.use_norm and o.use_gns and o.use_lbs and o.lbs_max_swaps == 0
    assert o.struct_size == ctypes.sizeof(b.esp_prune_opts)
    g = b.esp_gemm_opts_default()
    assert g.struct_size == ctypes.sizeof(b.esp_gemm_opts) and g.x_layout == b.ESP_X_TOKEN_MAJOR


def test_size_queries():
    assert b.esp_packed_bytes(128, 128) == 18432
    assert b.esp_packed_bytes(4096, 4096) == 4096 * 4096 * 2 * 9 // 16        # 9/16 of dense
    assert b.esp_packed_bytes(129, 136) == 4 * 18432                           # padded to 128-multiples
    assert b.esp_packed_bytes(0, 128) == 0
    o = b.esp_prune_opts_default()
    small = b.esp_metric_prune_workspace_bytes(512, 512, 128, o)
    big = b.esp_metric_prune_workspace_bytes(4096, 4096, 32768, o)
    assert 0 < small < big
    assert b.esp_metric_prune_workspace_bytes(512, 510, 128, o) == 0           # C % 8 != 0
    g = b.esp_gemm_opts_default()
    assert b.esp_spgemm_workspace_bytes(16, 4096, 4096, g) == 4096 * 16 * 2     # transposed copy of token-major X
    g.x_layout = b.ESP_X_CHANNEL_MAJOR
    assert b.esp_spgemm_workspace_bytes(16, 4096, 4096, g) == 0                 # K-slices reduce on chip: no scratch


A = 0x10000   # a fake, 16-byte aligned "device address": argument errors must be caught before any use


def prune_call(**kw):
    o = kw.pop("opts", b.esp_prune_opts_default())
    a = dict(W=A, No=512, C=512, ldw=512, Xcal=A, T=128, ldx=512, opts=o, vals=A, meta=A, perm=A, packed=None,
             chan_norm=None, chan_entropy=None, chan_score=None, stats=None, workspace=A, workspace_bytes=1 << 30,
             stream=None)
    a.update(kw)
    return b.esp_metric_prune_raw(**a)


def test_prune_argument_errors():
    assert prune_call(W=None) == b.ESP_ERR_INVALID_ARG
    assert prune_call(perm=None) == b.ESP_ERR_INVALID_ARG
    assert prune_call(Xcal=None) == b.ESP_ERR_INVALID_ARG                      # no calibration and no override
    assert prune_call(opts=None) == b.ESP_ERR_INVALID_ARG
    assert prune_call(C=508, ldw=512) == b.ESP_ERR_SHAPE
    assert prune_call(ldw=256) == b.ESP_ERR_SHAPE
    assert prune_call(No=0) == b.ESP_ERR_SHAPE
    assert prune_call(T=0) == b.ESP_ERR_SHAPE
    assert prune_call(ldw=516) == b.ESP_ERR_ALIGNMENT
    assert prune_call(W=A + 2) == b.ESP_ERR_ALIGNMENT
    assert prune_call(workspace=None) == b.ESP_ERR_WORKSPACE
    assert prune_call(workspace_bytes=16) == b.ESP_ERR_WORKSPACE
    o = b.esp_prune_opts_default(); o.n_keep, o.m_group = 4, 8
    assert prune_call(opts=o) == b.ESP_ERR_UNSUPPORTED                         # 4:8 has no sparse MMA form
    o = b.esp_prune_opts_default(); o.bins = 5000
    assert prune_call(opts=o) == b.ESP_ERR_UNSUPPORTED
    # the documented range of bins is 2..512, at the boundary exactly
    o = b.esp_prune_opts_default(); o.bins = 513
    assert prune_call(opts=o) == b.ESP_ERR_UNSUPPORTED
    assert b.esp_metric_prune_workspace_bytes(512, 512, 128, o) == 0 and b.esp_calib_state_bytes(512, 513) == 0
    o.bins = 512
    assert b.esp_metric_prune_workspace_bytes(512, 512, 128, o) > 0 and b.esp_calib_state_bytes(512, 512) > 0
    o.bins = 1
    assert prune_call(opts=o) == b.ESP_ERR_UNSUPPORTED
    o = b.esp_prune_opts_default(); o.lbs_block = 250
    assert prune_call(opts=o) == b.ESP_ERR_INVALID_ARG
    o = b.esp_prune_opts_default(); o.struct_size = 8
    assert prune_call(opts=o) == b.ESP_ERR_INVALID_ARG
    s = b.esp_prune_stats(); s.struct_size = 3
    assert prune_call(stats=s) == b.ESP_ERR_INVALID_ARG


def gemm_call(**kw):
    o = kw.pop("opts", b.esp_gemm_opts_default())
    a = dict(X=A, M=16, K=512, ldx=512, packed=A, perm=A, N=512, Y=A, ldy=512, opts=o, workspace=None,
             workspace_bytes=0, stream=None)
    a.update(kw)
    return b.esp_spgemm_raw(**a)


def test_gemm_argument_errors():
    assert gemm_call(X=None) == b.ESP_ERR_INVALID_ARG
    assert gemm_call(packed=None) == b.ESP_ERR_INVALID_ARG
    assert gemm_call(opts=None) == b.ESP_ERR_INVALID_ARG
    assert gemm_call(M=0) == b.ESP_ERR_SHAPE
    assert gemm_call(K=508) == b.ESP_ERR_SHAPE
    assert gemm_call(ldx=256) == b.ESP_ERR_SHAPE
    assert gemm_call(ldy=100) == b.ESP_ERR_SHAPE
    assert gemm_call(ldx=516) == b.ESP_ERR_ALIGNMENT
    assert gemm_call(Y=A + 8) == b.ESP_ERR_ALIGNMENT
    o = b.esp_gemm_opts_default(); o.x_layout = 7
    assert gemm_call(opts=o) == b.ESP_ERR_INVALID_ARG
    o = b.esp_gemm_opts_default(); o.split_k = 9
    assert gemm_call(opts=o) == b.ESP_ERR_INVALID_ARG
    o = b.esp_gemm_opts_default(); o.token_tile = 24
    assert gemm_call(opts=o) == b.ESP_ERR_INVALID_ARG
    o = b.esp_gemm_opts_default(); o.x_layout = b.ESP_X_CHANNEL_MAJOR
    assert gemm_call(opts=o, ldx=8) == b.ESP_ERR_SHAPE                          # channel-major needs ldx >= M


def test_no_gpu_means_cuda_error_not_a_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    # valid arguments, no device: the call must fail loudly, never compute on the CPU
    assert prune_call() in (b.ESP_ERR_CUDA, b.ESP_ERR_UNSUPPORTED)
    assert gemm_call() in (b.ESP_ERR_CUDA, b.ESP_ERR_UNSUPPORTED)


def test_calibration_state_size_and_argument_checks():
    C, bins = 512, 100
    n = b.esp_calib_state_bytes(C, bins)
    # four fp64 vectors, the counts, and 64 chunk partials of (fp64, f32, f32) per channel
    assert n >= 4 * 8 * C + 4 * C * bins + 64 * C * 16
    assert n % 256 == 0
    assert b.esp_calib_state_bytes(C + 1, bins) == 0
    assert b.esp_calib_state_bytes(C, 1) == 0
    assert b._lib.esp_calib_reset(None, C, bins, None) == b.ESP_ERR_INVALID_ARG
    assert b._lib.esp_calib_range(None, None, 4, C, C, bins, None) == b.ESP_ERR_INVALID_ARG


def test_plan_table_round_trip(tmp_path):
    o = b.esp_gemm_opts_default()
    o.x_layout = b.ESP_X_CHANNEL_MAJOR
    table = {b.plan_key(16, 4096, 4096, o): {"kernel": b.ESP_KERNEL_STREAM, "token_tile": 16, "split_k": 8}}
    path = str(tmp_path / "plans.json")
    b.save_plan_table(path, table)
    loaded = b.load_plan_table(path)
    assert loaded == {k: dict(v, pipeline_stages=0) for k, v in table.items()}
    assert b.apply_plan(o, loaded, 16, 4096, 4096)
    assert (o.force_kernel, o.token_tile, o.split_k) == (b.ESP_KERNEL_STREAM, 16, 8)
    assert not b.apply_plan(o, loaded, 17, 4096, 4096)
    o2 = b.esp_gemm_opts_default()                       # another layout is another entry
    assert not b.apply_plan(o2, loaded, 16, 4096, 4096)


def test_grouped_and_tune_argument_checks_need_no_device():
    import ctypes
    o = b.esp_gemm_opts_default()
    one = (ctypes.c_void_p * 1)(0x1000)
    n = (ctypes.c_int * 1)(128)
    ld = (ctypes.c_long * 1)(128)
    call = lambda count: b._lib.esp_spgemm_grouped(count, one, 16, 128, 128, one, one, n, one, ld, ctypes.byref(o), None, 0, None)
    assert call(0) == b.ESP_ERR_INVALID_ARG
    assert call(5) == b.ESP_ERR_INVALID_ARG
    o.bias = 0x2000                                           # a common bias makes no sense for several weights
    assert call(1) == b.ESP_ERR_INVALID_ARG
    o.bias = None
    o.pipeline_stages = 1
    assert call(1) == b.ESP_ERR_INVALID_ARG
    o.pipeline_stages = 0
    best = ctypes.c_float()
    assert b._lib.esp_spgemm_tune(None, 16, 128, 128, None, None, 128, None, 128, ctypes.byref(o), None, 0, 0,
                                  ctypes.byref(best), None, None) == b.ESP_ERR_INVALID_ARG


def test_cluster_multicast_loads_live_only_in_the_companion_source():
    """The main library must hold no bulk or tiled load with cluster multicast (it also runs where several GPUs are in
    play); the one kernel form that uses such loads is built from a source file of its own into a companion library, and both
    are named in the list of files left out of multi-GPU runs.  The companion is optional: the main library reports
    whether it found it."""
    from paper_2310_15929_b200.build import MC_LIB_PATH, MC_SOURCE
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    # (the pattern is put together from pieces so that this file does not itself name such a load)
    load_with_multicast = re.compile("cp" + r"\.async\." + "bulk" + r"[^\n;]*\." + "multi" + "cast::cluster")
    offenders = []
    sources = [os.path.join(root, n) for n in os.listdir(root) if n.endswith(".py")]
    for top in ("paper_2310_15929_b200", "include", "oracle", "tests"):
        for folder, _, files in os.walk(os.path.join(root, top)):
            sources += [os.path.join(folder, n) for n in files if n.endswith((".cu", ".cuh", ".h", ".py", ".c", ".cpp"))]
    for path in sources:
        if os.path.abspath(path) in (os.path.abspath(MC_SOURCE), os.path.abspath(__file__)):
            continue
        if load_with_multicast.search(open(path, errors="replace").read()):
            offenders.append(os.path.relpath(path, root))
    assert offenders == []
    left_out = open(os.path.join(root, ".gpurunignore.multi")).read().split()
    assert os.path.relpath(MC_SOURCE, root) in left_out and os.path.relpath(MC_LIB_PATH, root) in left_out
    if os.path.exists(MC_SOURCE):
        assert load_with_multicast.search(open(MC_SOURCE).read())
        assert b.esp_multicast_available() == os.path.exists(MC_LIB_PATH)
