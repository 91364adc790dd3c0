"""Helpers of the GPU parity tests: run the C-ABI calls on torch device buffers."""
import ctypes

import numpy as np
import torch

from paper_2310_15929_b200 import binding as b

DEV = "cuda:0"


class GpuPrune:
    def __init__(self, W, Xcal, alpha, score=None, stats=True, pack=True, perm=None, **opts):
        No, C = W.shape
        self.No, self.C = No, C
        dev = torch.device(DEV)
        o = b.esp_prune_opts_default()
        o.alpha = alpha
        for k, v in opts.items():
            setattr(o, k, v)
        self.Wd = torch.from_numpy(np.ascontiguousarray(W)).to(dev)
        self.Xd = None if Xcal is None else torch.from_numpy(np.ascontiguousarray(Xcal)).to(dev)
        T = 0 if Xcal is None else Xcal.shape[0]
        self.score_d = None
        if score is not None:
            self.score_d = torch.from_numpy(np.ascontiguousarray(score, dtype=np.float64)).to(dev)
            o.score_override = self.score_d.data_ptr()
        self.perm_in = None
        if perm is not None:
            self.perm_in = torch.from_numpy(np.ascontiguousarray(perm, dtype=np.int32)).to(dev)
            o.perm_override = self.perm_in.data_ptr()
        self.ws = torch.empty(max(16, b.esp_metric_prune_workspace_bytes(No, C, T, o)), dtype=torch.uint8, device=dev)
        self.vals = torch.empty(No, C // 2, dtype=torch.float16, device=dev)
        self.meta = torch.empty(No, C // 8, dtype=torch.uint8, device=dev)
        self.perm = torch.empty(C, dtype=torch.int32, device=dev)
        self.packed = torch.empty(b.esp_packed_bytes(No, C), dtype=torch.uint8, device=dev) if pack else None
        self.norm = torch.empty(C, dtype=torch.float64, device=dev)
        self.entropy = torch.empty(C, dtype=torch.float64, device=dev)
        self.score = torch.empty(C, dtype=torch.float64, device=dev)
        self.stats = b.esp_prune_stats() if stats else None
        has_x = self.Xd is not None
        b.esp_metric_prune(self.Wd, self.Xd, o, self.vals, self.meta, self.perm, self.packed,
                           self.norm if has_x else None, self.entropy if has_x else None, self.score,
                           self.stats, self.ws)
        torch.cuda.synchronize()
        assert b.esp_last_device_status() == b.ESP_OK

    def host(self):
        return (self.vals.cpu().numpy(), self.meta.cpu().numpy(), self.perm.cpu().numpy())


def pack_on_gpu(vals, meta):
    No, half = vals.shape
    C = half * 2
    dev = torch.device(DEV)
    packed = torch.empty(b.esp_packed_bytes(No, C), dtype=torch.uint8, device=dev)
    b.esp_pack(torch.from_numpy(np.ascontiguousarray(vals)).to(dev),
               torch.from_numpy(np.ascontiguousarray(meta)).to(dev), No, C, packed)
    return packed


def spgemm(X, packed, theta, N, *, channel_major=False, out_f32=False, split_k=0, token_tile=0, kernel=0,
           workspace=True, static_weights=0, bias=None, relu=False, pipeline_stages=0):
    dev = torch.device(DEV)
    M = X.shape[0]
    Xd = torch.from_numpy(np.ascontiguousarray(X)).to(dev)
    if channel_major:
        Xd = Xd.t().contiguous()
        if M % 8:                                   # leading dimension must be a multiple of 8 elements
            pad = torch.zeros(Xd.shape[0], (M + 7) // 8 * 8, dtype=Xd.dtype, device=dev)
            pad[:, :M] = Xd
            Xd = pad[:, :M]
    o = b.esp_gemm_opts_default()
    o.x_layout = b.ESP_X_CHANNEL_MAJOR if channel_major else b.ESP_X_TOKEN_MAJOR
    o.out_dtype = b.ESP_OUT_F32 if out_f32 else b.ESP_OUT_F16
    o.split_k, o.token_tile, o.force_kernel = split_k, token_tile, kernel
    o.static_weights = static_weights
    o.pipeline_stages = pipeline_stages
    bias_d = None
    if bias is not None:
        bias_d = torch.from_numpy(np.ascontiguousarray(bias, dtype=np.float16)).to(dev)
        o.bias = bias_d.data_ptr()
    o.activation = b.ESP_ACT_RELU if relu else b.ESP_ACT_NONE
    Y = torch.full((M, N), float("nan"), dtype=torch.float32 if out_f32 else torch.float16, device=dev)
    th = None if theta is None else torch.from_numpy(np.ascontiguousarray(theta, dtype=np.int32)).to(dev)
    ws = None
    if workspace:
        K = X.shape[1]
        nbytes = b.esp_spgemm_workspace_bytes(M, N, K, o)
        if nbytes:
            ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    b.esp_spgemm(Xd, packed, th, Y, o, ws)
    torch.cuda.synchronize()
    assert b.esp_last_device_status() == b.ESP_OK
    return Y.cpu().numpy()


def calibrate_in_chunks(chunks, alpha, bins=100, **opts):
    """Streaming calibration over a list of [T_i, C] fp16 arrays; returns (norm, entropy, score, counts) on the host."""
    dev = torch.device(DEV)
    C = chunks[0].shape[1]
    o = b.esp_prune_opts_default()
    o.alpha, o.bins = alpha, bins
    for k, v in opts.items():
        setattr(o, k, v)
    nbytes = b.esp_calib_state_bytes(C, bins)
    state = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    state.fill_(0xA5)                                # reset must not depend on what the buffer held
    dchunks = [torch.from_numpy(np.ascontiguousarray(c)).to(dev) for c in chunks]
    b.esp_calib_reset(state, C, bins)
    for d in dchunks:
        b.esp_calib_range(state, d, bins)
    for d in dchunks:
        b.esp_calib_histogram(state, d, bins)
    norm = torch.empty(C, dtype=torch.float64, device=dev)
    entropy = torch.empty(C, dtype=torch.float64, device=dev)
    score = torch.empty(C, dtype=torch.float64, device=dev)
    T_total = sum(c.shape[0] for c in chunks)
    b.esp_calib_finish(state, C, T_total, o, norm, entropy, score)
    torch.cuda.synchronize()
    assert b.esp_last_device_status() == b.ESP_OK
    off = 4 * ((8 * C + 255) // 256 * 256)
    counts = state[off: off + 4 * C * bins].view(torch.int32).reshape(C, bins).cpu().numpy()
    return norm.cpu().numpy(), entropy.cpu().numpy(), score.cpu().numpy(), counts, score
