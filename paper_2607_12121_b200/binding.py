"""Thin ctypes binding of ``libflashdiff.so``: argument marshalling only.

Every function mirrors one C entry point of ``include/flashdiff.h`` and takes torch CUDA
tensors (device memory and streams are all PyTorch is used for).  No step of the method runs
in Python.  Importing this module fails loudly if the shared library has not been built.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libflashdiff.so")

FD_OK = 0
FD_ERR_INVALID_ARG, FD_ERR_SHAPE, FD_ERR_STATE, FD_ERR_WORKSPACE = 1, 2, 3, 4
FD_ERR_UNSUPPORTED, FD_ERR_CUDA, FD_ERR_TIMEOUT = 5, 6, 7
FD_F32, FD_BF16 = 0, 1
FD_ENGINE_AUTO, FD_ENGINE_SIMT, FD_ENGINE_TC = 0, 1, 2

EXPORTS = ["fd_workspace_bytes", "fd_create", "fd_partition_regions", "fd_region_activity",
           "fd_regional_step", "fd_poll_status", "fd_launch_count", "fd_destroy", "fd_last_error",
           "fd_profile_enable", "fd_profile_read", "fd_region_activity_noalloc", "fd_selftest_bounded_wait",
           "fd_embed_latent", "fd_update_latent", "fd_regional_step_mass", "fd_region_activity_attn",
           "fd_sched_pack", "fd_sched_form_batch", "fd_rsearch_init", "fd_rsearch_update", "fd_set_block_variants",
           "fd_set_text_stream", "fd_set_cross_attention", "fd_set_fp8_operands", "fd_debug_buffer", "fd_set_fp8_text_stream"]
FD_NOALLOC_MAX_REGION_SLOTS = 16384
PROF_GROUPS = ["activity", "compact", "adaln", "ln_modulate", "gemm_qkv", "attention", "gemm_out", "gemm_fc1",
               "gemm_fc2", "partition", "sampler", "qk_variants", "cross_attention"]


class FdConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_blocks", "hidden", "n_heads", "head_dim", "mlp_dim", "cond_dim", "max_batch",
                 "max_tokens", "max_regions", "dtype", "engine")] + \
               [("ln_eps", ctypes.c_float), ("gate_eta", ctypes.c_float), ("max_skip_k", ctypes.c_int32)]


class FdWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2", "w_ada", "b_ada")]


class FdSamplerWeights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("w_in", "b_in", "pos", "w_out", "b_out")] + [("latent_dim", ctypes.c_int32)]


class FdBlockVariants(ctypes.Structure):
    _fields_ = [("q_norm_w", ctypes.c_void_p), ("k_norm_w", ctypes.c_void_p), ("qk_norm_eps", ctypes.c_float),
                ("rope_cos", ctypes.c_void_p), ("rope_sin", ctypes.c_void_p), ("q_norm_w_text", ctypes.c_void_p),
                ("k_norm_w_text", ctypes.c_void_p)]


class FdCrossAttention(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("w_q", "b_q", "w_o", "b_o", "ctx_kv")] + \
               [("n_ctx", ctypes.c_int32), ("ctx_batch", ctypes.c_int32)]


class FdFp8Operands(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("w8_qkv", "s_qkv", "w8_fc1", "s_fc1", "w8_fc2", "s_fc2", "a_scale")]


class FdRSearch(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("r_min", "r_max", "accepted", "candidate", "step", "dir", "have_ref",
                                              "fails_at_one", "converged")] + [("ref_perf", ctypes.c_double)]


class FlashDiffError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__("libflashdiff status %d: %s" % (status, text))
        self.status = status


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError("libflashdiff.so is missing: run `python -m paper_2607_12121_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.fd_workspace_bytes.restype = sz
    lib.fd_workspace_bytes.argtypes = [ctypes.POINTER(FdConfig)]
    lib.fd_create.restype = i32
    lib.fd_create.argtypes = [ctypes.POINTER(FdConfig), ctypes.POINTER(FdWeights), vp, sz, ctypes.POINTER(vp)]
    lib.fd_partition_regions.restype = i32
    lib.fd_partition_regions.argtypes = [vp, vp, i32, i32, i32, vp, i32, i32, i32, i32, vp, vp, vp]
    lib.fd_region_activity.restype = i32
    lib.fd_region_activity.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.fd_region_activity_noalloc.restype = i32
    lib.fd_region_activity_noalloc.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp, ctypes.c_float, i32, vp, vp, vp,
                                               vp, vp, vp, vp, vp]
    lib.fd_regional_step.restype = i32
    lib.fd_regional_step.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.fd_poll_status.restype = i32
    lib.fd_poll_status.argtypes = [vp, vp]
    lib.fd_profile_enable.restype = i32
    lib.fd_profile_enable.argtypes = [vp, i32]
    lib.fd_profile_read.restype = i32
    lib.fd_profile_read.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)]
    lib.fd_selftest_bounded_wait.restype = i32
    lib.fd_selftest_bounded_wait.argtypes = [vp, vp]
    lib.fd_regional_step_mass.restype = i32
    lib.fd_regional_step_mass.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.fd_region_activity_attn.restype = i32
    lib.fd_region_activity_attn.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.fd_sched_pack.restype = i32
    lib.fd_sched_pack.argtypes = [i32, vp, i32, vp, vp, vp]
    lib.fd_sched_form_batch.restype = i32
    lib.fd_sched_form_batch.argtypes = [i32, vp, vp, vp, vp, ctypes.c_int64, i32, vp]
    lib.fd_rsearch_init.restype = i32
    lib.fd_rsearch_init.argtypes = [ctypes.POINTER(FdRSearch), i32, i32, i32]
    lib.fd_rsearch_update.restype = i32
    lib.fd_rsearch_update.argtypes = [ctypes.POINTER(FdRSearch), ctypes.c_double, ctypes.POINTER(ctypes.c_int32)]
    lib.fd_embed_latent.restype = i32
    lib.fd_embed_latent.argtypes = [vp, ctypes.POINTER(FdSamplerWeights), vp, i32, i32, vp, vp]
    lib.fd_update_latent.restype = i32
    lib.fd_update_latent.argtypes = [vp, ctypes.POINTER(FdSamplerWeights), vp, vp, vp, vp, vp, i32, i32, vp, vp, vp]
    lib.fd_set_block_variants.restype = i32
    lib.fd_set_block_variants.argtypes = [vp, ctypes.POINTER(FdBlockVariants)]
    lib.fd_set_text_stream.restype = i32
    lib.fd_set_text_stream.argtypes = [vp, ctypes.POINTER(FdWeights)]
    lib.fd_debug_buffer.restype = i32
    lib.fd_debug_buffer.argtypes = [vp, ctypes.c_int, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_size_t)]
    lib.fd_set_fp8_operands.restype = i32
    lib.fd_set_fp8_operands.argtypes = [vp, ctypes.POINTER(FdFp8Operands)]
    lib.fd_set_fp8_text_stream.restype = i32
    lib.fd_set_fp8_text_stream.argtypes = [vp, ctypes.POINTER(FdFp8Operands)]
    lib.fd_set_cross_attention.restype = i32
    lib.fd_set_cross_attention.argtypes = [vp, ctypes.POINTER(FdCrossAttention)]
    lib.fd_launch_count.restype = ctypes.c_int64
    lib.fd_launch_count.argtypes = [vp]
    lib.fd_destroy.restype = i32
    lib.fd_destroy.argtypes = [vp]
    lib.fd_last_error.restype = ctypes.c_char_p
    lib.fd_last_error.argtypes = [vp]
    return lib


lib = _load()


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


def _check(ctx_handle, status: int):
    if status != FD_OK:
        text = lib.fd_last_error(ctx_handle)
        raise FlashDiffError(status, text.decode() if text else "")


def fd_workspace_bytes(cfg: FdConfig) -> int:
    return int(lib.fd_workspace_bytes(ctypes.byref(cfg)))


class Context:
    """Owns the fd_ctx handle plus the torch tensors the library borrows (weights, workspace)."""

    def __init__(self, cfg: FdConfig, weights: Dict[str, "object"], device="cuda"):
        import torch
        self.cfg = cfg
        self.dtype = torch.bfloat16 if cfg.dtype == FD_BF16 else torch.float32
        self.weights = weights
        for k, v in weights.items():
            assert v.is_cuda and v.is_contiguous() and v.dtype == self.dtype, k
        nbytes = fd_workspace_bytes(cfg)
        if nbytes == 0:
            raise FlashDiffError(FD_ERR_SHAPE, "fd_workspace_bytes rejected the configuration")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
        w = FdWeights(**{k: weights[k].data_ptr() for k, _ in FdWeights._fields_})
        handle = ctypes.c_void_p()
        with torch.cuda.device(self.workspace.device):
            st = lib.fd_create(ctypes.byref(cfg), ctypes.byref(w), self.workspace.data_ptr(), nbytes,
                               ctypes.byref(handle))
        _check(None, st)
        self.handle = handle

    def close(self) -> int:
        st = FD_OK
        if getattr(self, "handle", None):
            st = int(lib.fd_destroy(self.handle))
            self.handle = None
        return st

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def launches(self) -> int:
        return int(lib.fd_launch_count(self.handle))


def fd_create(cfg: FdConfig, weights: Dict[str, "object"], device="cuda") -> Context:
    return Context(cfg, weights, device)


def fd_destroy(ctx: Context) -> int:
    """Releases the context; returns FD_OK or a device-side status that was never polled."""
    return ctx.close()


def fd_partition_regions(ctx: Context, attn_map, R: int, labels_out, region_sizes_out=None, salient_cols=None,
                         min_region_tokens: int = 1, max_region_tokens: int = 0, stream=None) -> None:
    B, N, T = attn_map.shape
    T_s = 0 if salient_cols is None else int(salient_cols.numel())
    _check(ctx.handle, lib.fd_partition_regions(
        ctx.handle, _ptr(attn_map), B, N, T, _ptr(salient_cols), T_s, R, min_region_tokens, max_region_tokens,
        _ptr(labels_out), _ptr(region_sizes_out), _stream(stream)))


def fd_region_activity(ctx: Context, z_cur, z_prev, labels, R: int, eps, delta_state, skip_count, prev_active,
                       score_out, weight_out, mask_out, stream=None) -> None:
    B, N, D = z_cur.shape
    _check(ctx.handle, lib.fd_region_activity(
        ctx.handle, _ptr(z_cur), _ptr(z_prev), _ptr(labels), B, N, D, R, _ptr(eps), _ptr(delta_state),
        _ptr(skip_count), _ptr(prev_active), _ptr(score_out), _ptr(weight_out), _ptr(mask_out), _stream(stream)))


def fd_region_activity_noalloc(z_cur, z_prev, labels, R: int, eps, eta: float, max_skip_k: int, delta_state,
                               skip_count, prev_active, score_out, weight_out, mask_out, status_out=None,
                               stream=None) -> None:
    """The gate for callers that may not allocate device memory: no context, no workspace; the
    scratch is a fixed array inside the library (B * R <= FD_NOALLOC_MAX_REGION_SLOTS).  Calls on
    one device share that array, so they must not overlap on the GPU."""
    B, N, D = z_cur.shape
    _check(None, lib.fd_region_activity_noalloc(
        _ptr(z_cur), _ptr(z_prev), _ptr(labels), B, N, D, R, _ptr(eps), float(eta), int(max_skip_k),
        _ptr(delta_state), _ptr(skip_count), _ptr(prev_active), _ptr(score_out), _ptr(weight_out), _ptr(mask_out),
        _ptr(status_out), _stream(stream)))


def fd_regional_step(ctx: Context, x, cond, labels, mask, R: int, kv_cache, y, active_idx_out, cu_active_out,
                     stream=None) -> None:
    B, N, _ = x.shape
    _check(ctx.handle, lib.fd_regional_step(
        ctx.handle, _ptr(x), _ptr(cond), _ptr(labels), _ptr(mask), B, N, R, _ptr(kv_cache), _ptr(y),
        _ptr(active_idx_out), _ptr(cu_active_out), _stream(stream)))


def make_sampler_weights(tensors: dict, latent_dim: int) -> FdSamplerWeights:
    """fd_sampler_weights from device tensors w_in [H,D], b_in [H], pos [N,H], w_out [D,H], b_out [D]
    (keep the tensors alive while the struct is in use)."""
    return FdSamplerWeights(*[_ptr(tensors[k]) for k in ("w_in", "b_in", "pos", "w_out", "b_out")], int(latent_dim))


def fd_embed_latent(ctx: Context, sw: FdSamplerWeights, z, x_out, stream=None) -> None:
    """x_out[b,j,:] = z[b,j,:] w_in^T + b_in + pos[j,:]  (z [B,N,D] f32)."""
    B, N, _ = z.shape
    _check(ctx.handle, lib.fd_embed_latent(ctx.handle, ctypes.byref(sw), _ptr(z), B, N, _ptr(x_out), _stream(stream)))


def fd_update_latent(ctx: Context, sw: FdSamplerWeights, z, y, active_idx, cu_active, h, drift_cache, z_next,
                     stream=None) -> None:
    """Final layer on the active tokens' rows of y (refreshing drift_cache there), then
    z_next = z + h[b] * drift_cache for every token."""
    B, N, _ = z.shape
    _check(ctx.handle, lib.fd_update_latent(ctx.handle, ctypes.byref(sw), _ptr(z), _ptr(y), _ptr(active_idx),
                                            _ptr(cu_active), _ptr(h), B, N, _ptr(drift_cache), _ptr(z_next),
                                            _stream(stream)))


def fd_regional_step_mass(ctx: Context, x, cond, labels, mask, R: int, kv_cache, y, active_idx_out, cu_active_out,
                          region_mass_out, stream=None) -> None:
    """fd_regional_step that also writes region_mass_out [B,R] f64: the first block's own-region attention mass."""
    B, N, _ = x.shape
    _check(ctx.handle, lib.fd_regional_step_mass(
        ctx.handle, _ptr(x), _ptr(cond), _ptr(labels), _ptr(mask), B, N, R, _ptr(kv_cache), _ptr(y),
        _ptr(active_idx_out), _ptr(cu_active_out), _ptr(region_mass_out), _stream(stream)))


def fd_region_activity_attn(ctx: Context, region_mass, region_sizes, eps, rbar_state, delta_state, skip_count,
                            prev_active, importance_out, weight_out, mask_out, stream=None) -> None:
    """The gate on the attention-mass signal: Delta_i = |R_i - Rbar_i| with R_i = mass_i / size_i^2."""
    B, R = region_mass.shape
    _check(ctx.handle, lib.fd_region_activity_attn(
        ctx.handle, _ptr(region_mass), _ptr(region_sizes), B, R, _ptr(eps), _ptr(rbar_state), _ptr(delta_state),
        _ptr(skip_count), _ptr(prev_active), _ptr(importance_out), _ptr(weight_out), _ptr(mask_out), _stream(stream)))


def fd_set_block_variants(ctx: Context, q_norm_w=None, k_norm_w=None, qk_norm_eps: float = 1e-6, rope_cos=None,
                          rope_sin=None, q_norm_w_text=None, k_norm_w_text=None) -> None:
    """Switches the block variants on (device tensors: QK-RMSNorm weights [L, head_dim] of the context's dtype, rotary
    tables [max_tokens, head_dim/2] f32; *_text: the second stream's norm weights) or, with no tensors, off.  The
    context keeps the tensors alive."""
    ctx.variant_tensors = (q_norm_w, k_norm_w, rope_cos, rope_sin, q_norm_w_text, k_norm_w_text)
    if all(t is None for t in ctx.variant_tensors):
        _check(ctx.handle, lib.fd_set_block_variants(ctx.handle, None))
        return
    v = FdBlockVariants(_ptr(q_norm_w), _ptr(k_norm_w), float(qk_norm_eps), _ptr(rope_cos), _ptr(rope_sin),
                        _ptr(q_norm_w_text), _ptr(k_norm_w_text))
    _check(ctx.handle, lib.fd_set_block_variants(ctx.handle, ctypes.byref(v)))


def fd_set_text_stream(ctx: Context, text_weights: Optional[Dict[str, "object"]]) -> None:
    """Dual-stream blocks: the tokens with label R use ``text_weights`` (same keys and layout as the context's own
    weights; device tensors the context keeps alive); None returns to a single stream."""
    ctx.text_weights = text_weights
    if text_weights is None:
        _check(ctx.handle, lib.fd_set_text_stream(ctx.handle, None))
        return
    for k, t in text_weights.items():
        assert t.is_cuda and t.is_contiguous() and t.dtype == ctx.dtype, k
    w = FdWeights(**{k: text_weights[k].data_ptr() for k, _ in FdWeights._fields_})
    _check(ctx.handle, lib.fd_set_text_stream(ctx.handle, ctypes.byref(w)))


def fd_set_cross_attention(ctx: Context, cross: Optional[Dict[str, "object"]]) -> None:
    """Cross-attention to a fixed context in every block: ``cross`` holds device tensors of the context's dtype, w_q, w_o
    [L, H, H], b_q, b_o [L, H] and ctx_kv [L, B, 2, n_ctx, H] (the context keeps them alive); None switches it off."""
    ctx.cross = cross
    if cross is None:
        _check(ctx.handle, lib.fd_set_cross_attention(ctx.handle, None))
        return
    for k in ("w_q", "b_q", "w_o", "b_o", "ctx_kv"):
        t = cross[k]
        assert t.is_cuda and t.is_contiguous() and t.dtype == ctx.dtype, k
    kv = cross["ctx_kv"]
    assert kv.dim() == 5 and kv.shape[2] == 2
    x = FdCrossAttention(*(cross[k].data_ptr() for k in ("w_q", "b_q", "w_o", "b_o", "ctx_kv")), int(kv.shape[3]), int(kv.shape[1]))
    _check(ctx.handle, lib.fd_set_cross_attention(ctx.handle, ctypes.byref(x)))


FD_BUF_ACT, FD_BUF_HIDDEN, FD_BUF_RESID, FD_BUF_Q, FD_BUF_ATTN = 0, 1, 2, 3, 4


def fd_debug_buffer(ctx: Context, which: int):
    """(device address, size in bytes) of one of the step's intermediate buffers inside the context's workspace."""
    p, n = ctypes.c_void_p(), ctypes.c_size_t()
    _check(ctx.handle, lib.fd_debug_buffer(ctx.handle, int(which), ctypes.byref(p), ctypes.byref(n)))
    return int(p.value), int(n.value)


def fd_set_fp8_operands(ctx: Context, fp8: Optional[Dict[str, "object"]], text_stream: bool = False) -> None:
    """FP8 operands for QKV, fc1 and fc2: ``fp8`` holds device tensors w8_qkv, w8_fc1, w8_fc2 (uint8 E4M3 codes, [L, out,
    in]), s_qkv, s_fc1, s_fc2 (float32 [L, out]; the context keeps all six alive) and a_scale, a host float32 array
    [L, 3] of activation scales; None switches it off.  ``text_stream``: the second stream's set."""
    call = lib.fd_set_fp8_text_stream if text_stream else lib.fd_set_fp8_operands
    if text_stream:
        ctx.fp8_text = fp8
    else:
        ctx.fp8 = fp8
    if fp8 is None:
        _check(ctx.handle, call(ctx.handle, None))
        return
    import numpy as np
    for k in ("w8_qkv", "w8_fc1", "w8_fc2"):
        assert fp8[k].is_cuda and fp8[k].is_contiguous() and fp8[k].element_size() == 1, k
    for k in ("s_qkv", "s_fc1", "s_fc2"):
        assert fp8[k].is_cuda and fp8[k].is_contiguous() and str(fp8[k].dtype) == "torch.float32", k
    a = np.ascontiguousarray(fp8["a_scale"], dtype=np.float32)
    f = FdFp8Operands(*(fp8[k].data_ptr() for k in ("w8_qkv", "s_qkv", "w8_fc1", "s_fc1", "w8_fc2", "s_fc2")), a.ctypes.data)
    _check(ctx.handle, call(ctx.handle, ctypes.byref(f)))


def fd_sched_pack(load, cost, home):
    """Least-maximum-load packing (Sec. 4.3) of monotasks in the given order.  ``load`` [G] float64 numpy array is
    updated in place; returns the device of every monotask as an int32 array."""
    import numpy as np
    assert load.dtype == np.float64 and load.flags["C_CONTIGUOUS"]
    cost = np.ascontiguousarray(cost, np.float64)
    home = np.ascontiguousarray(home, np.int32)
    assign = np.empty(cost.size, np.int32)
    st = lib.fd_sched_pack(int(load.size), load.ctypes.data_as(ctypes.c_void_p), int(cost.size),
                           cost.ctypes.data_as(ctypes.c_void_p), home.ctypes.data_as(ctypes.c_void_p),
                           assign.ctypes.data_as(ctypes.c_void_p))
    if st != FD_OK:
        raise FlashDiffError(st, "fd_sched_pack: invalid argument")
    return assign


def fd_sched_form_batch(priority, arrival, active_tokens, resident, token_budget: int, max_resident: int):
    """Which requests run the next step (Sec. 4.3).  ``resident`` [n] uint8 numpy array is updated in place;
    returns the uint8 array of chosen requests."""
    import numpy as np
    assert resident.dtype == np.uint8 and resident.flags["C_CONTIGUOUS"]
    priority = np.ascontiguousarray(priority, np.int32)
    arrival = np.ascontiguousarray(arrival, np.int64)
    active_tokens = np.ascontiguousarray(active_tokens, np.int32)
    chosen = np.zeros(resident.size, np.uint8)
    st = lib.fd_sched_form_batch(int(resident.size), priority.ctypes.data_as(ctypes.c_void_p),
                                 arrival.ctypes.data_as(ctypes.c_void_p), active_tokens.ctypes.data_as(ctypes.c_void_p),
                                 resident.ctypes.data_as(ctypes.c_void_p), ctypes.c_int64(int(token_budget)),
                                 int(max_resident), chosen.ctypes.data_as(ctypes.c_void_p))
    if st != FD_OK:
        raise FlashDiffError(st, "fd_sched_form_batch: invalid argument")
    return chosen


def fd_rsearch_init(r_min: int, r_max: int, r_start: int) -> FdRSearch:
    """State of the adaptive patch-granularity search (Sec. 4.1); the first R to run is ``r_start``."""
    st = FdRSearch()
    rc = lib.fd_rsearch_init(ctypes.byref(st), int(r_min), int(r_max), int(r_start))
    if rc != FD_OK:
        raise FlashDiffError(rc, "fd_rsearch_init: invalid argument")
    return st


def fd_rsearch_update(st: FdRSearch, observed_perf: float) -> int:
    """Reports the performance observed with the R returned last; returns the R to run next."""
    nxt = ctypes.c_int32()
    rc = lib.fd_rsearch_update(ctypes.byref(st), float(observed_perf), ctypes.byref(nxt))
    if rc != FD_OK:
        raise FlashDiffError(rc, "fd_rsearch_update: invalid argument")
    return int(nxt.value)


def fd_poll_status(ctx: Context, stream=None) -> None:
    _check(ctx.handle, lib.fd_poll_status(ctx.handle, _stream(stream)))


def fd_selftest_bounded_wait(ctx: Context, stream=None) -> None:
    _check(ctx.handle, lib.fd_selftest_bounded_wait(ctx.handle, _stream(stream)))


def fd_profile_enable(ctx: Context, enable: bool) -> None:
    _check(ctx.handle, lib.fd_profile_enable(ctx.handle, 1 if enable else 0))


def fd_profile_read(ctx: Context, stream=None):
    """Returns {group: (milliseconds, kernels)} accumulated since the last read."""
    n = len(PROF_GROUPS)
    ms = (ctypes.c_float * n)()
    cnt = (ctypes.c_int32 * n)()
    _check(ctx.handle, lib.fd_profile_read(ctx.handle, _stream(stream), ms, cnt))
    return {PROF_GROUPS[i]: (float(ms[i]), int(cnt[i])) for i in range(n)}


def make_config(wl, max_batch=None, max_tokens=None, max_regions=None, n_blocks=None, engine=FD_ENGINE_AUTO,
                ln_eps=1e-6, gate_eta=1e-12, max_skip_k=5) -> FdConfig:
    """fd_config from a workload description (anything with L, H, heads, head_dim, M, Hc, B, N, R, dtype)."""
    return FdConfig(
        n_blocks=wl.L if n_blocks is None else n_blocks, hidden=wl.H, n_heads=wl.heads, head_dim=wl.head_dim,
        mlp_dim=wl.M, cond_dim=wl.Hc, max_batch=wl.B if max_batch is None else max_batch,
        max_tokens=wl.N if max_tokens is None else max_tokens,
        max_regions=wl.R if max_regions is None else max_regions,
        dtype=FD_BF16 if wl.dtype == "bf16" else FD_F32, engine=engine, ln_eps=ln_eps, gate_eta=gate_eta,
        max_skip_k=max_skip_k)
