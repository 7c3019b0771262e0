"""Shared helpers of the GPU parity tests: move seeded arrays to the device, call the C-ABI
through the binding, bring results back as numpy."""
from __future__ import annotations

import numpy as np
import torch

import gen
import oracle
import paper_2607_12121_b200 as fd


def tdtype(wl):
    return torch.bfloat16 if wl.dtype == "bf16" else torch.float32


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t if dtype is None else t.to(dtype)


def host(t) -> np.ndarray:
    return t.detach().float().cpu().numpy() if t.is_floating_point() else t.detach().cpu().numpy()


def make_ctx(wl, w_np, engine=fd.FD_ENGINE_AUTO, n_blocks=None, **kw):
    L = wl.L if n_blocks is None else n_blocks
    weights = {k: dev(v[:L], tdtype(wl)) for k, v in w_np.items()}
    cfg = fd.make_config(wl, n_blocks=L, engine=engine, **kw)
    return fd.fd_create(cfg, weights)


class StepBuffers:
    def __init__(self, wl, L):
        B, N, H = wl.B, wl.N, wl.H
        dt = tdtype(wl)
        self.kv = torch.zeros((L, B, 2, N, H), dtype=dt, device="cuda")
        self.y = torch.zeros((B, N, H), dtype=dt, device="cuda")
        self.active_idx = torch.full((B * N,), -1, dtype=torch.int32, device="cuda")
        self.cu_active = torch.zeros((B + 1,), dtype=torch.int32, device="cuda")


def gpu_step(ctx, wl, x, cond, labels, mask, buf: StepBuffers):
    fd.fd_regional_step(ctx, x, cond, labels, mask, wl.R, buf.kv, buf.y, buf.active_idx, buf.cu_active)
    fd.fd_poll_status(ctx)
    cu = host(buf.cu_active)
    return host(buf.active_idx)[: cu[-1]], cu


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def max_abs(a, b):
    return float(np.max(np.abs(np.asarray(a, np.float64) - np.asarray(b, np.float64)))) if np.size(a) else 0.0


def labels_for(wl, seed):
    """Uniform labels, or the oracle partition of the synthetic saliency map (+ text label R)."""
    if wl.labels != "partition":
        return gen.uniform_labels(wl)
    amap = gen.saliency_map(wl, seed)
    lab, _ = oracle.partition(amap, None, wl.R, wl.m_min, wl.m_max)
    text = np.full((wl.B, wl.n_text), wl.R, np.int32)
    return np.ascontiguousarray(np.concatenate([lab, text], axis=1))
