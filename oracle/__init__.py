"""TEST INFRASTRUCTURE -- CPU oracle of the region-selective denoising step.

Only ``tests/``, the smoke check and the CPU-baseline leg of the benchmark may import this
package; the CUDA library never does, and shares no code with it.  Parity status: every
function here is pinned by the CPU test-suite against closed forms, brute force, invariants
and independent library routines, except two conventions that nothing outside this build
fixes ("parity unpinned"): the choice of the root-mean-square as the magnitude of the latent
change, and the 16-bit width of the saliency quantisation.

* ``partition``      -- Patch Partitioner (paper Sec. 4.1, Appendix A.3)
* ``activity_gate``  -- Patch Gate (Sec. 4.2, Appendix A.1)
* ``compact``        -- active set -> ragged token index list (Algorithm 1, PatchGate output)
* ``regional_step``  -- all blocks on active tokens with stale K/V for skipped patches
                        (Sec. 3, Sec. 5, Appendix A.6)
* ``dense_step``     -- the ungated baseline trajectory, written separately
* ``sampler_embed``, ``sampler_update`` -- patch embedding and the latent update with cached drift
                        (Appendix A.1, Eq. sf-update)
"""
from __future__ import annotations

import ctypes
from typing import Dict, Optional

import numpy as np

from .build import build as _build
from .gate import activity_gate, attention_gate, attention_mass, compact, initial_state  # noqa: F401
from .sampler import embed as sampler_embed, update as sampler_update, token_drift  # noqa: F401
from .partitioner import partition, partition_request, saliency, quantise, allocate, best_cut  # noqa: F401

class _Stream(ctypes.Structure):          # fdo_stream of regional_block.c
    _fields_ = [(n, ctypes.c_void_p) for n in ("mod", "w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2",
                                               "qn_w", "kn_w")]


class _DenseWeights(ctypes.Structure):    # fdo_dense_weights of dense_block.c
    _fields_ = [(n, ctypes.c_void_p) for n in ("w_ada", "b_ada", "w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1", "w_fc2",
                                               "b_fc2", "qn_w", "kn_w")]


class _Cross(ctypes.Structure):           # fdo_cross / fdo_dense_cross
    _fields_ = [(n, ctypes.c_void_p) for n in ("w_q", "b_q", "w_o", "b_o", "ctx_kv")] + [("T", ctypes.c_int)]


class _Fp8(ctypes.Structure):             # fdo_fp8 / fdo_dense_fp8
    _fields_ = [(n, ctypes.c_void_p) for n in ("w_qkv", "s_qkv", "w_fc1", "s_fc1", "w_fc2", "s_fc2")] + \
               [(n, ctypes.c_float) for n in ("a_qkv", "a_fc1", "a_fc2")]


_lib = None
_f = ctypes.POINTER(ctypes.c_float)
_i = ctypes.POINTER(ctypes.c_int32)


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build())
        _lib.fdo_adaln.restype = ctypes.c_int
        _lib.fdo_regional_block.restype = ctypes.c_int
        _lib.fdo_dense_block.restype = ctypes.c_int
        _lib.fdo_regional_block_v.restype = ctypes.c_int
        _lib.fdo_dense_block_v.restype = ctypes.c_int
        _lib.fdo_regional_block_s.restype = ctypes.c_int
        _lib.fdo_dense_block_d.restype = ctypes.c_int
        _lib.fdo_regional_block_x.restype = ctypes.c_int
        _lib.fdo_dense_block_x.restype = ctypes.c_int
        _lib.fdo_regional_block_q.restype = ctypes.c_int
        _lib.fdo_dense_block_q.restype = ctypes.c_int
        _lib.fdo_regional_e4m3.restype = None
        _lib.fdo_dense_e4m3.restype = None
        _lib.fdo_regional_linear_fp8.restype = None
    return _lib


def _fp(a: np.ndarray):
    assert a.dtype == np.float32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_f)


def _ip(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.dtype == np.int32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_i)


def _c(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def adaln(cond: np.ndarray, w_ada: np.ndarray, b_ada: np.ndarray) -> np.ndarray:
    """mod [B,6H] = W_ada SiLU(cond) + b_ada for one block."""
    B, Hc = cond.shape
    H = w_ada.shape[0] // 6
    mod = np.empty((B, 6 * H), np.float32)
    rc = _load().fdo_adaln(B, H, Hc, _fp(_c(cond)), _fp(_c(w_ada)), _fp(_c(b_ada)), _fp(mod))
    assert rc == 0
    return mod


def _addr(a: Optional[np.ndarray], keep: list) -> Optional[int]:
    if a is None:
        return None
    a = _c(a)
    keep.append(a)
    return a.ctypes.data


def _cross_arg(v, l: int, B: int, H: int, keep: list):
    """fdo_cross of block ``l`` from variants["cross"] = {w_q [L,H,H], b_q [L,H], w_o, b_o, ctx_kv [L,B,2,T,H]}."""
    c = v.get("cross")
    if c is None:
        return None
    kvc = _c(c["ctx_kv"][l])
    assert kvc.shape[0] == B and kvc.shape[1] == 2 and kvc.shape[3] == H
    keep.append(kvc)
    st = _Cross(_addr(c["w_q"][l], keep), _addr(c["b_q"][l], keep), _addr(c["w_o"][l], keep), _addr(c["b_o"][l], keep),
                kvc.ctypes.data, int(kvc.shape[2]))
    keep.append(st)
    return ctypes.byref(st)


def _fp8_arg(v, l: int, keep: list):
    """fdo_fp8 of block ``l`` from variants["fp8"] = {w_qkv [L,3H,H], s_qkv [L,3H], w_fc1, s_fc1, w_fc2, s_fc2: the E4M3
    values of the quantised weights and their per-row scales; a_scale [L,3]: activation scales of QKV, fc1, fc2}
    (the second stream's: variants["text"]["fp8"], handed over as the dict itself)."""
    f = v.get("fp8")
    if f is None:
        return None
    a = np.asarray(f["a_scale"], np.float32)[l]
    st = _Fp8(*(_addr(f[k][l], keep) for k in ("w_qkv", "s_qkv", "w_fc1", "s_fc1", "w_fc2", "s_fc2")),
              float(a[0]), float(a[1]), float(a[2]))
    keep.append(st)
    return ctypes.byref(st)


def e4m3(x: np.ndarray, program: str = "regional") -> np.ndarray:
    """Nearest E4M3 value of every element (ties to even, saturating at 448), by either C program's quantiser."""
    x = _c(x)
    y = np.empty_like(x)
    getattr(_load(), "fdo_regional_e4m3" if program == "regional" else "fdo_dense_e4m3")(int(x.size), _fp(x), _fp(y))
    return y


def linear_fp8(x: np.ndarray, a_scale: float, w8: np.ndarray, w_scale: np.ndarray, bias: np.ndarray) -> np.ndarray:
    """One row through the FP8 projection of the regional program: x [K], w8 [O,K] E4M3 values, w_scale, bias [O]."""
    x, w8, w_scale, bias = _c(x), _c(w8), _c(w_scale), _c(bias)
    y = np.empty(w8.shape[0], np.float32)
    _load().fdo_regional_linear_fp8(_fp(x), ctypes.c_float(a_scale), _fp(w8), _fp(w_scale), _fp(bias), int(w8.shape[1]),
                                    int(w8.shape[0]), _fp(y))
    return y


def regional_block(u_in: np.ndarray, active_idx: np.ndarray, mod: np.ndarray, w: Dict[str, np.ndarray],
                   l: int, kv_l: np.ndarray, heads: int, ln_eps: float = 1e-6,
                   finish: Optional[np.ndarray] = None, variants=None, mod_text: Optional[np.ndarray] = None,
                   tok_text: Optional[np.ndarray] = None) -> np.ndarray:
    """One block over the compact rows ``u_in`` [A,H]; ``kv_l`` [B,2,N,H] is updated in place.
    Dual stream: ``variants["text"]`` holds the second stream's weights (same keys as ``w``, optionally its own
    q_norm_w / k_norm_w), ``mod_text`` [B,6H] its adaLN vectors and ``tok_text`` [B*N] u8 marks its tokens."""
    A, H = u_in.shape
    B, _, N, _ = kv_l.shape
    M = w["w_fc1"].shape[1]
    dh = H // heads
    assert kv_l.dtype == np.float32 and kv_l.flags["C_CONTIGUOUS"]
    u_out = np.zeros((A, H), np.float32)
    fin = None if finish is None else np.ascontiguousarray(finish, np.int32)
    v = variants or {}
    keep: list = []

    def stream(ws, md, qn, kn):
        return _Stream(_addr(md, keep), *[_addr(ws[k][l], keep) for k in ("w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1",
                                                                            "w_fc2", "b_fc2")],
                       _addr(None if qn is None else qn[l], keep), _addr(None if kn is None else kn[l], keep))

    img = stream(w, mod, v.get("q_norm_w"), v.get("k_norm_w"))
    txt, tt = None, None
    if v.get("text") is not None:
        t = v["text"]
        assert mod_text is not None and tok_text is not None
        txt = ctypes.byref(stream(t["weights"], mod_text, t.get("q_norm_w", v.get("q_norm_w")),
                                  t.get("k_norm_w", v.get("k_norm_w"))))
        tt = np.ascontiguousarray(tok_text, np.uint8)
        keep.append(tt)
    rc_, rs_ = _addr(v.get("rope_cos"), keep), _addr(v.get("rope_sin"), keep)
    if rc_ is not None:
        assert keep[-2].shape == (N, dh // 2)
    rc = _load().fdo_regional_block_q(
        B, N, H, heads, dh, M, A, _ip(np.ascontiguousarray(active_idx, np.int32)), ctypes.byref(img), txt,
        None if tt is None else tt.ctypes.data_as(ctypes.c_void_p), ctypes.c_float(ln_eps), _fp(_c(u_in)), _fp(u_out), _fp(kv_l),
        0 if fin is None else int(fin.size), _ip(fin), ctypes.c_float(float(v.get("qk_norm_eps", 1e-6))),
        ctypes.c_void_p(rc_), ctypes.c_void_p(rs_), _cross_arg(v, l, B, H, keep), _fp8_arg(v, l, keep),
        _fp8_arg(v.get("text") or {}, l, keep))
    assert rc == 0
    return u_out


def regional_step(x: np.ndarray, cond: np.ndarray, labels: np.ndarray, mask: np.ndarray,
                  w: Dict[str, np.ndarray], kv: np.ndarray, y: np.ndarray, heads: int, R: int,
                  ln_eps: float = 1e-6, n_blocks: Optional[int] = None, variants=None):
    """The whole block stack on active tokens.

    x [B,N,H]; kv [L,B,2,N,H] and y [B,N,H] are updated in place: rows of active tokens are
    rewritten, every other row keeps what it held (the cached K/V and the cached output of the
    step at which that token last ran).  Returns active_idx, cu_active.
    """
    B, N, H = x.shape
    L = w["w_qkv"].shape[0] if n_blocks is None else n_blocks
    active_idx, cu_active = compact(mask, labels, R)
    u = np.ascontiguousarray(x.reshape(B * N, H)[active_idx], np.float32)
    text = (variants or {}).get("text")
    tok_text = None if text is None else (np.asarray(labels) == R).reshape(-1).astype(np.uint8)   # always-active tokens
    for l in range(L):
        mod = adaln(cond, w["w_ada"][l], w["b_ada"][l])
        mod_t = None if text is None else adaln(cond, text["weights"]["w_ada"][l], text["weights"]["b_ada"][l])
        u = regional_block(u, active_idx, mod, w, l, kv[l], heads, ln_eps, variants=variants, mod_text=mod_t,
                           tok_text=tok_text)
    y.reshape(B * N, H)[active_idx] = u
    return active_idx, cu_active


def block0_projection(x: np.ndarray, cond: np.ndarray, w: Dict[str, np.ndarray], active_idx: np.ndarray,
                      part: int = 0, ln_eps: float = 1e-6) -> np.ndarray:
    """Rows of the first block's Q (part 0), K (1) or V (2) for the active tokens, [A,H] fp32: LayerNorm +
    adaLN modulation of the gathered rows, then that third of the QKV projection.  The queries, together with the
    block's key cache after the step, are what ``attention_mass`` needs."""
    B, N, H = x.shape
    mod = adaln(cond, w["w_ada"][0], w["b_ada"][0]).astype(np.float64)
    u = x.reshape(B * N, H)[active_idx].astype(np.float64)
    mean = u.mean(-1, keepdims=True)
    var = ((u - mean) ** 2).mean(-1, keepdims=True)
    b = np.asarray(active_idx, np.int64) // N
    un = (u - mean) / np.sqrt(var + ln_eps) * (1.0 + mod[b, H:2 * H]) + mod[b, 0:H]        # scale_msa, shift_msa
    rows = slice(part * H, (part + 1) * H)
    out = un @ w["w_qkv"][0][rows].astype(np.float64).T + w["b_qkv"][0][rows].astype(np.float64)
    return out.astype(np.float32)


def block0_queries(x, cond, w, active_idx, ln_eps: float = 1e-6) -> np.ndarray:
    return block0_projection(x, cond, w, active_idx, 0, ln_eps)


def dense_block(x: np.ndarray, cond: np.ndarray, w: Dict[str, np.ndarray], l: int, heads: int,
                ln_eps: float = 1e-6, variants=None):
    """One ungated block on whole matrices. Returns x_out [B,N,H], kv [B,2,N,H].  Dual stream: ``variants["text"]``
    = {"weights": second weight set, "n_text": trailing tokens of every request that belong to it}."""
    B, N, H = x.shape
    M = w["w_fc1"].shape[1]
    Hc = cond.shape[1]
    dh = H // heads
    x_out = np.empty((B, N, H), np.float32)
    kv = np.empty((B, 2, N, H), np.float32)
    v = variants or {}
    keep: list = []

    def weights(ws, qn, kn):
        return _DenseWeights(*[_addr(ws[k][l], keep) for k in ("w_ada", "b_ada", "w_qkv", "b_qkv", "w_o", "b_o", "w_fc1",
                                                                 "b_fc1", "w_fc2", "b_fc2")],
                             _addr(None if qn is None else qn[l], keep), _addr(None if kn is None else kn[l], keep))

    wi = weights(w, v.get("q_norm_w"), v.get("k_norm_w"))
    wt, n_text = None, 0
    if v.get("text") is not None:
        t = v["text"]
        wt = ctypes.byref(weights(t["weights"], t.get("q_norm_w", v.get("q_norm_w")), t.get("k_norm_w", v.get("k_norm_w"))))
        n_text = int(t["n_text"])
    rc_, rs_ = _addr(v.get("rope_cos"), keep), _addr(v.get("rope_sin"), keep)
    if rc_ is not None:
        assert keep[-2].shape == (N, dh // 2)
    rc = _load().fdo_dense_block_q(
        B, N, H, heads, dh, M, Hc, _fp(_c(cond)), ctypes.byref(wi), wt, n_text, ctypes.c_float(ln_eps), _fp(_c(x)), _fp(x_out),
        _fp(kv), ctypes.c_float(float(v.get("qk_norm_eps", 1e-6))), ctypes.c_void_p(rc_), ctypes.c_void_p(rs_),
        _cross_arg(v, l, B, H, keep), _fp8_arg(v, l, keep), _fp8_arg(v.get("text") or {}, l, keep))
    assert rc == 0
    return x_out, kv


def dense_step(x: np.ndarray, cond: np.ndarray, w: Dict[str, np.ndarray], heads: int,
               ln_eps: float = 1e-6, n_blocks: Optional[int] = None, variants=None):
    """The ungated block stack. Returns y [B,N,H] and kv [L,B,2,N,H]."""
    L = w["w_qkv"].shape[0] if n_blocks is None else n_blocks
    B, N, H = x.shape
    kv = np.empty((L, B, 2, N, H), np.float32)
    cur = np.ascontiguousarray(x, np.float32)
    for l in range(L):
        cur, kv[l] = dense_block(cur, cond, w, l, heads, ln_eps, variants=variants)
    return cur, kv


def qk_variants(q: np.ndarray, k: np.ndarray, heads: int, pos: Optional[np.ndarray] = None, q_norm_w=None, k_norm_w=None,
                qk_norm_eps: float = 1e-6, rope_cos=None, rope_sin=None, program: str = "regional"):
    """QK-RMSNorm and RoPE as one of the two C programs applies them to query / key rows [n,H] (copies are returned).
    ``program`` = "regional" takes the positions ``pos`` [n]; "dense" takes row t at position t."""
    q, k = _c(q).copy(), _c(k).copy()
    n, H = q.shape
    dh = H // heads
    opt = lambda a: None if a is None else _fp(_c(a))
    keep = [None if a is None else _c(a) for a in (q_norm_w, k_norm_w, rope_cos, rope_sin)]
    ptr = [None if a is None else _fp(a) for a in keep]
    if program == "regional":
        pos = np.arange(n, dtype=np.int32) if pos is None else np.ascontiguousarray(pos, np.int32)
        rc = _load().fdo_regional_qk_variants(n, heads, dh, _ip(pos), _fp(q), _fp(k), ptr[0], ptr[1],
                                              ctypes.c_float(qk_norm_eps), ptr[2], ptr[3])
    else:
        assert pos is None
        rc = _load().fdo_dense_qk_variants(n, heads, dh, _fp(q), _fp(k), ptr[0], ptr[1], ctypes.c_float(qk_norm_eps),
                                           ptr[2], ptr[3])
    assert rc == 0
    return q, k
