"""The attention stage on its own inputs: the library's query rows and its K/V cache are read back (fd_debug_buffer) and
softmax(q k^T / sqrt(d)) v is evaluated from its definition (paper Sec. 5: active queries against the keys and values of
every position) in fp64 on exactly those bf16 numbers, so that nothing upstream blurs the comparison.  The cache is given
a few very large keys late in the sequence: the scores of later key tiles then exceed the first tile's maximum by far
more than the rescaling threshold, which forces the accumulator rescaling (and the redo of a tile whose row sum ran out
of range) that ordinary inputs never reach."""
import numpy as np
import pytest
import torch

import gen
import paper_2607_12121_b200 as fd
from harness import StepBuffers, dev, gpu_step, labels_for, make_ctx

pytestmark = pytest.mark.gpu

LOG2E = 1.4426950408889634


def _buffer(ctx, which):
    ptr, nbytes = fd.fd_debug_buffer(ctx, which)
    off = ptr - ctx.workspace.data_ptr()
    return ctx.workspace[off:off + nbytes].view(torch.bfloat16)


@pytest.mark.parametrize("name,n_tok,env", [("audio_tc", None, {}), ("image_tc", None, {}), ("video_tc", None, {}),
                                            ("wide_tc", 900, {"FD_ATT_SPLIT": "2", "FD_TC_MAX_CTAS": "8"}),
                                            ("audio_tc", 700, {"FD_ATT_SPLIT": "2", "FD_TC_MAX_CTAS": "8"})])
def test_attention_on_its_own_inputs_with_giant_late_keys(monkeypatch, name, n_tok, env):
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    wl = gen.workload(name).replace(L=1)
    if name == "image_tc":                                       # five key tiles instead of two
        wl = wl.replace(grid=(24, 24), R=24, n_cells=24, m_min=8, m_max=64)
    if n_tok is not None:
        wl = wl.replace(grid=(n_tok,), R=10)
    seed = 21
    B, N, H, heads, dh = wl.B, wl.N, wl.H, wl.heads, wl.head_dim
    labels = labels_for(wl, seed)
    w = gen.block_weights(wl, seed, n_blocks=1)
    inp = gen.step_inputs(wl, seed, labels)
    ctx = make_ctx(wl, w, engine=fd.FD_ENGINE_TC, n_blocks=1)
    buf = StepBuffers(wl, 1)
    dt = torch.bfloat16
    gpu_step(ctx, wl, dev(inp["x_prev"], dt), dev(inp["cond"], dt), dev(labels), dev(np.ones((B, wl.R), np.uint8)), buf)

    # skipped regions: those that own most of the second half of the sequence; their keys there become 256 times larger
    mask = gen.region_mask(wl, 5, [0.5] * B)
    lab = labels.reshape(B, N)
    skipped_tok = np.zeros((B, N), bool)
    for b in range(B):
        skipped_tok[b] = (lab[b] < wl.R) & (mask[b][np.minimum(lab[b], wl.R - 1)] == 0)
    giant = skipped_tok & (np.arange(N)[None, :] >= N // 2) & (np.arange(N)[None, :] % 7 == 0)
    assert giant.sum() >= 4
    g = torch.from_numpy(giant).cuda()
    buf.kv[0, :, 0][g] = buf.kv[0, :, 0][g] * 256                     # exact in bf16

    idx, cu = gpu_step(ctx, wl, dev(inp["x_cur"], dt), dev(inp["cond"], dt), dev(labels), dev(mask), buf)
    A = int(cu[-1])
    assert 0 < A < B * N
    q_all = _buffer(ctx, fd.FD_BUF_Q)
    q_ld = q_all.numel() // (fd.fd_debug_buffer(ctx, fd.FD_BUF_ATTN)[1] // 2 // H)
    q = q_all[: A * q_ld].view(A, q_ld).to(torch.float64).cpu().numpy()
    o = _buffer(ctx, fd.FD_BUF_ATTN)[: A * H].view(A, H).to(torch.float64).cpu().numpy()
    kv = buf.kv[0].to(torch.float64).cpu().numpy()                     # [B, 2, N, H]: fresh rows of active tokens included
    hs = q_ld // heads                                                 # a head's stride in the query rows (80 for head dim 72)
    o_ref = np.empty((A, H))
    forced = 0
    for b in range(B):
        rows = np.arange(cu[b], cu[b + 1])
        if rows.size == 0:
            continue
        for h in range(heads):
            qh = q[rows][:, h * hs:h * hs + dh]
            s = qh @ kv[b, 0][:, h * dh:(h + 1) * dh].T / np.sqrt(dh)
            p = np.exp(s - s.max(1, keepdims=True))
            o_ref[rows, h * dh:(h + 1) * dh] = (p / p.sum(1, keepdims=True)) @ kv[b, 1][:, h * dh:(h + 1) * dh]
            # rows whose later key tiles (of either tile parity) outgrow that parity's first tile by more than 2^24
            for par in (0, 1):
                tiles = [s[:, t * 128:(t + 1) * 128].max(1) for t in range(par, (N + 127) // 128, 2)]
                if len(tiles) > 1:
                    forced += int(((np.max(tiles[1:], axis=0) - tiles[0]) * LOG2E > 24).sum())
    assert forced > 50, forced                                         # the rescaling path is what this case is about
    err = np.abs(o - o_ref)
    vmax = np.abs(kv[:, 1]).max()
    assert err.max() <= 2.0 ** -7 * max(1.0, vmax), (err.max(), vmax)   # P and the output are bf16: two roundings of 2^-9 each, with margin
    assert np.sqrt((err ** 2).sum() / (o_ref ** 2).sum()) <= 4e-3
    assert fd.fd_destroy(ctx) == fd.FD_OK
