"""Parity of avggt_frame_attn (frame attention of converted early global blocks, Sec. 4.2) with the
fp64 oracle, element by element, through the C ABI.  Tolerances as for the global layer."""

import numpy as np
import pytest
import torch

import paper_2512_02541_b200 as P
from oracle import avggt_oracle as orc
from paper_2512_02541_b200 import inputs

pytestmark = pytest.mark.gpu

MAX_ABS_TOL = 2e-2
MEAN_ABS_TOL = 2e-3


def _run(wl, seed=0, want_lse=True):
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                           diag=wl.diag, mean_fill=wl.mean_fill)
    ocfg = orc.SGAConfig(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma)
    Q, K, V = inputs.make_qkv(wl, seed=seed, device="cuda")
    layer = P.SubsampledGlobalAttention(params, want_lse=want_lse)
    O = torch.full_like(Q, float("nan"))
    layer.frame_attend(Q, K, V, out=O)
    layer.check_status()
    return ocfg, layer, Q, K, V, O


def _check(ocfg, layer, Q, K, V, O, rows=None):
    Qh, Kh, Vh = (t.float().cpu().numpy() for t in (Q, K, V))
    if rows is None:
        rows = np.arange(ocfg.n_tokens)
    want, want_lse = orc.frame_attn(ocfg, Qh, Kh, Vh, rows=rows, return_lse=True)
    idx = torch.as_tensor(rows, device=O.device)
    got = O[idx].float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all(), "unwritten or non-finite output rows"
    err = np.abs(got - want)
    assert err.max() <= MAX_ABS_TOL, f"max-abs {err.max():.4g}"
    assert err.mean() <= MEAN_ABS_TOL, f"mean-abs {err.mean():.4g}"
    if layer.lse is not None:
        assert np.abs(layer.lse[idx].cpu().numpy().astype(np.float64) - want_lse).max() <= 2e-3


@pytest.mark.parametrize("n_frames,grid,n_special,heads", [
    (1, (2, 61), 5, 2),     # 127 tokens per frame: one partial tile
    (3, (3, 41), 5, 2),     # 128 tokens per frame exactly: tiles end on frame boundaries
    (4, (4, 31), 5, 3),     # 129: a one-row second tile that reaches into the next frame
    (5, (16, 16), 5, 4),    # 261 tokens: two tiles of queries, three of keys
    (3, (20, 26), 0, 2),    # 520 tokens, no special tokens: three CTAs of queries per frame
    (7, (1, 1), 1, 1),      # two tokens per frame
])
def test_small_frames_all_rows(n_frames, grid, n_special, heads):
    wl = inputs.Workload("frames", n_frames, grid[0], grid[1], n_special, heads, 64, 4, 1, 2, "iid")
    ocfg, layer, Q, K, V, O = _run(wl, seed=n_frames)
    _check(ocfg, layer, Q, K, V, O)


def test_structured_logits():
    wl = inputs.Workload("proj_small", 6, 12, 12, 5, 16, 64, 4, 1, 2, "proj")
    ocfg, layer, Q, K, V, O = _run(wl, seed=11)
    _check(ocfg, layer, Q, K, V, O)


def test_frames_are_independent():
    """Changing one frame's K and V leaves every other frame's output bit-identical."""
    wl = inputs.Workload("indep", 4, 9, 15, 5, 2, 64, 4, 1, 2, "iid")      # 140 tokens: tiles straddle frames
    ocfg, layer, Q, K, V, O = _run(wl, seed=5, want_lse=False)
    L = wl.tokens_per_frame
    K2, V2 = K.clone(), V.clone()
    K2[L:2 * L] = K2[L:2 * L] * 0.5 + 1.0
    V2[L:2 * L] = -V2[L:2 * L]
    O2 = layer.frame_attend(Q, K2, V2)
    layer.check_status()
    assert torch.equal(O2[:L], O[:L]) and torch.equal(O2[2 * L:], O[2 * L:])
    assert not torch.equal(O2[L:2 * L], O[L:2 * L])


def test_vggt_100_frames_sampled_rows():
    """100 frames of 1374 tokens (the benchmark layer's shape) on sampled rows."""
    wl = inputs.WORKLOADS["vggt_n100_s4"]
    ocfg, layer, Q, K, V, O = _run(wl, want_lse=False)
    rows = inputs.sample_rows(wl, 256).numpy()
    _check(ocfg, layer, Q, K, V, O, rows=rows)
    assert torch.isfinite(O.float()).all()


def test_argument_errors_do_not_launch():
    wl = inputs.Workload("args", 2, 4, 4, 5, 2, 64, 4, 1, 2, "iid")
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma)
    Q, K, V = inputs.make_qkv(wl, seed=0, device="cuda")
    layer = P.SubsampledGlobalAttention(params)
    with pytest.raises(P.AvggtError) as ei:
        P.avggt_frame_attn(params, Q, None, V, Q.clone(), None, layer.attn_ws, layer.attn_ws.numel())
    assert ei.value.code == -1
    with pytest.raises(P.AvggtError) as ei:
        P.avggt_frame_attn(params, Q, K, V, Q.clone(), None, layer.attn_ws, 8)
    assert ei.value.code == -3
    with pytest.raises(P.AvggtError) as ei:
        P.avggt_frame_attn(params, Q.data_ptr() + 2, K, V, Q.clone(), None, layer.attn_ws, layer.attn_ws.numel())
    assert ei.value.code == -4
    torch.cuda.synchronize()
