"""Parity of the caller-chosen retained set (avggt_build_kv_indexed + avggt_global_attn_indexed) with the
fp64 oracle, through the C ABI.  Tolerances as for the grid layer."""

import numpy as np
import pytest
import torch

import paper_2512_02541_b200 as P
from oracle import avggt_oracle as orc
from paper_2512_02541_b200 import inputs

pytestmark = pytest.mark.gpu


def _run(wl, idx_np, seed=0):
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                           diag=wl.diag, mean_fill=wl.mean_fill)
    ocfg = orc.SGAConfig(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                         diag=bool(wl.diag), mean_fill=wl.mean_fill)
    Q, K, V = inputs.make_qkv(wl, seed=seed, device="cuda")
    H, d, n_tok, M = wl.n_heads, wl.head_dim, wl.n_tokens, len(idx_np)
    idx = torch.as_tensor(idx_np, dtype=torch.int32, device="cuda")
    Kc = torch.full((H, M, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    Vc = torch.full_like(Kc, float("nan"))
    slots = torch.full((n_tok,), 12345, dtype=torch.int32, device="cuda")
    kmean = torch.zeros((H, d), dtype=torch.float32, device="cuda")
    vmean = torch.zeros_like(kmean)
    bws, aws = P.avggt_workspace_bytes(params)
    ws_b = torch.empty((max(bws, 16),), dtype=torch.uint8, device="cuda")
    ws_a = torch.zeros((max(aws, 16),), dtype=torch.uint8, device="cuda")
    lse = torch.empty((n_tok, H), dtype=torch.float32, device="cuda")
    O = torch.full_like(Q, float("nan"))
    P.avggt_build_kv_indexed(params, idx, M, K, V, Kc, Vc, slots, kmean, vmean, ws_b, ws_b.numel())
    P.avggt_global_attn_indexed(params, M, slots, Q, K, V, Kc, Vc, kmean, vmean, O, lse, ws_a, ws_a.numel())
    torch.cuda.synchronize()
    P.avggt_check_status(ws_a)
    return ocfg, Q, K, V, Kc, Vc, slots, kmean, vmean, O, lse


def _check(wl, idx_np, seed, rows=None):
    ocfg, Q, K, V, Kc, Vc, slots, kmean, vmean, O, lse = _run(wl, idx_np, seed)
    Qh, Kh, Vh = (t.float().cpu().numpy() for t in (Q, K, V))
    n_tok = wl.n_tokens
    # the map and the gathered rows are exact
    want_slots = np.full(n_tok, -1, dtype=np.int32)
    want_slots[idx_np] = np.arange(len(idx_np), dtype=np.int32)
    np.testing.assert_array_equal(slots.cpu().numpy(), want_slots)
    np.testing.assert_array_equal(Kc.float().cpu().numpy().transpose(1, 0, 2), Kh[idx_np])
    np.testing.assert_array_equal(Vc.float().cpu().numpy().transpose(1, 0, 2), Vh[idx_np])
    dropped = want_slots < 0
    if ocfg.mean_fill != 0 and dropped.any():
        for got, src in ((kmean, Kh), (vmean, Vh)):
            want = src[dropped].mean(axis=0, dtype=np.float64)
            assert np.abs(got.cpu().numpy() - want).max() <= 1e-5 * max(float(np.abs(src).mean()), 1e-6)
    if rows is None:
        rows = np.arange(n_tok)
    want, want_lse = orc.global_attn_indexed(ocfg, idx_np, Qh, Kh, Vh, rows=rows, return_lse=True)
    ridx = torch.as_tensor(rows, device="cuda")
    got = O[ridx].float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    err = np.abs(got - want)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())
    assert np.abs(lse[ridx].cpu().numpy() - want_lse).max() <= 2e-3


@pytest.mark.parametrize("diag,mean_fill", [(0, 0), (1, 0), (0, 2), (1, 2), (1, 1)])
def test_random_subset(diag, mean_fill):
    wl = inputs.Workload("rand", 3, 9, 11, 5, 4, 64, 4, diag, mean_fill, "iid")
    rng = np.random.default_rng(100 + 10 * diag + mean_fill)
    idx = np.sort(rng.permutation(wl.n_tokens)[:137]).astype(np.int32)      # a ragged tail, special tokens dropped too
    _check(wl, idx, seed=3)


@pytest.mark.parametrize("diag,mean_fill", [(0, 2), (0, 1), (1, 2), (1, 1), (1, 0)])
def test_nothing_retained_is_the_single_mean_pair_layer(diag, mean_fill):
    """G2M (Sec. 5.4): no retained keys at all; one mean pair over every token (special tokens included) and,
    with the diagonal on, the query's own column.  Several query tiles and a ragged tail."""
    wl = inputs.Workload("g2m", 3, 10, 13, 5, 4, 64, 4, diag, mean_fill, "proj")
    _check(wl, np.zeros(0, dtype=np.int32), seed=7)


def test_nothing_retained_and_no_other_column_is_rejected():
    wl = inputs.Workload("g2m_none", 2, 4, 4, 5, 2, 64, 4, 0, 0, "iid")
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma, diag=0, mean_fill=0)
    Q, K, V = inputs.make_qkv(wl, seed=0, device="cuda")
    slots = torch.empty((wl.n_tokens,), dtype=torch.int32, device="cuda")
    ws = torch.empty((1 << 20,), dtype=torch.uint8, device="cuda")
    with pytest.raises(P.AvggtError) as ei:
        P.avggt_build_kv_indexed(params, None, 0, K, V, None, None, slots, None, None, ws, ws.numel())
    assert ei.value.code == -1
    torch.cuda.synchronize()


def test_grid_subset_given_as_a_list_equals_the_grid_layer():
    wl = inputs.Workload("grid_as_list", 4, 12, 12, 5, 8, 64, 4, 1, 2, "proj")
    ocfg = orc.SGAConfig(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma)
    idx = orc.build_index(ocfg)
    _check(wl, idx, seed=4)
    # bit-identical to the window-rule entry points on the same inputs
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma)
    Q, K, V = inputs.make_qkv(wl, seed=4, device="cuda")
    layer = P.SubsampledGlobalAttention(params)
    O_rule = layer.forward(Q, K, V)
    layer.check_status()
    O_list = _run(wl, idx, seed=4)[9]
    assert torch.equal(O_rule, O_list)


def test_everything_kept_is_dense():
    wl = inputs.Workload("all", 2, 8, 9, 5, 2, 64, 9, 1, 2, "iid")
    _check(wl, np.arange(wl.n_tokens, dtype=np.int32), seed=5)


def test_larger_random_quarter():
    """20 frames of the VGGT grid with a random quarter of all tokens retained, on sampled rows."""
    wl = inputs.WORKLOADS["vggt_n100_s4"].with_(n_frames=20, name="vggt_n20_rand")
    rng = np.random.default_rng(9)
    idx = np.sort(rng.permutation(wl.n_tokens)[: wl.n_tokens // 4]).astype(np.int32)
    _check(wl, idx, seed=6, rows=inputs.sample_rows(wl, 96).numpy())


def test_argument_errors_do_not_launch():
    wl = inputs.Workload("args", 2, 4, 4, 5, 2, 64, 4, 1, 2, "iid")
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma)
    Q, K, V = inputs.make_qkv(wl, seed=0, device="cuda")
    idx = torch.arange(0, wl.n_tokens, 2, dtype=torch.int32, device="cuda")
    M = idx.numel()
    Kc = torch.empty((2, M, 64), dtype=torch.bfloat16, device="cuda"); Vc = torch.empty_like(Kc)
    slots = torch.empty((wl.n_tokens,), dtype=torch.int32, device="cuda")
    km = torch.zeros((2, 64), device="cuda"); vm = torch.zeros_like(km)
    bws, aws = P.avggt_workspace_bytes(params)
    ws = torch.empty((max(bws, aws, 16),), dtype=torch.uint8, device="cuda")
    with pytest.raises(P.AvggtError) as ei:      # more retained tokens than tokens
        P.avggt_build_kv_indexed(params, idx, wl.n_tokens + 1, K, V, Kc, Vc, slots, km, vm, ws, ws.numel())
    assert ei.value.code == -1
    with pytest.raises(P.AvggtError) as ei:      # no map
        P.avggt_global_attn_indexed(params, M, None, Q, K, V, Kc, Vc, km, vm, Q.clone(), None, ws, ws.numel())
    assert ei.value.code == -1
    with pytest.raises(P.AvggtError) as ei:      # workspace too small
        P.avggt_build_kv_indexed(params, idx, M, K, V, Kc, Vc, slots, km, vm, ws, 8)
    assert ei.value.code == -3
    torch.cuda.synchronize()
