"""avggt_project_build_kv (the K/V projection with the compaction in its epilogue) against the fp64 oracle,
through the C ABI.

Tolerances, from the arithmetic: the kernel accumulates bf16 x bf16 products in fp32 and rounds once to bf16, so
each stored value lies within half a bf16 step (at most 2^-8 of its size) of the exact projection, plus the fp32 accumulation error
(bounded here by 2e-6 of the sum of the absolute products).  The compact rows are bit copies of the kernel's own
full rows, the index list is exact, and the mean pair (fp32 sums of the un-rounded projections) is within 1e-5 of
the summand scale, as for avggt_build_kv.
"""

import numpy as np
import pytest
import torch

import paper_2512_02541_b200 as P
from oracle import avggt_oracle as orc
from paper_2512_02541_b200 import inputs

pytestmark = pytest.mark.gpu


def _run(wl, C, seed, with_bias=True, want_full=True):
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                           diag=wl.diag, mean_fill=wl.mean_fill, keep_first_frame=bool(wl.keep_first_frame))
    ocfg = orc.SGAConfig(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                         diag=bool(wl.diag), mean_fill=wl.mean_fill, keep_first_frame=bool(wl.keep_first_frame))
    gen = torch.Generator(device="cuda").manual_seed(seed)
    H, d, n_tok = wl.n_heads, wl.head_dim, wl.n_tokens
    X = torch.randn((n_tok, C), generator=gen, device="cuda").bfloat16()
    Wk = (torch.randn((H * d, C), generator=gen, device="cuda") * C ** -0.5).bfloat16()
    Wv = (torch.randn((H * d, C), generator=gen, device="cuda") * C ** -0.5).bfloat16()
    bk = torch.randn((H * d,), generator=gen, device="cuda") if with_bias else None
    bv = torch.randn((H * d,), generator=gen, device="cuda") if with_bias else None
    M, n_dropped = P.avggt_kv_count(params)
    K = torch.full((n_tok, H, d), float("nan"), dtype=torch.bfloat16, device="cuda") if want_full else None
    V = torch.full_like(K, float("nan")) if want_full else None
    Kc = torch.full((H, M, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    Vc = torch.full_like(Kc, float("nan"))
    idx = torch.full((M,), -1, dtype=torch.int32, device="cuda")
    kmean = torch.full((H, d), float("nan"), device="cuda")
    vmean = torch.full_like(kmean, float("nan"))
    wsb = P.avggt_project_workspace_bytes(params, C)
    ws = torch.zeros((wsb,), dtype=torch.uint8, device="cuda")
    P.avggt_project_build_kv(params, C, X, Wk, Wv, bk, bv, K, V, Kc, Vc, idx, kmean, vmean, ws, ws.numel())
    torch.cuda.synchronize()
    P.avggt_check_status(ws)
    host = lambda t: None if t is None else t.float().cpu().numpy().astype(np.float64)
    want = orc.project_build_kv(ocfg, host(X), host(Wk), host(Wv), host(bk), host(bv))
    absprod_k = np.abs(host(X)) @ np.abs(host(Wk)).T + (np.abs(host(bk)) if with_bias else 0.0)
    absprod_v = np.abs(host(X)) @ np.abs(host(Wv)).T + (np.abs(host(bv)) if with_bias else 0.0)
    return ocfg, dict(K=K, V=V, Kc=Kc, Vc=Vc, idx=idx, kmean=kmean, vmean=vmean), want, (absprod_k, absprod_v), (host(X), host(Wk), host(Wv), host(bk), host(bv))


def _check(wl, C, seed, with_bias=True, want_full=True):
    ocfg, got, want, absprod, hosts = _run(wl, C, seed, with_bias, want_full)
    K_b, V_b, Kc_w, Vc_w, idx_w, kmean_w, vmean_w = want
    H, d, n_tok = wl.n_heads, wl.head_dim, wl.n_tokens
    X, Wk, Wv, bk, bv = hosts
    np.testing.assert_array_equal(got["idx"].cpu().numpy(), idx_w)
    exact = [X @ Wk.T + (bk if bk is not None else 0.0), X @ Wv.T + (bv if bv is not None else 0.0)]
    for which, (full, compact, compact_w) in enumerate(((got["K"], got["Kc"], Kc_w), (got["V"], got["Vc"], Vc_w))):
        ex = exact[which].reshape(n_tok, H, d)
        bound = 2.0 ** -8 * np.abs(ex) * (1 + 1e-3) + 2e-6 * absprod[which].reshape(n_tok, H, d) + 1e-30
        c = compact.float().cpu().numpy().astype(np.float64).transpose(1, 0, 2)             # [M, H, d]
        assert np.isfinite(c).all()
        assert (np.abs(c - ex[idx_w]) <= bound[idx_w]).all()
        # nearly all values are the oracle's rounded values bit for bit (a few sit next to a rounding boundary)
        assert (c == compact_w).mean() > 0.995
        if full is not None:
            f = full.float().cpu().numpy().astype(np.float64)
            assert np.isfinite(f).all()
            assert (np.abs(f - ex) <= bound).all()
            np.testing.assert_array_equal(c, f[idx_w])                                      # compact rows = the kernel's own rows
    if ocfg.mean_fill != 0 and kmean_w is not None:
        for g, w, ex in ((got["kmean"], kmean_w, exact[0]), (got["vmean"], vmean_w, exact[1])):
            scale = max(float(np.abs(ex).mean()), 1e-6)
            assert np.abs(g.cpu().numpy().astype(np.float64) - w).max() <= 1e-5 * scale


@pytest.mark.parametrize("C", (64, 192, 1024))
@pytest.mark.parametrize("sigma", (1, 4, 9))
def test_small_shapes(C, sigma):
    wl = inputs.Workload("proj", 3, 9, 11, 5, 4, 64, sigma, 1, 2, "iid")          # 312 tokens: tiles 128, 128, 56
    _check(wl, C, seed=10 + sigma)


def test_heads_not_a_multiple_of_four_and_no_bias_and_no_full_arrays():
    wl = inputs.Workload("proj_h6", 2, 7, 9, 5, 6, 64, 2, 1, 2, "iid")            # 384 output columns: one and a half column tiles
    _check(wl, 128, seed=3, with_bias=False, want_full=False)
    wl = inputs.Workload("proj_h1", 5, 6, 6, 0, 1, 64, 6, 1, 1, "iid", keep_first_frame=1)
    _check(wl, 64, seed=4)


def test_vggt_shape_twenty_frames():
    """20 frames of the VGGT layer (27,480 tokens, 1024 channels, 16 heads): many tiles per CTA, both accumulators in use."""
    wl = inputs.WORKLOADS["vggt_n100_s4"].with_(n_frames=20, name="vggt_n20_s4")
    _check(wl, 1024, seed=5)


def test_results_are_deterministic_and_feed_the_attention():
    wl = inputs.Workload("proj_det", 4, 12, 12, 5, 8, 64, 4, 1, 2, "iid")
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma)
    ocfg, got1, want, _, hosts = _run(wl, 256, seed=8)
    _, got2, _, _, _ = _run(wl, 256, seed=8)
    for k in ("K", "V", "Kc", "Vc", "idx", "kmean", "vmean"):
        assert torch.equal(got1[k], got2[k]), k
    # the fused outputs through the attention kernel against the oracle on the same (rounded) K and V
    gen = torch.Generator(device="cuda").manual_seed(99)
    Q = (torch.randn((wl.n_tokens, wl.n_heads, wl.head_dim), generator=gen, device="cuda") * 2).bfloat16()
    _, aws = P.avggt_workspace_bytes(params)
    ws = torch.zeros((aws,), dtype=torch.uint8, device="cuda")
    O = torch.full_like(Q, float("nan"))
    P.avggt_global_attn(params, Q, got1["K"], got1["V"], got1["Kc"], got1["Vc"], got1["kmean"], got1["vmean"], O, None, ws, ws.numel())
    torch.cuda.synchronize()
    P.avggt_check_status(ws)
    Kh, Vh = got1["K"].float().cpu().numpy(), got1["V"].float().cpu().numpy()
    ref = orc.global_attn_blocked(ocfg, Q.float().cpu().numpy(), Kh, Vh, np.arange(wl.n_tokens))
    err = np.abs(O.float().cpu().numpy().astype(np.float64) - ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3


def test_argument_errors_do_not_launch():
    wl = inputs.Workload("proj_args", 2, 4, 4, 5, 2, 64, 4, 1, 2, "iid")
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma)
    X = torch.zeros((wl.n_tokens, 96), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((128, 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.AvggtError) as ei:       # channels not a multiple of 64
        P.avggt_project_workspace_bytes(params, 96)
    assert ei.value.code == -2
    X = torch.zeros((wl.n_tokens, 128), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((128, 128), dtype=torch.bfloat16, device="cuda")
    M, _ = P.avggt_kv_count(params)
    Kc = torch.zeros((2, M, 64), dtype=torch.bfloat16, device="cuda")
    km = torch.zeros((2, 64), device="cuda")
    ws = torch.zeros((P.avggt_project_workspace_bytes(params, 128),), dtype=torch.uint8, device="cuda")
    with pytest.raises(P.AvggtError) as ei:       # workspace too small
        P.avggt_project_build_kv(params, 128, X, W, W, None, None, None, None, Kc, Kc.clone(), None, km, km.clone(), ws, 64)
    assert ei.value.code == -3
    with pytest.raises(P.AvggtError) as ei:       # K without V
        P.avggt_project_build_kv(params, 128, X, W, W, None, None, torch.zeros((wl.n_tokens, 2, 64), dtype=torch.bfloat16, device="cuda"),
                                 None, Kc, Kc.clone(), None, km, km.clone(), ws, ws.numel())
    assert ei.value.code == -1
    torch.cuda.synchronize()
