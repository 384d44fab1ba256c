"""Parity of the CUDA path (through the C ABI) with the fp64 oracle, element by element.

Tolerances (stated by the target for bf16 inputs with fp32 accumulation):
max-abs error <= 2e-2 and mean-abs error <= 2e-3 on the attention output;
compacted K/V and indices bit-exact; mean pair within 1e-5 relative to its scale.
"""

import numpy as np
import pytest
import torch

import paper_2512_02541_b200 as P
from oracle import avggt_oracle as orc
from paper_2512_02541_b200 import inputs

pytestmark = pytest.mark.gpu

MAX_ABS_TOL = 2e-2
MEAN_ABS_TOL = 2e-3


def _cfgs(wl):
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                           diag=wl.diag, mean_fill=wl.mean_fill, keep_first_frame=bool(wl.keep_first_frame))
    ocfg = orc.SGAConfig(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                         diag=bool(wl.diag), mean_fill=wl.mean_fill, keep_first_frame=bool(wl.keep_first_frame))
    return params, ocfg


def _host(t):
    """bf16 device tensor -> float32 numpy (exact)."""
    return t.float().cpu().numpy()


def _run_gpu(wl, seed=0, want_lse=False):
    params, ocfg = _cfgs(wl)
    Q, K, V = inputs.make_qkv(wl, seed=seed, device="cuda")
    layer = P.SubsampledGlobalAttention(params, want_lse=want_lse)
    # poison the outputs so that unwritten rows show up
    O = torch.full_like(Q, float("nan"))
    layer.Kc.fill_(float("nan")); layer.Vc.fill_(float("nan")); layer.idx.fill_(-1)
    layer.forward(Q, K, V, out=O)
    layer.check_status()
    return params, ocfg, layer, Q, K, V, O


def _check_build(ocfg, layer, K, V):
    Kh, Vh = _host(K), _host(V)
    Kc, Vc, idx, kmean, vmean = orc.build_kv(ocfg, Kh, Vh)
    assert layer.M == len(idx)
    np.testing.assert_array_equal(layer.idx.cpu().numpy(), idx)
    # head-major [H, M, d] on the device; bf16 values are exact in fp32/fp64
    np.testing.assert_array_equal(_host(layer.Kc).transpose(1, 0, 2).astype(np.float64), Kc)
    np.testing.assert_array_equal(_host(layer.Vc).transpose(1, 0, 2).astype(np.float64), Vc)
    if ocfg.mean_fill != 0 and kmean is not None:
        for got, want, src in ((layer.kmean, kmean, Kh), (layer.vmean, vmean, Vh)):
            scale = max(float(np.abs(src).mean()), 1e-6)     # size of the summands
            assert np.abs(got.cpu().numpy().astype(np.float64) - want).max() <= 1e-5 * scale
    return Kh, Vh


def _stratified_rows(wl, ocfg, n_rows):
    """Sample of query rows for the full-size checks: ``inputs.sample_rows`` (sequence ends, tile-boundary
    classes, tail, random rows) plus, for the first, the last and five frames in between, one special
    token, one retained patch and one dropped patch, so that every kind of row (and with it every
    combination of the diagonal and mean terms) is met in frame 0 and well inside the sequence."""
    L = wl.tokens_per_frame
    rng = np.random.default_rng(5)
    frames = sorted({0, wl.n_frames - 1, *rng.integers(0, wl.n_frames, 5).tolist(), wl.n_frames // 2})
    must = []
    for f in frames:
        kept = orc.kept_slot_mask(ocfg, f)
        special = np.arange(L) < wl.n_special
        for members in (np.flatnonzero(special), np.flatnonzero(kept & ~special), np.flatnonzero(~kept)):
            if len(members):
                must.append(f * L + int(rng.choice(members)))
    return inputs.sample_rows(wl, n_rows, must_include=must).numpy()


def _check_attn(ocfg, Q, Kh, Vh, O, rows=None, lse=None):
    Qh = _host(Q)
    if rows is None:
        rows = np.arange(ocfg.n_tokens)
    want, want_lse = orc.global_attn_blocked(ocfg, Qh, Kh, Vh, rows, return_lse=True)
    got = O[torch.as_tensor(rows, device=O.device)].float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all(), "unwritten or non-finite output rows"
    err = np.abs(got - want)
    assert err.max() <= MAX_ABS_TOL, f"max-abs {err.max():.4g}"
    assert err.mean() <= MEAN_ABS_TOL, f"mean-abs {err.mean():.4g}"
    if lse is not None:
        got_lse = lse[torch.as_tensor(rows, device=lse.device)].cpu().numpy().astype(np.float64)
        assert np.abs(got_lse - want_lse).max() <= 2e-3
    return err.max(), err.mean()


def test_tiny_config_all_rows():
    """N=4, 16x16 grid, s=2, diagonal + mean-fill: every row against the oracle."""
    wl = inputs.WORKLOADS["tiny_n4_g16_s2"]
    params, ocfg, layer, Q, K, V, O = _run_gpu(wl, want_lse=True)
    assert (layer.M, layer.n_dropped) == (532, 512)
    Kh, Vh = _check_build(ocfg, layer, K, V)
    _check_attn(ocfg, Q, Kh, Vh, O, lse=layer.lse)


SMALL = inputs.Workload("small", 3, 7, 9, 5, 4, 64, 4, 1, 2, "iid")


@pytest.mark.parametrize("sigma", (1, 2, 4, 6, 9))
@pytest.mark.parametrize("diag,mean_fill", [(0, 0), (1, 0), (0, 2), (1, 2), (1, 1)])
def test_switches_and_factors(sigma, diag, mean_fill):
    wl = SMALL.with_(sigma=sigma, diag=diag, mean_fill=mean_fill)
    params, ocfg, layer, Q, K, V, O = _run_gpu(wl, seed=sigma, want_lse=True)
    Kh, Vh = _check_build(ocfg, layer, K, V)
    _check_attn(ocfg, Q, Kh, Vh, O, lse=layer.lse)


@pytest.mark.parametrize("n_frames,grid", [
    (1, (2, 61)),     # 127 tokens: one partial query tile
    (1, (3, 41)),     # 128 tokens exactly
    (1, (4, 31)),     # 129 tokens: a one-row tail tile
    (3, (10, 17)),    # 525 tokens, compact length with a ragged tail
    (7, (16, 16)),    # 1827 tokens
    (2, (1, 1)),      # grid smaller than every stride: nothing is dropped
    (5, (37, 37)),    # the VGGT patch grid
])
@pytest.mark.parametrize("sigma", (2, 9))
def test_ragged_sizes(n_frames, grid, sigma):
    wl = inputs.Workload("ragged", n_frames, grid[0], grid[1], 5, 2, 64, sigma, 1, 2, "iid")
    params, ocfg, layer, Q, K, V, O = _run_gpu(wl, seed=7)
    Kh, Vh = _check_build(ocfg, layer, K, V)
    _check_attn(ocfg, Q, Kh, Vh, O)


def test_no_special_tokens_and_keep_first_frame():
    wl = inputs.Workload("nospecial", 3, 9, 8, 0, 2, 64, 6, 1, 2, "iid")
    params, ocfg, layer, Q, K, V, O = _run_gpu(wl, seed=3)
    Kh, Vh = _check_build(ocfg, layer, K, V)
    _check_attn(ocfg, Q, Kh, Vh, O)
    wl = inputs.Workload("kff", 4, 9, 8, 5, 2, 64, 4, 1, 2, "iid", keep_first_frame=1)
    params, ocfg, layer, Q, K, V, O = _run_gpu(wl, seed=4)
    Kh, Vh = _check_build(ocfg, layer, K, V)
    _check_attn(ocfg, Q, Kh, Vh, O)


def test_many_heads_and_odd_head_count():
    for H in (1, 3, 16, 32):
        wl = inputs.Workload("heads", 2, 6, 6, 5, H, 64, 4, 1, 2, "iid")
        params, ocfg, layer, Q, K, V, O = _run_gpu(wl, seed=H)
        Kh, Vh = _check_build(ocfg, layer, K, V)
        _check_attn(ocfg, Q, Kh, Vh, O)


def test_large_logits_and_dominant_diagonal():
    """Self logits far above the rest (the structure the paper reports for middle layers)."""
    wl = inputs.Workload("proj_small", 6, 12, 12, 5, 16, 64, 4, 1, 2, "proj")
    params, ocfg, layer, Q, K, V, O = _run_gpu(wl, seed=11)
    Kh, Vh = _check_build(ocfg, layer, K, V)
    _check_attn(ocfg, Q, Kh, Vh, O)


def test_vggt_100_frames_sampled_rows():
    """The 100-frame benchmark configuration (37x37 grid, s=4) in the launch configuration
    bench.py times, checked on a stratified sample of 2048 rows (the oracle's blocked form:
    one matrix product per head over the sampled rows, the arithmetic per row unchanged)."""
    wl = inputs.WORKLOADS["vggt_n100_s4"]
    params, ocfg, layer, Q, K, V, O = _run_gpu(wl)
    assert (layer.M, layer.n_dropped) == (36600, 100800)
    Kh, Vh = _check_build(ocfg, layer, K, V)
    rows = _stratified_rows(wl, ocfg, 2048)
    _check_attn(ocfg, Q, Kh, Vh, O, rows=rows)
    # a handful of the same rows through the oracle's row-by-row form as well
    few = rows[:: max(1, len(rows) // 12)]
    want = orc.global_attn(ocfg, _host(Q), Kh, Vh, rows=few)
    got = O[torch.as_tensor(few, device=O.device)].float().cpu().numpy().astype(np.float64)
    assert np.abs(got - want).max() <= MAX_ABS_TOL
    # properties that hold at any size: every row written and finite
    assert torch.isfinite(O.float()).all()


@pytest.mark.parametrize("name,n_rows", [
    ("vggt_n300_s6", 512),    # 412,200 queries x 75,600 compact keys
    ("vggt_n800_s9", 512),    # 1,099,200 queries x 139,200 compact keys: the long-context case bench.py times
    ("vggt_n333_s1", 160),    # dense layer (both switches off), 457,542 x 457,542
    ("vggt_n333_s2", 256),    # the factor sweep at 333 frames
    ("vggt_n333_s4", 512),
    ("vggt_n333_s6", 512),
    ("vggt_n333_s9", 512),
])
def test_full_size_configs_sampled_rows(name, n_rows):
    """Every larger benchmark configuration at full size, in the launch configuration bench.py times:
    compaction checked in full against the oracle, attention on a stratified sample of rows
    (the oracle's blocked form over the sample), and every output row finite."""
    wl = inputs.WORKLOADS[name]
    params, ocfg, layer, Q, K, V, O = _run_gpu(wl)
    Kh, Vh = _check_build(ocfg, layer, K, V)
    rows = _stratified_rows(wl, ocfg, n_rows)
    _check_attn(ocfg, Q, Kh, Vh, O, rows=rows)
    assert torch.isfinite(O.float()).all()
    del Q, K, V, O, layer
    torch.cuda.empty_cache()


def test_results_are_deterministic():
    wl = inputs.Workload("det", 5, 16, 16, 5, 4, 64, 4, 1, 2, "iid")
    params, _ = _cfgs(wl)
    Q, K, V = inputs.make_qkv(wl, seed=1, device="cuda")
    layer = P.SubsampledGlobalAttention(params)
    O1 = layer.forward(Q, K, V).clone()
    km1 = layer.kmean.clone()
    O2 = layer.forward(Q, K, V)
    torch.cuda.synchronize()
    assert torch.equal(O1, O2) and torch.equal(km1, layer.kmean)


def test_argument_errors_do_not_launch():
    params, _ = _cfgs(SMALL)
    Q, K, V = inputs.make_qkv(SMALL, seed=0, device="cuda")
    layer = P.SubsampledGlobalAttention(params)
    with pytest.raises(P.AvggtError) as ei:      # workspace too small
        P.avggt_build_kv(params, K, V, layer.Kc, layer.Vc, layer.idx, layer.kmean, layer.vmean, layer.build_ws, 8)
    assert ei.value.code == -3
    with pytest.raises(P.AvggtError) as ei:      # misaligned pointer
        P.avggt_build_kv(params, K.data_ptr() + 2, V, layer.Kc, layer.Vc, layer.idx, layer.kmean, layer.vmean,
                         layer.build_ws, layer.build_ws.numel())
    assert ei.value.code == -4
    with pytest.raises(P.AvggtError) as ei:      # diag needs K and V
        P.avggt_global_attn(params, Q, None, None, layer.Kc, layer.Vc, layer.kmean, layer.vmean, Q.clone(), None,
                            layer.attn_ws, layer.attn_ws.numel())
    assert ei.value.code == -1
    torch.cuda.synchronize()


def _random_workloads(n, seed=2024):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        out.append(inputs.Workload(
            f"fuzz{i}", int(rng.integers(1, 7)), int(rng.integers(1, 24)), int(rng.integers(1, 24)),
            int(rng.integers(0, 7)), int(rng.choice([1, 2, 3, 5, 8, 16, 32])), 64, int(rng.choice([1, 2, 4, 6, 9])),
            int(rng.integers(0, 2)), int(rng.integers(0, 3)), str(rng.choice(["iid", "proj"])),
            keep_first_frame=int(rng.integers(0, 2))))
    return out


@pytest.mark.parametrize("wl", _random_workloads(16), ids=lambda w: f"{w.name}-N{w.n_frames}-g{w.grid_h}x{w.grid_w}-s{w.n_special}-H{w.n_heads}-sig{w.sigma}-d{w.diag}-m{w.mean_fill}-k{w.keep_first_frame}")
def test_seeded_random_shapes(wl):
    """Sixteen seeded draws over frames, grid, special tokens, heads, factor, switches, value recipe and
    the first-frame flag: compaction exact, attention and log-sum-exp within tolerance on every row."""
    params, ocfg, layer, Q, K, V, O = _run_gpu(wl, seed=17, want_lse=True)
    Kh, Vh = _check_build(ocfg, layer, K, V)
    _check_attn(ocfg, Q, Kh, Vh, O, lse=layer.lse)


@pytest.mark.parametrize("scale", (0.05, 0.3))
def test_caller_given_softmax_scale(scale):
    """A softmax scale other than 1/sqrt(d), in both the global and the frame entry points."""
    wl = inputs.Workload("scale", 3, 9, 9, 5, 4, 64, 4, 1, 2, "iid")
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                           softmax_scale=scale)
    ocfg = orc.SGAConfig(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                         softmax_scale=scale)
    Q, K, V = inputs.make_qkv(wl, seed=12, device="cuda")
    layer = P.SubsampledGlobalAttention(params, want_lse=True)
    O = layer.forward(Q, K, V)
    layer.check_status()
    Kh, Vh = _host(K), _host(V)
    _check_attn(ocfg, Q, Kh, Vh, O, lse=layer.lse)
    Of = layer.frame_attend(Q, K, V)
    layer.check_status()
    want = orc.frame_attn(ocfg, _host(Q), Kh, Vh)
    err = np.abs(Of.float().cpu().numpy().astype(np.float64) - want)
    assert err.max() <= MAX_ABS_TOL and err.mean() <= MEAN_ABS_TOL


def test_extreme_values_stay_finite():
    """Logits of a few hundred in magnitude with alternating sign between key tiles: the reference maximum
    jumps late and far, the accumulator is rescaled by tiny factors, nothing overflows."""
    wl = inputs.Workload("extreme", 4, 12, 12, 5, 2, 64, 2, 1, 2, "iid")
    params, ocfg = _cfgs(wl)
    Q, K, V = inputs.make_qkv(wl, seed=13, device="cuda")
    K = (K.float() * 6.0).bfloat16()                      # scale * q.k of the order of +-150
    L = wl.tokens_per_frame
    K[2 * L:] = (K[2 * L:].float() * 2.0).bfloat16()      # later frames (later key tiles) reach further out
    layer = P.SubsampledGlobalAttention(params, want_lse=True)
    O = layer.forward(Q, K, V)
    layer.check_status()
    assert torch.isfinite(O.float()).all() and torch.isfinite(layer.lse).all()
    Kh, Vh = _host(K), _host(V)
    _check_attn(ocfg, Q, Kh, Vh, O, lse=None)


def test_host_buffer_forward_matches_the_device_forward():
    """forward_host (K/V first, Q in groups of frames on a copy stream, outputs leaving on another) gives the very
    bits of forward on resident tensors, for a frame count that does not divide into the groups, with and without
    the uncompressed first frame; also for calls that follow one another without a wait."""
    for kff in (0, 1):
        wl = inputs.Workload("host", 11, 12, 13, 5, 4, 64, 4, 1, 2, "proj", keep_first_frame=kff)
        params, ocfg = _cfgs(wl)
        Q, K, V = inputs.make_qkv(wl, seed=21, device="cuda")
        layer = P.SubsampledGlobalAttention(params)
        O = layer.forward(Q, K, V).clone()
        layer.check_status()
        hQ, hK, hV = (t.cpu().pin_memory() for t in (Q, K, V))
        hO = torch.full_like(hQ, float("nan")).pin_memory()
        for n_chunks in (1, 4, 50):
            hO.fill_(float("nan"))
            layer.forward_host(hQ, hK, hV, hO, n_chunks=n_chunks)
            layer.check_status()
            assert torch.equal(hO, O.cpu()), n_chunks
        # three calls in a row without waiting in between, on two different inputs: the K and V of a call travel
        # (to the other of the two device buffers) while the attention of the call before runs
        Q2, K2, V2 = inputs.make_qkv(wl, seed=22, device="cuda")
        O2 = layer.forward(Q2, K2, V2).clone()
        layer.check_status()
        hQ2, hK2, hV2 = (t.cpu().pin_memory() for t in (Q2, K2, V2))
        outs = [torch.full_like(hQ, float("nan")).pin_memory() for _ in range(3)]
        layer.forward_host(hQ, hK, hV, outs[0], n_chunks=4)
        layer.forward_host(hQ2, hK2, hV2, outs[1], n_chunks=4)
        layer.forward_host(hQ, hK, hV, outs[2], n_chunks=4)
        layer.check_status()
        assert torch.equal(outs[0], O.cpu()) and torch.equal(outs[1], O2.cpu()) and torch.equal(outs[2], O.cpu())
