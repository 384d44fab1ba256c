"""Pins of the fp64 oracle against things other than itself.

Every check here compares ``oracle/avggt_oracle.py`` with something the paper
or the mathematics fixes: a library routine in the special case that reduces to
it (dense attention), an independently written brute force (the "filled
matrix"), closed forms, invariants, counts, and the FLOP figures the paper
prints.  None of them needs a GPU.
"""

import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import avggt_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SIGMAS = (1, 2, 4, 6, 9)


def _rand_qkv(cfg, seed, q_gain=1.5):
    rng = np.random.default_rng(seed)
    shape = (cfg.n_tokens, cfg.n_heads, cfg.head_dim)
    return (q_gain * rng.standard_normal(shape), rng.standard_normal(shape), rng.standard_normal(shape))


def _tiny(sigma, diag=True, mean_fill=2, **kw):
    base = dict(n_frames=2, grid_h=4, grid_w=5, n_special=2, n_heads=2, head_dim=8,
                sigma=sigma, diag=diag, mean_fill=mean_fill)
    base.update(kw)
    return orc.SGAConfig(**base)


# --------------------------------------------------------------------------
# independent brute force: the dense N_q x N_q problem with dropped columns
# filled by the mean pair and the diagonal restored, then a plain row softmax
# --------------------------------------------------------------------------

def _dropped_by_slicing(cfg):
    """Dropped-token mask built by numpy strided slicing (not by the oracle's
    per-slot modulo rule)."""
    s_h, s_w = {1: (1, 1), 2: (1, 2), 4: (2, 2), 6: (2, 3), 9: (3, 3)}[cfg.sigma]
    L = cfg.n_special + cfg.grid_h * cfg.grid_w
    out = np.zeros((cfg.n_frames, L), dtype=bool)
    for f in range(cfg.n_frames):
        grid = np.ones((cfg.grid_h, cfg.grid_w), dtype=bool)
        grid[::s_h, ::s_w] = False
        if cfg.keep_first_frame and f == 0:
            grid[:] = False
        out[f, cfg.n_special:] = grid.reshape(-1)
    return out.reshape(-1)


def _brute_force(cfg, Q, K, V, D=None):
    n_tok, H, d = Q.shape
    scale = 1.0 / math.sqrt(d) if cfg.softmax_scale <= 0 else cfg.softmax_scale
    if D is None:
        D = _dropped_by_slicing(cfg)
    O = np.zeros((n_tok, H, d))
    for h in range(H):
        if D.any():
            kbar = np.sum(K[D, h, :], axis=0) / D.sum()
            vbar = np.sum(V[D, h, :], axis=0) / D.sum()
        for i in range(n_tok):
            keys, vals = [], []
            for j in range(n_tok):
                if not D[j]:
                    keys.append(K[j, h]); vals.append(V[j, h])            # retained column
                elif cfg.diag and j == i:
                    keys.append(K[j, h]); vals.append(V[j, h])            # restored diagonal
                elif cfg.mean_fill == 2:
                    keys.append(kbar); vals.append(vbar)                  # filled column
            if cfg.mean_fill == 1:
                n_rest = int(D.sum()) - (1 if (cfg.diag and D[i]) else 0)
                if n_rest > 0:
                    keys.append(kbar); vals.append(vbar)                  # one unit-weight column
            logits = [scale * sum(Q[i, h, t] * k[t] for t in range(d)) for k in keys]
            mx = max(logits)
            e = [math.exp(l - mx) for l in logits]
            z = sum(e)
            for w, v in zip(e, vals):
                O[i, h] += (w / z) * v
    return O


@pytest.mark.parametrize("sigma", SIGMAS)
@pytest.mark.parametrize("diag,mean_fill", list(itertools.product((False, True), (0, 1, 2))))
def test_matches_filled_matrix_brute_force(sigma, diag, mean_fill):
    cfg = _tiny(sigma, diag, mean_fill)
    Q, K, V = _rand_qkv(cfg, seed=100 * sigma + 10 * int(diag) + mean_fill)
    np.testing.assert_allclose(orc.global_attn(cfg, Q, K, V), _brute_force(cfg, Q, K, V), rtol=0, atol=1e-12)


def test_brute_force_keep_first_frame():
    cfg = _tiny(4, True, 2, keep_first_frame=True, n_frames=3)
    Q, K, V = _rand_qkv(cfg, seed=5)
    np.testing.assert_allclose(orc.global_attn(cfg, Q, K, V), _brute_force(cfg, Q, K, V), rtol=0, atol=1e-12)


# --------------------------------------------------------------------------
# special case that reduces to a library routine: sigma = 1 is dense attention
# --------------------------------------------------------------------------

@pytest.mark.parametrize("diag,mean_fill", [(False, 0), (True, 2), (True, 1)])
def test_sigma1_is_dense_sdpa(diag, mean_fill):
    cfg = orc.SGAConfig(3, 5, 7, 5, 4, 16, sigma=1, diag=diag, mean_fill=mean_fill)
    Q, K, V = _rand_qkv(cfg, seed=3)
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2)[None] for a in (Q, K, V))   # [1,H,T,d]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(orc.global_attn(cfg, Q, K, V), ref, rtol=0, atol=1e-12)


def test_grid_not_larger_than_stride_is_dense():
    # a 1 x 1 patch grid has nothing to drop at any factor
    cfg = orc.SGAConfig(4, 1, 1, 2, 2, 8, sigma=9)
    Q, K, V = _rand_qkv(cfg, seed=4)
    dense = orc.global_attn(orc.SGAConfig(4, 1, 1, 2, 2, 8, sigma=1, diag=False, mean_fill=0), Q, K, V)
    np.testing.assert_allclose(orc.global_attn(cfg, Q, K, V), dense, rtol=0, atol=1e-13)


# --------------------------------------------------------------------------
# closed forms and invariants
# --------------------------------------------------------------------------

@pytest.mark.parametrize("sigma", (2, 4, 6, 9))
@pytest.mark.parametrize("diag", (False, True))
def test_identical_dropped_rows_make_fill_exact(sigma, diag):
    """If every dropped K/V row is the same vector, filling the dropped columns
    with their mean changes nothing: count-weighted mean-fill equals dense."""
    cfg = _tiny(sigma, diag, 2, n_frames=3)
    Q, K, V = _rand_qkv(cfg, seed=7)
    D = orc.dropped_token_mask(cfg)
    K[D] = K[D][0]
    V[D] = V[D][0]
    dense = orc.global_attn(_tiny(1, False, 0, n_frames=3), Q, K, V)
    np.testing.assert_allclose(orc.global_attn(cfg, Q, K, V), dense, rtol=0, atol=1e-12)


@pytest.mark.parametrize("mean_fill", (0, 1, 2))
def test_weights_are_jointly_normalised(mean_fill):
    cfg = _tiny(4, True, mean_fill)
    Q, K, V = _rand_qkv(cfg, seed=11)
    _, weights = orc.global_attn(cfg, Q, K, V, return_weights=True)
    D = orc.dropped_token_mask(cfg)
    for i, w in enumerate(weights):
        total = w["subset"].sum(axis=1)
        assert (w["diag"] is not None) == bool(D[i])           # diagonal only where the own column is not in S
        assert (w["mean"] is not None) == (mean_fill != 0)
        for part in (w["diag"], w["mean"]):
            if part is not None:
                total = total + part
                assert np.all(part > 0)
        np.testing.assert_allclose(total, 1.0, rtol=0, atol=1e-13)
    # all-ones values must come back as ones whatever the weights are
    O = orc.global_attn(cfg, Q, K, np.ones_like(V))
    np.testing.assert_allclose(O, 1.0, rtol=0, atol=1e-13)


def test_mean_weight_modes_differ_by_count():
    """mode 2 = mode 1 with the mean logit raised by ln(count): check on the
    ratio of mean weight to a retained column's weight."""
    cfg1, cfg2 = _tiny(4, True, 1), _tiny(4, True, 2)
    Q, K, V = _rand_qkv(cfg1, seed=13)
    _, w1 = orc.global_attn(cfg1, Q, K, V, return_weights=True)
    _, w2 = orc.global_attn(cfg2, Q, K, V, return_weights=True)
    D = orc.dropped_token_mask(cfg1)
    n_d = int(D.sum())
    for i in range(cfg1.n_tokens):
        count = n_d - (1 if D[i] else 0)
        r1 = w1[i]["mean"] / w1[i]["subset"][:, 0]
        r2 = w2[i]["mean"] / w2[i]["subset"][:, 0]
        np.testing.assert_allclose(r2, count * r1, rtol=1e-12)


@pytest.mark.parametrize("sigma", (2, 9))
def test_shift_invariances(sigma):
    cfg = _tiny(sigma, True, 2)
    Q, K, V = _rand_qkv(cfg, seed=17)
    rng = np.random.default_rng(1)
    base = orc.global_attn(cfg, Q, K, V)
    ck = rng.standard_normal((cfg.n_heads, cfg.head_dim))
    cv = rng.standard_normal((cfg.n_heads, cfg.head_dim))
    # a constant added to every key shifts all logits of a row equally
    np.testing.assert_allclose(orc.global_attn(cfg, Q, K + ck, V), base, rtol=0, atol=1e-11)
    # a constant added to every value is passed through by the normalised weights
    np.testing.assert_allclose(orc.global_attn(cfg, Q, K, V + cv), base + cv, rtol=0, atol=1e-11)


def test_frame_permutation_equivariance():
    cfg = _tiny(4, True, 2, n_frames=4)
    Q, K, V = _rand_qkv(cfg, seed=19)
    L = cfg.tokens_per_frame
    perm = np.array([2, 0, 3, 1])
    tok = (perm[:, None] * L + np.arange(L)[None, :]).reshape(-1)
    base = orc.global_attn(cfg, Q, K, V)
    np.testing.assert_allclose(orc.global_attn(cfg, Q[tok], K[tok], V[tok]), base[tok], rtol=0, atol=1e-12)


def test_diagonal_dominates_when_self_logit_is_huge():
    """A dropped query whose own key is far larger than every other logit must
    return (almost) its own value: catches a dropped or misindexed diagonal."""
    cfg = _tiny(4, True, 2)
    Q, K, V = _rand_qkv(cfg, seed=23, q_gain=1.0)
    D = np.flatnonzero(orc.dropped_token_mask(cfg))
    i = int(D[3])
    K[i] = 40.0 * Q[i] / np.linalg.norm(Q[i], axis=-1, keepdims=True) ** 2 * math.sqrt(cfg.head_dim)
    O = orc.global_attn(cfg, Q, K, V, rows=[i])
    np.testing.assert_allclose(O[0], V[i], rtol=0, atol=1e-8)
    off = orc.global_attn(_tiny(4, False, 0), Q, K, V, rows=[i])
    assert np.abs(off[0] - V[i]).max() > 1e-2


# --------------------------------------------------------------------------
# index set and counts
# --------------------------------------------------------------------------

@pytest.mark.parametrize("sigma", SIGMAS)
@pytest.mark.parametrize("grid", [(37, 37), (16, 16), (28, 37), (3, 2), (1, 1)])
@pytest.mark.parametrize("kff", (False, True))
def test_index_set_and_counts(sigma, grid, kff):
    h, w = grid
    cfg = orc.SGAConfig(3, h, w, 5, 2, 8, sigma=sigma, keep_first_frame=kff)
    s_h, s_w = orc.strides_for_sigma(sigma)
    assert s_h * s_w == sigma and s_h <= s_w
    idx = orc.build_index(cfg)
    expect = np.flatnonzero(~_dropped_by_slicing(cfg))
    assert idx.dtype == np.int32
    np.testing.assert_array_equal(idx, expect)
    assert np.all(np.diff(idx) > 0)
    kept_per_frame = math.ceil(h / s_h) * math.ceil(w / s_w)
    M = 3 * (5 + kept_per_frame) + (h * w - kept_per_frame if kff else 0)
    assert orc.kv_count(cfg) == (M, 3 * (5 + h * w) - M)


def test_unknown_sigma_rejected():
    with pytest.raises(ValueError):
        orc.strides_for_sigma(3)


def test_factor_two_keeps_about_half():
    # supplementary: a factor of 2 keeps about 50% of the patch tokens
    cfg = orc.SGAConfig(1, 37, 37, 5, 1, 8, sigma=2)
    kept = orc.kept_slot_mask(cfg, 0)[5:].mean()
    assert abs(kept - 0.5) < 0.02


def test_printed_flops_pin_window_rule():
    """The paper's whole-model FLOPs at 800 frames differ between subsampling
    factors only through the number of retained keys M in the 15 subsampled
    global layers (24 global blocks, the first 9 converted to frame attention):
    delta = 15 * 2 * (N*L) * C * (M_a - M_b) multiply-adds.  The printed
    differences agree to the printed precision only if partial edge windows
    keep their first token and frame 0 is left uncompressed (VGGT)."""
    printed = {}
    with open(os.path.join(GOLDEN, "flops_7scenes_800_vggt.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                s, v = line.split()
                printed[int(s)] = float(v)
    N, gh, gw, C, layers = 800, 28, 37, 1024, 15          # 392 x 518 px at patch 14
    n_tok = N * (gh * gw + 5)

    def m_of(sigma, kff=True):
        return orc.kv_count(orc.SGAConfig(N, gh, gw, 5, 16, 64, sigma=sigma, keep_first_frame=kff))[0]

    for a, b in ((2, 4), (4, 6), (6, 9)):
        delta = layers * 2 * n_tok * C * (m_of(a) - m_of(b)) / 1e15
        assert abs(delta - (printed[a] - printed[b])) <= 0.0015, (a, b, delta)
    # the floor rule (dropping partial windows) misses by far more than the rounding
    floor_m = {2: 28 * 18, 4: 14 * 18, 9: 9 * 12}
    bad = layers * 2 * n_tok * C * 799 * (floor_m[2] - floor_m[4]) / 1e15
    assert abs(bad - (printed[2] - printed[4])) > 0.1


# --------------------------------------------------------------------------
# compaction and the blocked evaluation
# --------------------------------------------------------------------------

def test_build_kv_gathers_and_averages():
    cfg = _tiny(6, True, 2, n_frames=3)
    _, K, V = _rand_qkv(cfg, seed=29)
    Kc, Vc, idx, kmean, vmean = orc.build_kv(cfg, K, V)
    D = _dropped_by_slicing(cfg)
    for m, t in enumerate(idx):
        assert not D[t]
        np.testing.assert_array_equal(Kc[m], K[t])
        np.testing.assert_array_equal(Vc[m], V[t])
    acc_k = np.zeros_like(K[0]); acc_v = np.zeros_like(V[0])
    for t in np.flatnonzero(D):
        acc_k += K[t]; acc_v += V[t]
    np.testing.assert_allclose(kmean, acc_k / D.sum(), rtol=0, atol=1e-14)
    np.testing.assert_allclose(vmean, acc_v / D.sum(), rtol=0, atol=1e-14)


@pytest.mark.parametrize("sigma,diag,mean_fill", [(1, False, 0), (2, True, 2), (4, True, 1), (9, False, 2), (6, True, 0)])
def test_blocked_equals_rowwise(sigma, diag, mean_fill):
    cfg = orc.SGAConfig(3, 7, 6, 5, 3, 16, sigma=sigma, diag=diag, mean_fill=mean_fill)
    Q, K, V = _rand_qkv(cfg, seed=31)
    rows = np.arange(0, cfg.n_tokens, 3)
    O_b, lse_b = orc.global_attn_blocked(cfg, Q, K, V, rows, return_lse=True)
    O_r, lse_r = orc.global_attn(cfg, Q, K, V, rows=rows, return_lse=True)
    np.testing.assert_allclose(O_b, O_r, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse_b, lse_r, rtol=0, atol=1e-12)
    # float32 inputs (how bf16 tensors reach the oracle) are widened, not computed in
    np.testing.assert_allclose(
        orc.global_attn_blocked(cfg, Q.astype(np.float32), K.astype(np.float32), V.astype(np.float32), rows),
        orc.global_attn(cfg, Q.astype(np.float32).astype(np.float64), K.astype(np.float32).astype(np.float64),
                        V.astype(np.float32).astype(np.float64), rows=rows), rtol=0, atol=1e-12)


def test_lse_is_log_of_summed_exponentials():
    """The normaliser against a direct enumeration of the present columns."""
    cfg = _tiny(4, True, 2)
    Q, K, V = _rand_qkv(cfg, seed=37)
    _, lse = orc.global_attn(cfg, Q, K, V, return_lse=True)
    D = _dropped_by_slicing(cfg)
    scale = 1.0 / math.sqrt(cfg.head_dim)
    for i in (0, 3, 9, cfg.n_tokens - 1):
        for h in range(cfg.n_heads):
            kbar = K[D, h].mean(axis=0)
            tot = sum(math.exp(scale * float(Q[i, h] @ K[j, h])) for j in range(cfg.n_tokens) if not D[j] or j == i)
            tot += (int(D.sum()) - int(D[i])) * math.exp(scale * float(Q[i, h] @ kbar))
            assert abs(lse[i, h] - math.log(tot)) < 1e-12


# --------------------------------------------------------------------------
# frame attention of converted early global blocks (Sec. 4.2)
# --------------------------------------------------------------------------

def test_frame_attn_is_per_frame_library_sdpa():
    """Skipping the (B, N L, C) rearrangement means N independent dense attentions: each frame
    against a library routine, in the (B N, L, C) layout the paper names."""
    cfg = orc.SGAConfig(4, 3, 5, 2, 3, 16, sigma=4)
    Q, K, V = _rand_qkv(cfg, seed=21)
    L, H, d = cfg.tokens_per_frame, cfg.n_heads, cfg.head_dim
    tq, tk, tv = (torch.from_numpy(a).reshape(cfg.n_frames, L, H, d).permute(0, 2, 1, 3) for a in (Q, K, V))   # [N,H,L,d]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).reshape(-1, H, d).numpy()
    got, lse = orc.frame_attn(cfg, Q, K, V, return_lse=True)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-12)
    # the normaliser against its definition, frame by frame
    logits = np.einsum("nlhd,nmhd->nhlm", Q.reshape(cfg.n_frames, L, H, d), K.reshape(cfg.n_frames, L, H, d)) / math.sqrt(d)
    want_lse = np.log(np.exp(logits).sum(axis=-1)).transpose(0, 2, 1).reshape(-1, H)
    np.testing.assert_allclose(lse, want_lse, rtol=0, atol=1e-12)


def test_frame_attn_equals_one_frame_global_attention():
    """With a single frame, global and frame attention are the same layer (the O((N L)^2) -> O(N L^2)
    statement at N = 1), and other frames' tokens cannot influence a frame's output."""
    cfg = orc.SGAConfig(3, 4, 4, 5, 2, 8, sigma=2)
    Q, K, V = _rand_qkv(cfg, seed=22)
    L = cfg.tokens_per_frame
    one = orc.SGAConfig(1, 4, 4, 5, 2, 8, sigma=1, diag=False, mean_fill=0)
    got = orc.frame_attn(cfg, Q, K, V)
    for f in range(cfg.n_frames):
        sl = slice(f * L, (f + 1) * L)
        np.testing.assert_allclose(got[sl], orc.global_attn(one, Q[sl], K[sl], V[sl]), rtol=0, atol=1e-12)
    K2, V2 = K.copy(), V.copy()
    K2[L:2 * L] += 5.0                       # disturb frame 1 only
    V2[L:2 * L] -= 3.0
    got2 = orc.frame_attn(cfg, Q, K2, V2)
    np.testing.assert_array_equal(got2[:L], got[:L])
    np.testing.assert_array_equal(got2[2 * L:], got[2 * L:])
    assert np.abs(got2[L:2 * L] - got[L:2 * L]).max() > 1e-3


def test_frame_attn_rows_and_switches():
    """A subset of rows gives the same rows; sigma, diag and mean_fill play no part."""
    a = orc.SGAConfig(3, 3, 4, 1, 2, 8, sigma=9, diag=True, mean_fill=2)
    b = orc.SGAConfig(3, 3, 4, 1, 2, 8, sigma=1, diag=False, mean_fill=0)
    Q, K, V = _rand_qkv(a, seed=23)
    full = orc.frame_attn(a, Q, K, V)
    rows = np.array([0, 12, 13, 25, 38])
    np.testing.assert_array_equal(orc.frame_attn(a, Q, K, V, rows=rows), full[rows])
    np.testing.assert_array_equal(orc.frame_attn(b, Q, K, V), full)


# --------------------------------------------------------------------------
# caller-chosen retained set (the supplement's alternative selectors)
# --------------------------------------------------------------------------

@pytest.mark.parametrize("sigma", (2, 6))
@pytest.mark.parametrize("diag,mean_fill", [(False, 0), (True, 0), (False, 2), (True, 2), (True, 1)])
def test_indexed_with_the_grid_subset_is_the_grid_layer(sigma, diag, mean_fill):
    cfg = _tiny(sigma, diag, mean_fill)
    Q, K, V = _rand_qkv(cfg, seed=31 + sigma)
    got, lse = orc.global_attn_indexed(cfg, orc.build_index(cfg), Q, K, V, return_lse=True)
    want, want_lse = orc.global_attn(cfg, Q, K, V, return_lse=True)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, want_lse, rtol=0, atol=1e-12)


@pytest.mark.parametrize("diag,mean_fill", list(itertools.product((False, True), (0, 1, 2))))
def test_indexed_random_subset_matches_filled_matrix_brute_force(diag, mean_fill):
    cfg = _tiny(4, diag, mean_fill)
    Q, K, V = _rand_qkv(cfg, seed=41 + 2 * int(diag) + mean_fill)
    rng = np.random.default_rng(7)
    idx = rng.permutation(cfg.n_tokens)[:17]              # unsorted on purpose; drops special tokens too
    D = np.ones(cfg.n_tokens, dtype=bool)
    D[idx] = False
    np.testing.assert_allclose(orc.global_attn_indexed(cfg, idx, Q, K, V), _brute_force(cfg, Q, K, V, D=D), rtol=0, atol=1e-12)


def test_indexed_keeping_everything_is_dense_sdpa():
    cfg = orc.SGAConfig(2, 3, 4, 1, 2, 8, sigma=9, diag=True, mean_fill=2)
    Q, K, V = _rand_qkv(cfg, seed=51)
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2)[None] for a in (Q, K, V))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(orc.global_attn_indexed(cfg, np.arange(cfg.n_tokens), Q, K, V), ref, rtol=0, atol=1e-12)



@pytest.mark.parametrize("mean_fill", (1, 2))
def test_indexed_with_nothing_retained_is_the_mean_value(mean_fill):
    """G2M (Sec. 5.4): all Keys/Values replaced by one mean pair.  Without the diagonal the softmax has a
    single column, so every output row is the plain mean of V over all tokens, whatever Q and K are."""
    cfg = _tiny(4, False, mean_fill)
    Q, K, V = _rand_qkv(cfg, seed=61)
    got, lse = orc.global_attn_indexed(cfg, np.zeros(0, dtype=np.int64), Q, K, V, return_lse=True)
    want = np.broadcast_to(V.mean(axis=0), got.shape)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    # one column of logit scale * q.kmean (+ ln N in fill mode): the normaliser is that logit itself
    lm = cfg.scale * np.einsum("nhd,hd->nh", Q, K.mean(axis=0)) + (math.log(cfg.n_tokens) if mean_fill == 2 else 0.0)
    np.testing.assert_allclose(lse, lm, rtol=0, atol=1e-10)


@pytest.mark.parametrize("mean_fill", (0, 1, 2))
def test_indexed_with_nothing_retained_and_the_diagonal_matches_filled_matrix_brute_force(mean_fill):
    cfg = _tiny(2, True, mean_fill)
    Q, K, V = _rand_qkv(cfg, seed=63)
    D = np.ones(cfg.n_tokens, dtype=bool)
    np.testing.assert_allclose(orc.global_attn_indexed(cfg, np.zeros(0, dtype=np.int64), Q, K, V),
                               _brute_force(cfg, Q, K, V, D=D), rtol=0, atol=1e-12)


# --------------------------------------------------------------------------
# projection with the compaction in its epilogue
# --------------------------------------------------------------------------

def test_round_to_bf16_matches_the_library_conversion():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38, 1e-40]]).astype(np.float32)
    want = torch.from_numpy(x).bfloat16().float().numpy()
    np.testing.assert_array_equal(orc.round_to_bf16(x).astype(np.float32), want)


def test_projection_with_identity_weights_is_the_plain_compaction():
    cfg = orc.SGAConfig(3, 4, 5, 2, 2, 8, sigma=4)
    rng = np.random.default_rng(5)
    C = cfg.n_heads * cfg.head_dim
    X = torch.from_numpy(rng.standard_normal((cfg.n_tokens, C))).bfloat16().double().numpy()      # on the bf16 grid already
    eye = np.eye(C)
    K_b, V_b, Kc, Vc, idx, kmean, vmean = orc.project_build_kv(cfg, X, eye, 2.0 * eye)
    Kc_w, Vc_w, idx_w, kmean_w, vmean_w = orc.build_kv(cfg, X.reshape(cfg.n_tokens, cfg.n_heads, cfg.head_dim),
                                                      2.0 * X.reshape(cfg.n_tokens, cfg.n_heads, cfg.head_dim))
    np.testing.assert_array_equal(idx, idx_w)
    np.testing.assert_array_equal(Kc, Kc_w)
    np.testing.assert_array_equal(Vc, Vc_w)
    np.testing.assert_allclose(kmean, kmean_w, rtol=0, atol=1e-13)
    np.testing.assert_allclose(vmean, vmean_w, rtol=0, atol=1e-13)


def test_projection_mean_is_the_projected_mean_of_the_dropped_tokens():
    """Linearity: the mean of the projected keys over D equals the projection of the mean token of D."""
    cfg = orc.SGAConfig(2, 5, 6, 3, 2, 8, sigma=6)
    rng = np.random.default_rng(6)
    C = 24
    X = rng.standard_normal((cfg.n_tokens, C))
    Wk, Wv = rng.standard_normal((16, C)), rng.standard_normal((16, C))
    bk, bv = rng.standard_normal(16), rng.standard_normal(16)
    K_b, V_b, Kc, Vc, idx, kmean, vmean = orc.project_build_kv(cfg, X, Wk, Wv, bk, bv)
    xbar = X[_dropped_by_slicing(cfg)].mean(axis=0)
    np.testing.assert_allclose(kmean.reshape(-1), Wk @ xbar + bk, rtol=0, atol=1e-12)
    np.testing.assert_allclose(vmean.reshape(-1), Wv @ xbar + bv, rtol=0, atol=1e-12)
    # the stored projections are the rounded ones, row by row what a plain loop gives
    i = 7
    want = np.array([sum(X[i, c] * Wk[o, c] for c in range(C)) + bk[o] for o in range(16)])
    np.testing.assert_array_equal(K_b[i].reshape(-1), orc.round_to_bf16(want))
    np.testing.assert_array_equal(Kc, K_b[idx])
