"""fp64 CPU oracle for Subsampling Global Attention (SGA), Sec. 4.3 of the AVGGT paper.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
library's CUDA path must compute.  It is imported by the tests, by the smoke
check and by the benchmark's CPU-baseline leg and by nothing else; the product
never routes through it.  It shares no code with the CUDA path and imports
nothing from the package.

What it computes (all in float64, inputs are the caller's arrays widened
exactly):

  * the K/V index subset S of Sec. 4.3 "Subsampling Strategy": all special
    tokens of every frame plus the first patch token of every s_h x s_w window
    of the n_h x n_w patch grid, sigma = s_h * s_w with the printed
    sigma -> (s_h, s_w) table;
  * the compacted K_S, V_S and the mean Key/Value pair over the dropped patch
    tokens (Sec. 4.3 "Enhanced Subsampling with Diagonal Preservation");
  * attention of every query over three disjoint components under one softmax
    (same paragraph and the caption of the SGA figure): (i) the retained
    subset S, (ii) the query's own diagonal column, (iii) one mean component
    standing for all dropped patches.

The algorithm is an approximation of dense attention, so the steps below are
taken in the paper's order; there is no tiling, fusion or reordering.

Readings where the paper is silent (each is pinned by a test, except the
first, which the paper does not decide):

  * weight of the mean component.  ``mean_fill == 2`` (primary): every dropped
    column is *filled* with the mean pair, i.e. the single mean column enters
    the softmax with multiplicity c_i = number of columns it stands for
    (logit + ln c_i).  ``mean_fill == 1``: the mean pair is one extra column
    of unit weight.  PARITY UNPINNED between the two modes: the paper's text
    does not choose.  Within mode 2 the result is pinned by a filled-matrix
    brute force and by the closed form "all dropped rows equal => dense".
  * partial edge windows keep their first token (strided slice [::s_h, ::s_w]).
  * "disjoint ... without redundancy": the diagonal term exists only for
    queries whose own column is not already in S, and for such a query the
    mean column stands for the *other* |D| - 1 dropped columns.
  * the mean pair itself is the plain mean over all dropped patch tokens of
    all frames, per head (it is not leave-one-out).
  * |D| = 0 (sigma = 1, or strides >= grid): no mean and no diagonal term;
    the layer is dense softmax attention.
  * softmax scale 1/sqrt(d) unless given; no mask, bias or dropout.
  * token order in a frame: special tokens in slots [0, n_special), then the
    patch grid row-major.  Compact order is ascending global token index.
  * keep_first_frame (VGGT variant of Sec. 4.3): frame 0 keeps every patch.
"""

from dataclasses import dataclass
import math

import numpy as np

# Sec. 4.3, "Subsampling Strategy": the printed sigma -> (s_h, s_w) table.
# sigma = 1 is the un-subsampled (dense) layer.
_SIGMA_TABLE = {1: (1, 1), 2: (1, 2), 4: (2, 2), 6: (2, 3), 9: (3, 3)}


@dataclass(frozen=True)
class SGAConfig:
    """Problem statement of Sec. 4.1 (notation) and Sec. 4.3."""

    n_frames: int            # N
    grid_h: int              # n_h
    grid_w: int              # n_w
    n_special: int           # camera + register tokens per frame
    n_heads: int             # H
    head_dim: int            # d
    sigma: int               # total subsampling factor
    diag: bool = True        # diagonal preservation
    mean_fill: int = 2       # 0 off | 1 unit weight | 2 count-weighted fill
    keep_first_frame: bool = False
    softmax_scale: float = 0.0   # <= 0 -> 1/sqrt(d)

    @property
    def tokens_per_frame(self):   # L = T + n_special
        return self.n_special + self.grid_h * self.grid_w

    @property
    def n_tokens(self):           # N * L
        return self.n_frames * self.tokens_per_frame

    @property
    def scale(self):
        return self.softmax_scale if self.softmax_scale > 0 else 1.0 / math.sqrt(self.head_dim)


def strides_for_sigma(sigma):
    """sigma -> (s_h, s_w), Sec. 4.3 'Subsampling Strategy'."""
    if sigma not in _SIGMA_TABLE:
        raise ValueError(f"sigma={sigma} is not one of {sorted(_SIGMA_TABLE)}")
    return _SIGMA_TABLE[sigma]


def kept_slot_mask(cfg, frame):
    """Boolean mask over the L token slots of one frame: True = slot is in S.

    Sec. 4.3: all special tokens are preserved; of the patch grid the first
    token of each s_h x s_w window is retained.
    """
    s_h, s_w = strides_for_sigma(cfg.sigma)
    L = cfg.tokens_per_frame
    mask = np.zeros(L, dtype=bool)
    for u in range(L):
        if u < cfg.n_special:
            mask[u] = True
            continue
        p = u - cfg.n_special
        r, c = divmod(p, cfg.grid_w)
        if cfg.keep_first_frame and frame == 0:
            mask[u] = True
        else:
            mask[u] = (r % s_h == 0) and (c % s_w == 0)
    return mask


def kept_token_mask(cfg):
    """Boolean mask over all N*L tokens: True = token is in S."""
    return np.concatenate([kept_slot_mask(cfg, f) for f in range(cfg.n_frames)])


def dropped_token_mask(cfg):
    """D: patch tokens that are not in S (special tokens are never dropped)."""
    return ~kept_token_mask(cfg)


def build_index(cfg):
    """idx[m] = global token index of the m-th compact key (ascending)."""
    return np.flatnonzero(kept_token_mask(cfg)).astype(np.int32)


def kv_count(cfg):
    """(M, |D|): number of compact keys and of dropped patch tokens."""
    kept = kept_token_mask(cfg)
    return int(kept.sum()), int((~kept).sum())


def build_kv(cfg, K, V):
    """Gather K_S, V_S and the mean pair over D.

    K, V: arrays [N*L, H, d] (any real dtype; every value that is used is
    widened to float64 before any arithmetic).
    Returns (Kc [M,H,d], Vc [M,H,d], idx [M] int32, kmean [H,d], vmean [H,d]).
    kmean/vmean are None when D is empty.
    """
    K = np.asarray(K)
    V = np.asarray(V)
    assert K.shape == (cfg.n_tokens, cfg.n_heads, cfg.head_dim) and V.shape == K.shape
    idx = build_index(cfg)
    dropped = dropped_token_mask(cfg)
    Kc = K[idx].astype(np.float64)
    Vc = V[idx].astype(np.float64)
    if dropped.any():
        kmean = K[dropped].mean(axis=0, dtype=np.float64)
        vmean = V[dropped].mean(axis=0, dtype=np.float64)
    else:
        kmean = vmean = None
    return Kc, Vc, idx, kmean, vmean


def global_attn(cfg, Q, K, V, rows=None, return_weights=False, return_lse=False):
    """Subsampled global attention for the query rows ``rows`` (default: all).

    Q, K, V: [N*L, H, d].  Returns O [len(rows), H, d] float64, and with
    ``return_weights`` also a list (one entry per row) of dicts with the
    softmax weights of the three components per head:
    {'subset': [H, M], 'diag': [H] or None, 'mean': [H] or None}; with
    ``return_lse`` also the natural-log normaliser ln(sum of exponentials of
    all present logits) as [len(rows), H].
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    H, d = cfg.n_heads, cfg.head_dim
    assert Q.shape == (cfg.n_tokens, H, d) and K.shape == Q.shape and V.shape == Q.shape
    scale = cfg.scale

    Kc, Vc, idx, kmean, vmean = build_kv(cfg, K, V)
    dropped = dropped_token_mask(cfg)
    n_dropped = int(dropped.sum())
    # [H, M, d] views so that one matmul per head serves as the "scores" step
    Kc_h = np.ascontiguousarray(Kc.transpose(1, 0, 2))
    Vc_h = np.ascontiguousarray(Vc.transpose(1, 0, 2))

    if rows is None:
        rows = np.arange(cfg.n_tokens)
    rows = np.asarray(rows, dtype=np.int64)
    O = np.empty((len(rows), H, d), dtype=np.float64)
    lse = np.empty((len(rows), H), dtype=np.float64)
    weights = [] if return_weights else None

    for out_i, i in enumerate(rows):
        q = Q[i]                                        # [H, d]
        # (i) retained subset S
        logit_s = scale * np.einsum("hd,hmd->hm", q, Kc_h)   # [H, M]
        # (ii) diagonal: only if the query's own column is not already in S
        has_diag = bool(cfg.diag) and bool(dropped[i])
        # (iii) mean component standing for the dropped columns that are not
        # represented otherwise: all of D, minus the diagonal one if present
        count = n_dropped - (1 if has_diag else 0)
        has_mean = cfg.mean_fill != 0 and count > 0
        parts = [logit_s]
        if has_diag:
            logit_d = scale * np.einsum("hd,hd->h", q, K[i])
            parts.append(logit_d[:, None])
        if has_mean:
            logit_m = scale * np.einsum("hd,hd->h", q, kmean)
            if cfg.mean_fill == 2:
                logit_m = logit_m + math.log(count)
            parts.append(logit_m[:, None])
        logits = np.concatenate(parts, axis=1)          # [H, M (+1) (+1)]
        # one shared softmax normalisation over all components
        mx = logits.max(axis=1, keepdims=True)
        p = np.exp(logits - mx)
        z = p.sum(axis=1, keepdims=True)
        p /= z
        lse[out_i] = (mx + np.log(z))[:, 0]
        M = logit_s.shape[1]
        o = np.einsum("hm,hmd->hd", p[:, :M], Vc_h)
        col = M
        w = {"subset": p[:, :M], "diag": None, "mean": None}
        if has_diag:
            o += p[:, col:col + 1] * V[i]
            w["diag"] = p[:, col]
            col += 1
        if has_mean:
            o += p[:, col:col + 1] * vmean
            w["mean"] = p[:, col]
        O[out_i] = o
        if return_weights:
            weights.append(w)
    out = (O,)
    if return_weights:
        out += (weights,)
    if return_lse:
        out += (lse,)
    return out[0] if len(out) == 1 else out


def global_attn_blocked(cfg, Q, K, V, rows, return_lse=False):
    """Same result as ``global_attn`` for many rows at once (one matmul per
    head over all requested rows instead of one per row).  Used where the
    per-row loop would take minutes; checked against ``global_attn`` in the
    tests.  The arithmetic per row is unchanged.
    """
    Q, K, V = np.asarray(Q), np.asarray(K), np.asarray(V)
    H, d = cfg.n_heads, cfg.head_dim
    scale = cfg.scale
    rows = np.asarray(rows, dtype=np.int64)
    Kc, Vc, idx, kmean, vmean = build_kv(cfg, K, V)
    Q_r = Q[rows].astype(np.float64)      # only the requested rows are widened
    K_r = K[rows].astype(np.float64)
    V_r = V[rows].astype(np.float64)
    dropped = dropped_token_mask(cfg)
    n_dropped = int(dropped.sum())
    O = np.empty((len(rows), H, d), dtype=np.float64)
    lse = np.empty((len(rows), H), dtype=np.float64)
    row_dropped = dropped[rows]
    has_diag = row_dropped & bool(cfg.diag)
    count = n_dropped - has_diag.astype(np.int64)
    has_mean = (count > 0) & (cfg.mean_fill != 0)
    NEG = -np.inf
    for h in range(H):
        q = Q_r[:, h, :]                                 # [R, d]
        logit_s = scale * (q @ Kc[:, h, :].T)            # [R, M]
        logit_d = np.where(has_diag, scale * np.sum(q * K_r[:, h, :], axis=1), NEG)
        if kmean is not None:
            lm = scale * (q @ kmean[h])
            if cfg.mean_fill == 2:
                lm = lm + np.log(np.maximum(count, 1))
            logit_m = np.where(has_mean, lm, NEG)
        else:
            logit_m = np.full(len(rows), NEG)
        mx = np.maximum(np.maximum(logit_s.max(axis=1), logit_d), logit_m)
        p_s = np.exp(logit_s - mx[:, None])
        p_d = np.exp(logit_d - mx)
        p_m = np.exp(logit_m - mx)
        z = p_s.sum(axis=1) + p_d + p_m
        o = p_s @ Vc[:, h, :]
        o += p_d[:, None] * V_r[:, h, :]
        if kmean is not None:
            o += p_m[:, None] * vmean[h][None, :]
        O[:, h, :] = o / z[:, None]
        lse[:, h] = mx + np.log(z)
    return (O, lse) if return_lse else O


def frame_attn(cfg, Q, K, V, rows=None, return_lse=False):
    """Frame attention of a converted early global block (Sec. 4.2, "Global-to-Frame Attention
    Conversion"): the (B, N L, C) rearrangement is skipped, so every token attends to the L tokens
    of its own frame only (special tokens included), with plain softmax attention.  Nothing is
    subsampled; sigma, diag and mean_fill of ``cfg`` play no part.

    Q, K, V: [N*L, H, d].  Returns O [len(rows), H, d] float64 (and the natural-log normaliser
    [len(rows), H] with ``return_lse``) for the query rows ``rows`` (default: all), one row at a
    time: logits over the frame's keys, one softmax, weighted sum of the frame's values.
    """
    Q, K, V = np.asarray(Q), np.asarray(K), np.asarray(V)
    H, d, L = cfg.n_heads, cfg.head_dim, cfg.tokens_per_frame
    assert Q.shape == (cfg.n_tokens, H, d) and K.shape == Q.shape and V.shape == Q.shape
    scale = cfg.scale
    if rows is None:
        rows = np.arange(cfg.n_tokens)
    rows = np.asarray(rows, dtype=np.int64)
    O = np.empty((len(rows), H, d), dtype=np.float64)
    lse = np.empty((len(rows), H), dtype=np.float64)
    for out_i, i in enumerate(rows):
        f = int(i) // L                                   # the query's frame
        Kf = K[f * L:(f + 1) * L].astype(np.float64)      # [L, H, d]
        Vf = V[f * L:(f + 1) * L].astype(np.float64)
        q = Q[i].astype(np.float64)                       # [H, d]
        logits = scale * np.einsum("hd,lhd->hl", q, Kf)   # [H, L]
        mx = logits.max(axis=1, keepdims=True)
        p = np.exp(logits - mx)
        z = p.sum(axis=1, keepdims=True)
        O[out_i] = np.einsum("hl,lhd->hd", p / z, Vf)
        lse[out_i] = (mx + np.log(z))[:, 0]
    return (O, lse) if return_lse else O


def global_attn_indexed(cfg, idx, Q, K, V, rows=None, return_lse=False):
    """The same layer with a caller-chosen retained set (the alternative selectors of the
    supplement, "Comparison with other subsampling strategies": random, high/low-norm or feature
    based picks instead of the fixed grid).  ``idx`` lists the retained token indices (any order,
    no repeats; the caller includes the special tokens it wants kept).  D is every token not in
    ``idx``; everything else follows Sec. 4.3 exactly as in ``global_attn``: logits over the
    retained set, the query's own column if it is in D (diag), one mean pair over D entering with
    weight 1 or with the count of columns it stands for (mean_fill 1 / 2), one shared softmax.
    The retained keys are taken in ascending token order.

    An empty ``idx`` is the paper's G2M variant (Sec. 5.4, "Effect of the Early Global Attention
    Layers"): every Key/Value, special tokens included, is replaced by the one mean pair over the
    whole sequence.  With ``diag`` off every output row is then that mean Value; with ``diag`` on
    each query sees its own column and the mean pair.
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    H, d = cfg.n_heads, cfg.head_dim
    assert Q.shape == (cfg.n_tokens, H, d) and K.shape == Q.shape and V.shape == Q.shape
    idx = np.sort(np.asarray(idx, dtype=np.int64))
    assert len(np.unique(idx)) == len(idx) and (len(idx) == 0 or (idx[0] >= 0 and idx[-1] < cfg.n_tokens))
    scale = cfg.scale
    dropped = np.ones(cfg.n_tokens, dtype=bool)
    dropped[idx] = False
    n_dropped = int(dropped.sum())
    Kc, Vc = K[idx], V[idx]                               # [M, H, d]
    kmean = K[dropped].mean(axis=0) if n_dropped else None
    vmean = V[dropped].mean(axis=0) if n_dropped else None
    if rows is None:
        rows = np.arange(cfg.n_tokens)
    rows = np.asarray(rows, dtype=np.int64)
    O = np.empty((len(rows), H, d), dtype=np.float64)
    lse = np.empty((len(rows), H), dtype=np.float64)
    for out_i, i in enumerate(rows):
        q = Q[i]
        parts = [scale * np.einsum("hd,mhd->hm", q, Kc)]
        vals = [Vc.transpose(1, 0, 2)]                    # [H, M, d]
        has_diag = bool(cfg.diag) and bool(dropped[i])
        if has_diag:
            parts.append((scale * np.einsum("hd,hd->h", q, K[i]))[:, None])
            vals.append(V[i][:, None, :])
        count = n_dropped - (1 if has_diag else 0)
        if cfg.mean_fill != 0 and count > 0:
            lm = scale * np.einsum("hd,hd->h", q, kmean)
            if cfg.mean_fill == 2:
                lm = lm + math.log(count)
            parts.append(lm[:, None])
            vals.append(vmean[:, None, :])
        logits = np.concatenate(parts, axis=1)
        values = np.concatenate(vals, axis=1)             # [H, cols, d]
        mx = logits.max(axis=1, keepdims=True)
        p = np.exp(logits - mx)
        z = p.sum(axis=1, keepdims=True)
        O[out_i] = np.einsum("hc,hcd->hd", p / z, values)
        lse[out_i] = (mx + np.log(z))[:, 0]
    return (O, lse) if return_lse else O



def round_to_bf16(x):
    """Round-to-nearest-even of real values to the bfloat16 grid (returned as float64): the value is first taken
    to float32, whose upper 16 bits are then rounded (the carry of the lower half, ties to even)."""
    f = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    bits = f.view(np.uint32).astype(np.uint64)
    lower = bits & 0xFFFF
    upper = bits >> 16
    round_up = (lower > 0x8000) | ((lower == 0x8000) & ((upper & 1) == 1))
    upper = upper + round_up.astype(np.uint64)
    out = (upper << 16).astype(np.uint32).view(np.float32)
    out = np.where(np.isfinite(f), out, f)
    return out.astype(np.float64)


def project_build_kv(cfg, X, Wk, Wv, bias_k=None, bias_v=None):
    """K/V projection followed by the compaction of Sec. 4.3, as one operation (the projection's epilogue does
    the compaction, so that diagonal preservation and mean-fill cost no second pass over K and V).

    X [N*L, C]; Wk, Wv [H*d, C] (one row per output, as a linear layer stores its weight); biases [H*d] or None.
    K = X Wk^T + bias_k and V likewise, in float64.  Returns
      K_b, V_b  [N*L, H, d]: the projections rounded to bfloat16 (what the layer stores and attends to),
      Kc, Vc    [M, H, d]:   their retained rows, idx [M],
      kmean, vmean [H, d]:   mean over the dropped patch tokens of the projections BEFORE the rounding
                             (None when nothing is dropped).
    """
    X = np.asarray(X, dtype=np.float64)
    H, d = cfg.n_heads, cfg.head_dim
    assert X.shape[0] == cfg.n_tokens and Wk.shape == (H * d, X.shape[1]) and Wv.shape == Wk.shape
    K = X @ np.asarray(Wk, dtype=np.float64).T
    V = X @ np.asarray(Wv, dtype=np.float64).T
    if bias_k is not None:
        K = K + np.asarray(bias_k, dtype=np.float64)[None, :]
    if bias_v is not None:
        V = V + np.asarray(bias_v, dtype=np.float64)[None, :]
    K = K.reshape(cfg.n_tokens, H, d)
    V = V.reshape(cfg.n_tokens, H, d)
    K_b, V_b = round_to_bf16(K), round_to_bf16(V)
    idx = build_index(cfg)
    dropped = dropped_token_mask(cfg)
    kmean = K[dropped].mean(axis=0) if dropped.any() else None
    vmean = V[dropped].mean(axis=0) if dropped.any() else None
    return K_b, V_b, K_b[idx], V_b[idx], idx, kmean, vmean
