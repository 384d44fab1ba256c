"""Seeded synthetic Q/K/V generators shaped like the paper's workloads.

This module holds no arithmetic of the method: it only names the workload
shapes (frames, patch grid, special tokens, heads, head dim, subsampling
factor, switches) and draws random tensors.  Both the CUDA path's tests and the
CPU oracle's tests feed from it, so that they see the same numbers.

Two value recipes:

  * ``iid``:  Q, K, V ~ N(0, 1) independently, Q multiplied by 3 so that
    q.k / sqrt(d) has a standard deviation of about 3.
  * ``proj``: token features x = g + 0.5 * c with g ~ N(0, 1) per token and
    c ~ N(0, 1) per patch position, shared by all frames (special tokens get no
    shared part), projected as Q = x W_q, K = x W_q, V = x W_v with
    W ~ N(0, 1/C).  Sharing the projection between Q and K makes the query's
    own key and the same patch position in other frames score high, which is
    the structure Sec. 3.1 of the paper reports for the middle global layers.

The paper evaluates on image datasets and trained weights that are not
available here; only the shapes of those workloads (10 to 800 frames, five
special tokens, the patch-14 grid of a 518-pixel image, 16 heads of 64) are
taken from it.
"""

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_frames: int
    grid_h: int
    grid_w: int
    n_special: int
    n_heads: int
    head_dim: int
    sigma: int
    diag: int
    mean_fill: int
    recipe: str = "proj"
    keep_first_frame: int = 0

    @property
    def tokens_per_frame(self):
        return self.n_special + self.grid_h * self.grid_w

    @property
    def n_tokens(self):
        return self.n_frames * self.tokens_per_frame

    def with_(self, **kw):
        return replace(self, **kw)


def _vggt(name, n_frames, sigma, diag=1, mean_fill=2):
    return Workload(name, n_frames, 37, 37, 5, 16, 64, sigma, diag, mean_fill, "proj")


WORKLOADS = {
    # tiny case the CPU oracle finishes in seconds
    "tiny_n4_g16_s2": Workload("tiny_n4_g16_s2", 4, 16, 16, 5, 16, 64, 2, 1, 2, "iid"),
    # VGGT-shaped layers
    # 30 frames: larger than L2 but small enough for a full profiler capture
    "vggt_n30_s4": _vggt("vggt_n30_s4", 30, 4),
    "vggt_n30_s9": _vggt("vggt_n30_s9", 30, 9),
    "vggt_n100_s4": _vggt("vggt_n100_s4", 100, 4),
    "vggt_n300_s6": _vggt("vggt_n300_s6", 300, 6),
    "vggt_n800_s9": _vggt("vggt_n800_s9", 800, 9),
    # factor sweep at 333 frames; s=1 is the dense layer with both switches off
    "vggt_n333_s1": _vggt("vggt_n333_s1", 333, 1, diag=0, mean_fill=0),
    "vggt_n333_s2": _vggt("vggt_n333_s2", 333, 2),
    "vggt_n333_s4": _vggt("vggt_n333_s4", 333, 4),
    "vggt_n333_s6": _vggt("vggt_n333_s6", 333, 6),
    "vggt_n333_s9": _vggt("vggt_n333_s9", 333, 9),
}


def make_qkv(wl, seed=0, device="cpu", frames_per_chunk=16, frame_range=None):
    """Return (Q, K, V), each a bf16 tensor [N*L, H, d] on ``device``.

    The generator is seeded per call; CPU and CUDA generators give different
    streams, so a parity test draws once and hands the same tensors (copied to
    the host) to the oracle.  ``frame_range = (f0, f1)`` returns only the rows
    of frames [f0, f1) of the very same tensors (all frames are still drawn, so
    every rank of a frame-sharded run sees its part of one common problem).
    """
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    L, H, d = wl.tokens_per_frame, wl.n_heads, wl.head_dim
    n_tok = wl.n_tokens
    shape = (n_tok, H, d)
    k0, k1 = (0, wl.n_frames) if frame_range is None else frame_range
    if wl.recipe == "iid":
        Q = torch.randn(shape, generator=gen, device=device, dtype=torch.float32) * 3.0
        K = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        V = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        return tuple(t[k0 * L:k1 * L].bfloat16().contiguous() for t in (Q, K, V))
    if wl.recipe != "proj":
        raise ValueError(f"unknown recipe {wl.recipe!r}")
    shape = ((k1 - k0) * L, H, d)

    C = H * d
    w_q = torch.randn((C, C), generator=gen, device=device, dtype=torch.float32) * (C ** -0.5)
    w_v = torch.randn((C, C), generator=gen, device=device, dtype=torch.float32) * (C ** -0.5)
    shared = torch.randn((wl.grid_h * wl.grid_w, C), generator=gen, device=device, dtype=torch.float32)
    Q = torch.empty(shape, device=device, dtype=torch.bfloat16)
    K = torch.empty(shape, device=device, dtype=torch.bfloat16)
    V = torch.empty(shape, device=device, dtype=torch.bfloat16)
    for f0 in range(0, wl.n_frames, frames_per_chunk):
        nf = min(frames_per_chunk, wl.n_frames - f0)
        x = torch.randn((nf, L, C), generator=gen, device=device, dtype=torch.float32)
        x[:, wl.n_special:, :] += 0.5 * shared
        a, b = max(f0, k0), min(f0 + nf, k1)          # frames of this chunk that the caller keeps
        if a >= b:
            continue
        x = x[a - f0:b - f0].reshape((b - a) * L, C)
        qk = (x @ w_q).bfloat16().reshape((b - a) * L, H, d)
        Q[(a - k0) * L:(b - k0) * L] = qk
        K[(a - k0) * L:(b - k0) * L] = qk
        V[(a - k0) * L:(b - k0) * L] = (x @ w_v).bfloat16().reshape((b - a) * L, H, d)
    return Q, K, V


def sample_rows(wl, n_rows, seed=0, tile=128, must_include=()):
    """A fixed, stratified sample of query rows for parity checks on workloads
    too large for the oracle to cover in full: the first and last rows, the
    special tokens of the first and last frame, rows on both sides of tile
    boundaries at the start, in the middle and at the end of the sequence (every
    position class of a row within a pair of tiles: row mod 2*tile in
    {0, tile-1, tile, 2*tile-1}), the ragged tail tile, the rows the caller
    names in ``must_include``, and uniformly random rows up to ``n_rows``.
    """
    n_tok, L = wl.n_tokens, wl.tokens_per_frame
    if n_rows >= n_tok:
        return torch.arange(n_tok)
    picks = set(int(r) for r in must_include)
    picks.update(range(min(wl.n_special + 3, n_tok)))                      # frame 0 specials + first patches
    picks.update(range((wl.n_frames - 1) * L, (wl.n_frames - 1) * L + wl.n_special + 3))
    picks.update(range(max(0, n_tok - 4), n_tok))                          # very last rows
    tail0 = (n_tok // tile) * tile
    picks.update(range(max(0, tail0 - 2), min(n_tok, tail0 + 2)))          # around the tail tile
    pair = 2 * tile
    n_pairs = max(1, n_tok // pair)
    for b in sorted({0, 1, n_pairs // 3, n_pairs // 2, (2 * n_pairs) // 3, max(0, n_pairs - 2), n_pairs - 1}):
        for off in (0, 1, tile - 1, tile, tile + 1, pair - 1):
            picks.add(b * pair + off)
    picks = {p for p in picks if 0 <= p < n_tok}
    gen = torch.Generator()
    gen.manual_seed(seed)
    extra = torch.randperm(n_tok, generator=gen)[: max(0, n_rows - len(picks))].tolist()
    picks.update(extra)
    return torch.tensor(sorted(picks), dtype=torch.int64)
