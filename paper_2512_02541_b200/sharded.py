"""Frame-sharded subsampled global attention: one process per GPU, each owning a contiguous
range of frames.

The layer has one exchange step (Sec. 4.3 defines the retained set S and the mean pair over the
whole sequence): every rank compacts the K/V of its own frames, the compact arrays are
all-gathered (they are a 1/sigma fraction of K/V), the per-rank mean sums are all-reduced, and
each rank then attends with its own queries against the whole sequence's compact keys
(``avggt_global_attn_shard``).  The gathered arrays land in this GPU's own memory before any
kernel reads them.  PyTorch supplies the process group, the collectives and the buffers; every
step of the path itself runs in the library's kernels.
"""

import torch
import torch.distributed as dist

from . import binding as B


def shard_frames(n_frames, world, rank):
    """Contiguous frame range [f0, f1) of ``rank``: sizes differ by at most one, earlier ranks get the extra."""
    base, extra = divmod(n_frames, world)
    f0 = rank * base + min(rank, extra)
    return f0, f0 + base + (1 if rank < extra else 0)


def assemble_compact(per_rank, kept_counts):
    """per_rank[r]: [H, >= kept_counts[r], d] (possibly padded along the key axis) -> [H, sum(kept), d],
    the ranks' compact keys one after the other, i.e. in ascending token order."""
    H, _, d = per_rank[0].shape
    out = per_rank[0].new_empty((H, int(sum(kept_counts)), d))
    off = 0
    for t, m in zip(per_rank, kept_counts):
        out[:, off:off + m, :] = t[:, :m, :]
        off += m
    return out


def gather_compact(local, kept_counts, group=None):
    """All-gather of the head-major compact arrays [H, M_r, d] of all ranks into [H, sum_r M_r, d].
    ``kept_counts``: M_r of every rank (a pure function of the frame split, known everywhere)."""
    world = dist.get_world_size(group)
    H, m_loc, d = local.shape
    m_max = int(max(kept_counts))
    padded = local.new_zeros((H, m_max, d))
    padded[:, :m_loc, :] = local
    # moved as bytes: a plain copy, whatever the backend knows about bf16
    gathered = [torch.empty((H, m_max, d * local.element_size()), dtype=torch.uint8, device=local.device)
                for _ in range(world)]
    dist.all_gather(gathered, padded.view(torch.uint8), group=group)
    return assemble_compact([g.view(local.dtype) for g in gathered], kept_counts)


def combine_means(local_mean, local_count, group=None):
    """Mean over all ranks' dropped tokens from each rank's mean and count: all-reduce of the sums
    mean_r * count_r and of the counts.  Returns (mean [H, d] float32, total count)."""
    packed = torch.cat([(local_mean.float() * float(local_count)).reshape(-1),
                        torch.tensor([float(local_count)], dtype=torch.float32, device=local_mean.device)])
    packed = packed.double()          # counts of the order of 1e6 and sums of as many terms: keep the reduction exact enough
    dist.all_reduce(packed, op=dist.ReduceOp.SUM, group=group)
    total = packed[-1].item()
    mean = (packed[:-1] / max(total, 1.0)).float().reshape(local_mean.shape)
    return mean, int(round(total))


class FrameShardedAttention:
    """One rank of a frame-sharded layer.  ``make_params_for(n_local_frames, keep_first)`` returns the
    avggt_params of a shard; the rank that owns frame 0 carries the keep-first-frame flag, if any."""

    def __init__(self, n_frames, grid_h, grid_w, n_special, n_heads, head_dim, sigma, diag=1, mean_fill=B.AVGGT_MEAN_FILL,
                 keep_first_frame=False, group=None, device="cuda"):
        if not torch.cuda.is_available():
            raise RuntimeError("libavggt needs a CUDA device (sm_100); there is no CPU fallback")
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.device = torch.device(device)
        mk = lambda n, kff: B.make_params(n, grid_h, grid_w, n_special, n_heads, head_dim, sigma, diag=diag,
                                          mean_fill=mean_fill, keep_first_frame=kff)
        ranges = [shard_frames(n_frames, self.world, r) for r in range(self.world)]
        if any(f1 <= f0 for f0, f1 in ranges):
            raise ValueError("more ranks than frames")
        self.kept, self.dropped = [], []
        for r, (f0, f1) in enumerate(ranges):
            m, nd = B.avggt_kv_count(mk(f1 - f0, keep_first_frame and r == 0))
            self.kept.append(m)
            self.dropped.append(nd)
        f0, f1 = ranges[self.rank]
        self.params = mk(f1 - f0, keep_first_frame and self.rank == 0)
        self.n_local_tokens = (f1 - f0) * self.params.tokens_per_frame
        H, d = n_heads, head_dim
        dev = self.device
        with torch.cuda.device(dev):
            bws, aws = B.avggt_workspace_bytes(self.params)
        m_loc = self.kept[self.rank]
        self.Kc_loc = torch.empty((H, m_loc, d), dtype=torch.bfloat16, device=dev)
        self.Vc_loc = torch.empty_like(self.Kc_loc)
        self.kmean_loc = torch.zeros((H, d), dtype=torch.float32, device=dev)
        self.vmean_loc = torch.zeros_like(self.kmean_loc)
        self.build_ws = torch.empty((max(bws, 16),), dtype=torch.uint8, device=dev)
        self.attn_ws = torch.zeros((max(aws, 16),), dtype=torch.uint8, device=dev)
        self.mean_fill = mean_fill

    def forward(self, Q, K, V, out=None):
        """Q, K, V: this rank's rows, bf16 [n_local_frames * L, H, d].  Returns this rank's rows of O."""
        if out is None:
            out = torch.empty_like(Q)
        stream = torch.cuda.current_stream(self.device).cuda_stream
        with torch.cuda.device(self.device):
            B.avggt_build_kv(self.params, K, V, self.Kc_loc, self.Vc_loc, None, self.kmean_loc, self.vmean_loc,
                             self.build_ws, self.build_ws.numel(), stream)
            Kc = gather_compact(self.Kc_loc, self.kept, self.group)
            Vc = gather_compact(self.Vc_loc, self.kept, self.group)
            n_dropped = sum(self.dropped)
            if self.mean_fill != 0 and n_dropped > 0:
                kmean, _ = combine_means(self.kmean_loc, self.dropped[self.rank], self.group)
                vmean, _ = combine_means(self.vmean_loc, self.dropped[self.rank], self.group)
            else:
                kmean, vmean = self.kmean_loc, self.vmean_loc
            self._keep = (Kc, Vc, kmean, vmean)        # alive until the kernel has run
            B.avggt_global_attn_shard(self.params, sum(self.kept), n_dropped, Q, K, V, Kc, Vc, kmean, vmean, out, None,
                                      self.attn_ws, self.attn_ws.numel(), stream)
        return out

    def check_status(self):
        torch.cuda.synchronize(self.device)
        B.avggt_check_status(self.attn_ws)
