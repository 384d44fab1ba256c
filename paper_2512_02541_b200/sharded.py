"""Frame-sharded subsampled global attention: one process per GPU, each owning a contiguous
range of frames.

The layer has one exchange step (Sec. 4.3 defines the retained set S and the mean pair over the
whole sequence).  Every rank compacts the K/V of its own frames straight into its slot of one
exchange buffer and leaves its mean un-normalised (``avggt_build_kv_shard``); one all-gather
moves the slots (compact K and V together, a 1/sigma fraction of K/V), one all-reduce adds the
sums; ``avggt_shard_assemble`` lays the ranks' compact rows out in ascending token order and
divides the sums by the total count; each rank then attends with its own queries against the
whole sequence's compact keys (``avggt_global_attn_shard``).  The gathered data lands in this
GPU's own memory before any kernel reads it.  PyTorch supplies the process group, the two
collectives and the buffers; every arithmetic step of the path runs in the library's kernels.
"""

import torch
import torch.distributed as dist

from . import binding as B


def shard_frames(n_frames, world, rank):
    """Contiguous frame range [f0, f1) of ``rank``: sizes differ by at most one, earlier ranks get the extra."""
    base, extra = divmod(n_frames, world)
    f0 = rank * base + min(rank, extra)
    return f0, f0 + base + (1 if rank < extra else 0)


def exchange(gathered, rank, sums=None, group=None):
    """The two collectives of the exchange step.

    ``gathered``: [world][...] buffer whose slice ``gathered[rank]`` this rank has filled; after the
    call every slice holds its owner's data (in-place all-gather, moved as bytes).
    ``sums``: float tensor every rank has filled with its partial sums; after the call, their total.
    """
    flat = gathered.view(torch.uint8).view(gathered.shape[0], -1)
    dist.all_gather_into_tensor(flat.view(-1), flat[rank], group=group)
    if sums is not None:
        dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=group)


class FrameShardedAttention:
    """One rank of a frame-sharded layer.  The rank that owns frame 0 carries the keep-first-frame flag, if any."""

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
        self.ranges = [shard_frames(n_frames, self.world, r) for r in range(self.world)]
        if any(f1 <= f0 for f0, f1 in self.ranges):
            raise ValueError("more ranks than frames")
        self.kept, self.dropped = [], []
        for r, (f0, f1) in enumerate(self.ranges):
            m, nd = B.avggt_kv_count(mk(f1 - f0, keep_first_frame and r == 0))
            self.kept.append(m)
            self.dropped.append(nd)
        f0, f1 = self.ranges[self.rank]
        self.params = mk(f1 - f0, keep_first_frame and self.rank == 0)
        self.n_local_tokens = (f1 - f0) * self.params.tokens_per_frame
        self.slot_rows = max(self.kept)
        self.n_kept_total = sum(self.kept)
        self.n_dropped_total = sum(self.dropped)
        H, d = n_heads, head_dim
        dev = self.device
        with torch.cuda.device(dev):
            bws, aws = B.avggt_workspace_bytes(self.params)
        # zeroed once: the padding rows of a slot are never written and never read as keys, but they travel
        self.gathered = torch.zeros((self.world, 2, H, self.slot_rows, d), dtype=torch.bfloat16, device=dev)
        self.sums = torch.zeros((2, H, d), dtype=torch.float32, device=dev)
        self.Kc = torch.empty((H, self.n_kept_total, d), dtype=torch.bfloat16, device=dev)
        self.Vc = torch.empty_like(self.Kc)
        self.kmean = torch.zeros((H, d), dtype=torch.float32, device=dev)
        self.vmean = torch.zeros_like(self.kmean)
        self.build_ws = torch.empty((max(bws, 16),), dtype=torch.uint8, device=dev)
        self.attn_ws = torch.zeros((max(aws, 16),), dtype=torch.uint8, device=dev)
        self.mean_fill = mean_fill

    def _stream(self):
        return torch.cuda.current_stream(self.device).cuda_stream

    def build_kv(self, K, V):
        """Compaction of this rank's rows into its slot of the exchange buffer, sums of its dropped rows."""
        with torch.cuda.device(self.device):
            B.avggt_build_kv_shard(self.params, K, V, self.gathered[self.rank], self.slot_rows, None, self.sums,
                                   self.build_ws, self.build_ws.numel(), self._stream())

    def exchange(self):
        """All-gather of the slots, all-reduce of the sums, assembly of the whole sequence's compact K/V and mean pair."""
        with torch.cuda.device(self.device):
            want_mean = self.mean_fill != 0 and self.n_dropped_total > 0
            if self.world > 1:
                exchange(self.gathered, self.rank, self.sums if want_mean else None, self.group)
            B.avggt_shard_assemble(self.params, self.gathered, self.kept, self.slot_rows, self.sums, self.n_dropped_total,
                                   self.Kc, self.Vc, self.kmean, self.vmean, self._stream())

    def attend(self, Q, K, V, out=None):
        if out is None:
            out = torch.empty_like(Q)
        with torch.cuda.device(self.device):
            B.avggt_global_attn_shard(self.params, self.n_kept_total, self.n_dropped_total, Q, K, V, self.Kc, self.Vc,
                                      self.kmean, self.vmean, out, None, self.attn_ws, self.attn_ws.numel(), self._stream())
        return out

    def forward(self, Q, K, V, out=None):
        """Q, K, V: this rank's rows, bf16 [n_local_frames * L, H, d].  Returns this rank's rows of O."""
        self.build_kv(K, V)
        self.exchange()
        return self.attend(Q, K, V, out)

    def check_status(self):
        torch.cuda.synchronize(self.device)
        B.avggt_check_status(self.attn_ws)
