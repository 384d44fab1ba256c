"""Buffer management around the two library calls (PyTorch is used for device memory and streams only)."""

import torch

from . import binding as B


class SubsampledGlobalAttention:
    """Owns the compact K/V, the mean pair, the index list and the workspaces of one problem shape
    and runs the two C-ABI calls on the current CUDA stream.

    ``forward(Q, K, V)`` takes bf16 CUDA tensors [N*L, H, d] and returns O of the same shape.
    """

    def __init__(self, params, device="cuda", want_lse=False):
        if not torch.cuda.is_available():
            raise RuntimeError("libavggt needs a CUDA device (sm_100); there is no CPU fallback")
        self.params = params
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.M, self.n_dropped = B.avggt_kv_count(params)
            self.build_ws_bytes, self.attn_ws_bytes = B.avggt_workspace_bytes(params)
        H, d = params.n_heads, params.head_dim
        self.n_tok = params.n_frames * params.tokens_per_frame
        dev = self.device
        self.Kc = torch.empty((H, self.M, d), dtype=torch.bfloat16, device=dev)
        self.Vc = torch.empty((H, self.M, d), dtype=torch.bfloat16, device=dev)
        self.idx = torch.empty((self.M,), dtype=torch.int32, device=dev)
        self.kmean = torch.zeros((H, d), dtype=torch.float32, device=dev)
        self.vmean = torch.zeros((H, d), dtype=torch.float32, device=dev)
        self.build_ws = torch.empty((max(self.build_ws_bytes, 16),), dtype=torch.uint8, device=dev)
        self.attn_ws = torch.zeros((max(self.attn_ws_bytes, 16),), dtype=torch.uint8, device=dev)
        self.lse = torch.empty((self.n_tok, H), dtype=torch.float32, device=dev) if want_lse else None

    def _stream(self):
        return torch.cuda.current_stream(self.device).cuda_stream

    def build_kv(self, K, V):
        B.avggt_build_kv(self.params, K, V, self.Kc, self.Vc, self.idx, self.kmean, self.vmean,
                         self.build_ws, self.build_ws.numel(), self._stream())

    def attend(self, Q, K, V, out=None):
        if out is None:
            out = torch.empty_like(Q)
        B.avggt_global_attn(self.params, Q, K, V, self.Kc, self.Vc, self.kmean, self.vmean, out, self.lse,
                            self.attn_ws, self.attn_ws.numel(), self._stream())
        return out

    def frame_attend(self, Q, K, V, out=None):
        """Frame attention (a converted early global block): each frame attends to itself only."""
        self._check_inputs(Q, K, V)
        if out is None:
            out = torch.empty_like(Q)
        with torch.cuda.device(self.device):
            B.avggt_frame_attn(self.params, Q, K, V, out, self.lse, self.attn_ws, self.attn_ws.numel(), self._stream())
        return out

    def forward(self, Q, K, V, out=None):
        self._check_inputs(Q, K, V)
        with torch.cuda.device(self.device):
            self.build_kv(K, V)
            return self.attend(Q, K, V, out)

    __call__ = forward

    def forward_host(self, hQ, hK, hV, hO, n_chunks=8):
        """The layer on host buffers (pinned memory), with the copies hidden behind the kernels.

        K and V go to the device first (the compaction and the mean need all of them); Q then arrives in
        ``n_chunks`` groups of frames on a copy stream while the attention of the previous group runs
        (``avggt_global_attn_shard``: the queries of a frame range against the whole sequence's compact keys), and
        every group's output leaves on a second copy stream.  Everything is ordered with events and the call
        returns without waiting for the device: the current stream waits for the last output copy.  The device
        copies of K and V alternate between two buffers, so that the K and V of a call made right after this one
        travel while this one's attention runs; Q and O have one buffer, guarded group by group.  The device
        staging buffers are allocated on first use.
        """
        p = self.params
        dev = self.device
        cur = torch.cuda.current_stream(dev)
        if not hasattr(self, "_host_path"):
            shape = (self.n_tok, p.n_heads, p.head_dim)
            new = lambda: torch.empty(shape, dtype=torch.bfloat16, device=dev)
            self._host_path = dict(
                Q=new(), O=new(), K=[new(), new()], V=[new(), new()], h2d=torch.cuda.Stream(dev), d2h=torch.cuda.Stream(dev),
                calls=0,
                kv_free=[None, None],    # per K/V buffer: the call that used it last has finished with it
                bounds=None,             # frame groups of the previous call
                q_free=[], o_free=[],    # per group of the previous call: its attention has read Q / its output copy has left O
                # one status block per group of frames, so that no launch clears what an earlier one reported
                ws=torch.zeros((max(1, p.n_frames), max(self.attn_ws_bytes, 256)), dtype=torch.uint8, device=dev))
        hp = self._host_path
        which = hp["calls"] & 1
        hp["calls"] += 1
        dQ, dK, dV, dO, h2d, d2h = hp["Q"], hp["K"][which], hp["V"][which], hp["O"], hp["h2d"], hp["d2h"]
        L = p.tokens_per_frame
        n_chunks = max(1, min(n_chunks, p.n_frames))
        bounds = [round(i * p.n_frames / n_chunks) for i in range(n_chunks + 1)]
        same_groups = hp["bounds"] == bounds
        keep_first = bool(p.flags & B.AVGGT_FLAG_KEEP_FIRST_FRAME)
        if not same_groups:
            # the previous call cut the frames differently: wait for all of it before Q and O are touched
            h2d.wait_stream(cur)
            h2d.wait_stream(d2h)
        with torch.cuda.device(dev):
            with torch.cuda.stream(h2d):
                if hp["kv_free"][which] is not None:
                    h2d.wait_event(hp["kv_free"][which])
                dK.copy_(hK, non_blocking=True)
                dV.copy_(hV, non_blocking=True)
                kv_ready = torch.cuda.Event()
                kv_ready.record(h2d)
                q_ready = []
                for c in range(n_chunks):
                    sl = slice(bounds[c] * L, bounds[c + 1] * L)
                    if same_groups:
                        h2d.wait_event(hp["q_free"][c])
                    dQ[sl].copy_(hQ[sl], non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(h2d)
                    q_ready.append(ev)
            cur.wait_event(kv_ready)
            self.build_kv(dK, dV)
            q_free, o_free = [], []
            for c in range(n_chunks):
                f0, f1 = bounds[c], bounds[c + 1]
                sl = slice(f0 * L, f1 * L)
                cp = B.make_params(f1 - f0, p.grid_h, p.grid_w, p.n_special, p.n_heads, p.head_dim, p.sigma, diag=p.diag,
                                   mean_fill=p.mean_fill, softmax_scale=p.softmax_scale,
                                   keep_first_frame=keep_first and f0 == 0)
                cur.wait_event(q_ready[c])
                if same_groups:
                    cur.wait_event(hp["o_free"][c])
                B.avggt_global_attn_shard(cp, self.M, self.n_dropped, dQ[sl], dK[sl], dV[sl], self.Kc, self.Vc, self.kmean,
                                          self.vmean, dO[sl], None, hp["ws"][c], hp["ws"][c].numel(), cur.cuda_stream)
                done = torch.cuda.Event()
                done.record(cur)
                q_free.append(done)
                d2h.wait_event(done)
                with torch.cuda.stream(d2h):
                    hO[sl].copy_(dO[sl], non_blocking=True)
                    left = torch.cuda.Event()
                    left.record(d2h)
                    o_free.append(left)
            hp["kv_free"][which] = q_free[-1]
            hp["bounds"], hp["q_free"], hp["o_free"] = bounds, q_free, o_free
            cur.wait_stream(d2h)
        return hO

    def check_status(self):
        """Synchronises the device and raises if a device-side wait gave up."""
        torch.cuda.synchronize(self.device)
        B.avggt_check_status(self.attn_ws)
        if hasattr(self, "_host_path"):
            for ws in self._host_path["ws"]:
                B.avggt_check_status(ws)

    def _check_inputs(self, *tensors):
        shape = (self.n_tok, self.params.n_heads, self.params.head_dim)
        for t in tensors:
            if t.dtype != torch.bfloat16 or tuple(t.shape) != shape or not t.is_contiguous() or t.device.type != "cuda":
                raise ValueError(f"expected contiguous bf16 CUDA tensors of shape {shape}")
