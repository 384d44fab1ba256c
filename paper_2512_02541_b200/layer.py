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

    def check_status(self):
        """Synchronises the device and raises if a device-side wait gave up."""
        torch.cuda.synchronize(self.device)
        B.avggt_check_status(self.attn_ws)

    def _check_inputs(self, *tensors):
        shape = (self.n_tok, self.params.n_heads, self.params.head_dim)
        for t in tensors:
            if t.dtype != torch.bfloat16 or tuple(t.shape) != shape or not t.is_contiguous() or t.device.type != "cuda":
                raise ValueError(f"expected contiguous bf16 CUDA tensors of shape {shape}")
