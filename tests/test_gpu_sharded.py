"""Frame-sharded layer on one GPU: the shards of a two- or three-rank split are computed one after the
other (no kernel waits on another) through the entry points a rank calls (`avggt_build_kv_shard`,
`avggt_shard_assemble`, `avggt_global_attn_shard`), and every shard's output is checked against the
fp64 oracle of the whole sequence.  The collectives themselves are covered by the two-rank gloo test
on the CPU."""

import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

import paper_2512_02541_b200 as P
from oracle import avggt_oracle as orc
from paper_2512_02541_b200 import inputs, sharded

pytestmark = pytest.mark.gpu


def _shard_run(wl, world, keep_first=False, seed=0):
    """Returns (Q, K, V, O, Kc, Vc, kmean, vmean) of the whole sequence, O assembled from `world` sequentially
    computed shards.  The all-gather is stood in for by every shard writing its own slot of one common exchange
    buffer, the all-reduce by adding the shards' sums."""
    Q, K, V = inputs.make_qkv(wl, seed=seed, device="cuda")
    L, H, d = wl.tokens_per_frame, wl.n_heads, wl.head_dim
    mk = lambda n, kff: P.make_params(n, wl.grid_h, wl.grid_w, wl.n_special, H, d, wl.sigma, diag=wl.diag,
                                      mean_fill=wl.mean_fill, keep_first_frame=kff)
    ranges = [sharded.shard_frames(wl.n_frames, world, r) for r in range(world)]
    params = [mk(f1 - f0, keep_first and r == 0) for r, (f0, f1) in enumerate(ranges)]
    counts = [P.avggt_kv_count(p) for p in params]
    kept, dropped = [c[0] for c in counts], [c[1] for c in counts]
    slot_rows = max(kept)
    gathered = torch.zeros((world, 2, H, slot_rows, d), dtype=torch.bfloat16, device="cuda")
    total = torch.zeros((2, H, d), device="cuda")
    for r, (f0, f1) in enumerate(ranges):
        bws, _ = P.avggt_workspace_bytes(params[r])
        sums = torch.full((2, H, d), float("nan"), device="cuda")
        ws = torch.empty((max(bws, 16),), dtype=torch.uint8, device="cuda")
        P.avggt_build_kv_shard(params[r], K[f0 * L:f1 * L], V[f0 * L:f1 * L], gathered[r], slot_rows, None, sums, ws, ws.numel())
        total += sums
    n_dropped = sum(dropped)
    Kc = torch.full((H, sum(kept), d), float("nan"), dtype=torch.bfloat16, device="cuda")
    Vc = torch.full_like(Kc, float("nan"))
    kmean = torch.zeros((H, d), device="cuda"); vmean = torch.zeros_like(kmean)
    P.avggt_shard_assemble(params[0], gathered, kept, slot_rows, total, n_dropped, Kc, Vc, kmean, vmean)
    torch.cuda.synchronize()
    O = torch.full_like(Q, float("nan"))
    for r, (f0, f1) in enumerate(ranges):
        _, aws = P.avggt_workspace_bytes(params[r])
        ws = torch.zeros((max(aws, 16),), dtype=torch.uint8, device="cuda")
        sl = slice(f0 * L, f1 * L)
        P.avggt_global_attn_shard(params[r], sum(kept), n_dropped, Q[sl], K[sl], V[sl], Kc, Vc, kmean, vmean, O[sl], None,
                                  ws, ws.numel())
        torch.cuda.synchronize()
        P.avggt_check_status(ws)
    return Q, K, V, O, Kc, Vc, kmean, vmean


@pytest.mark.parametrize("world", (2, 3))
@pytest.mark.parametrize("keep_first", (False, True))
def test_shards_reproduce_the_whole_sequence(world, keep_first):
    wl = inputs.Workload("shard", 5, 11, 13, 5, 4, 64, 4, 1, 2, "proj", keep_first_frame=int(keep_first))
    Q, K, V, O, Kc, Vc, kmean, vmean = _shard_run(wl, world, keep_first, seed=8)
    ocfg = orc.SGAConfig(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                         keep_first_frame=keep_first)
    Qh, Kh, Vh = (t.float().cpu().numpy() for t in (Q, K, V))
    # the assembled compact arrays are those of the unsharded layer, bit for bit
    Kc_w, Vc_w, idx, kmean_w, vmean_w = orc.build_kv(ocfg, Kh, Vh)
    np.testing.assert_array_equal(Kc.float().cpu().numpy().transpose(1, 0, 2), Kc_w)
    np.testing.assert_array_equal(Vc.float().cpu().numpy().transpose(1, 0, 2), Vc_w)
    for got_m, want_m, src in ((kmean, kmean_w, Kh), (vmean, vmean_w, Vh)):
        assert np.abs(got_m.cpu().numpy().astype(np.float64) - want_m).max() <= 1e-5 * float(np.abs(src).mean())
    want = orc.global_attn_blocked(ocfg, Qh, Kh, Vh, np.arange(wl.n_tokens))
    got = O.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    err = np.abs(got - want)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (err.max(), err.mean())


def test_class_with_a_one_rank_group():
    """FrameShardedAttention end to end with a process group of one rank (NCCL on this GPU)."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        wl = inputs.Workload("one", 4, 10, 10, 5, 4, 64, 4, 1, 2, "proj")
        Q, K, V = inputs.make_qkv(wl, seed=2, device="cuda")
        layer = sharded.FrameShardedAttention(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma)
        O = layer.forward(Q, K, V)
        layer.check_status()
        params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma)
        ref = P.SubsampledGlobalAttention(params)
        O_ref = ref.forward(Q, K, V)
        ref.check_status()
        assert torch.equal(O, O_ref)
    finally:
        dist.destroy_process_group()
