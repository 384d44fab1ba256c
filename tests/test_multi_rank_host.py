"""Host-side logic of the multi-GPU path, run as two gloo ranks on the CPU.

`bench.py --gpus N` splits the frames of one problem over the ranks and reports the whole-job rate
against the slowest rank's device time.  What needs no GPU is covered here: the max-over-ranks
reduction, the aggregate, that only rank 0 of the reference arm prints, the frame split, and the
two collectives of the exchange step on the exchange buffer's geometry.
"""

import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank r "measured" (10 + r) ms for the steps and (100 - r) ms end to end
    got = bench.max_over_ranks([10.0 + rank, 100.0 - rank], "cpu", world)
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as fh:
        json.dump(got, fh)
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_two_gloo_ranks(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        got = json.load(open(tmp_path / f"rank{r}.json"))
        assert got == [11.0, 100.0]          # slowest rank of each measurement, on every rank


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks([3.5, 2.0], "cpu", 1) == [3.5, 2.0]
    # 2000 queries over all ranks per step, slowest step 4 ms -> 500k queries/s for the whole job
    assert bench.whole_job_throughput(2000, 4.0) == pytest.approx(5.0e5)


def test_reference_arm_prints_on_rank_zero_only():
    """Under torchrun the reference arm (the CPU oracle) runs on rank 0; the other ranks exit 0 silently."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--workload", "tiny_n4_g16_s2"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""
    env["RANK"] = "0"
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--workload", "tiny_n4_g16_s2"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2


# --------------------------------------------------------------------------
# frame-sharded layer: the exchange step (all-gather of compact K/V, all-reduce of the mean sums)
# --------------------------------------------------------------------------

def test_shard_frames_covers_all_frames_evenly():
    from paper_2512_02541_b200.sharded import shard_frames
    for n, w in [(100, 8), (7, 3), (8, 8), (333, 4), (5, 1)]:
        ranges = [shard_frames(n, w, r) for r in range(w)]
        assert ranges[0][0] == 0 and ranges[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
        sizes = [f1 - f0 for f0, f1 in ranges]
        assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)


def _exchange_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2512_02541_b200.sharded import exchange
    H, d = 3, 8
    kept = [5, 9]                                  # uneven shards: padding rows in rank 0's slot
    slot_rows = max(kept)
    gen = torch.Generator().manual_seed(100 + rank)
    mine = torch.randn((2, H, kept[rank], d), generator=gen).bfloat16()
    gathered = torch.zeros((world, 2, H, slot_rows, d), dtype=torch.bfloat16)
    gathered[rank, :, :, :kept[rank]] = mine        # what the shard compaction writes: its own slot only
    sums = torch.randn((2, H, d), generator=gen)
    mine_sums = sums.clone()
    exchange(gathered, rank, sums)
    torch.save({"mine": mine, "mine_sums": mine_sums, "gathered": gathered, "sums": sums}, os.path.join(out_dir, f"x{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_exchange_step_two_gloo_ranks(tmp_path):
    world = 2
    mp.spawn(_exchange_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    got = [torch.load(tmp_path / f"x{r}.pt") for r in range(world)]
    kept = [5, 9]
    want_sums = got[0]["mine_sums"] + got[1]["mine_sums"]
    for r in range(world):
        g = got[r]["gathered"]
        for o in range(world):                      # every rank holds every owner's slot, padding untouched
            assert torch.equal(g[o, :, :, :kept[o]], got[o]["mine"])
            assert not g[o, :, :, kept[o]:].any()
        assert torch.allclose(got[r]["sums"], want_sums, rtol=0, atol=1e-6)
