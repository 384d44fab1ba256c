#!/usr/bin/env python
"""Benchmark of the subsampled global-attention hot path on B200.

One step = one pass of the whole path over one synthetic batch:
``avggt_build_kv`` (K/V compaction + mean-fill reduction) followed by
``avggt_global_attn`` (fused tcgen05 attention), on the VGGT-shaped layer at 100
frames (37x37 patch grid, 5 special tokens, 16 heads x 64, factor 4, diagonal +
mean-fill on).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

With N > 1 (under torchrun) every rank runs an independent replica of the same
problem; there is no data-path collective.  ``--impl reference`` times the fp64
CPU oracle on the host cores on a bounded sample of the same workload.
"""

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2512_02541_b200 import inputs  # noqa: E402

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/; None where no capture covers the workload.  The attention kernel is captured on the 30-frame copy of
# the layer (profiles/global_attn_kernel_vggt_n30_s4.md); its traffic is proportional to the frame count, so the
# 100-frame figure is that capture x 100/30.  The compaction kernel is captured on the 100-frame workload itself.
_ATTN_N30 = 0.299442e9 + 0.068250e9
NCU_TRAFFIC = {
    "vggt_n30_s4": {"global_attn_kernel": _ATTN_N30},
    "vggt_n100_s4": {"global_attn_kernel": _ATTN_N30 * 100 / 30, "build_kv_kernel": 0.562844e9 + 0.103259e9},
}

METRIC = "subsampled_global_attn_queries_per_sec"
UNIT = "queries/s"
DEFAULT_WORKLOAD = "vggt_n100_s4"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def _oracle_cfg(wl):
    from oracle import avggt_oracle as orc
    return orc, orc.SGAConfig(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                              diag=bool(wl.diag), mean_fill=wl.mean_fill, keep_first_frame=bool(wl.keep_first_frame))


def _threads_used():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def time_oracle(wl, n_rows, steps, warmup, seed=0):
    """Times the oracle (as it stands) on ``n_rows`` sampled query rows per step.  -> (queries/s, ms/step, sample)"""
    orc, ocfg = _oracle_cfg(wl)
    Q, K, V = inputs.make_qkv(wl, seed=seed, device="cpu")
    Qh, Kh, Vh = (t.float().numpy() for t in (Q, K, V))
    rows = inputs.sample_rows(wl, n_rows).numpy()
    for _ in range(warmup):
        orc.global_attn_blocked(ocfg, Qh, Kh, Vh, rows[: max(8, len(rows) // 8)])
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        orc.global_attn_blocked(ocfg, Qh, Kh, Vh, rows)
        times.append(time.perf_counter() - t0)
    per_step = sum(times) / len(times)
    sample = (f"{len(rows)} stratified query rows x all {wl.n_heads} heads x all compact keys of {wl.name}, "
              "K/V compaction and mean included in every step")
    return len(rows) / per_step, per_step * 1e3, sample


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_rows = 512
    qps, ms, sample = time_oracle(wl, n_rows, max(1, args.steps), min(args.warmup, 1))
    line = {
        "impl": "reference", "metric": METRIC, "value": qps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": wl.name, "sample_rows_per_step": n_rows},
        "cpu_baseline": {"value": qps, "unit": UNIT, "cores": _threads_used(), "kind": "oracle", "sample": sample},
        "e2e": {"value": qps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device):
        self.proc = None
        self.path = None
        try:
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.fh = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={uuid}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.fh,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.fh.close()
        sm, reasons, smax, power = [], set(), None, []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        with open(self.path) as fh:
            for line in fh:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0])); smax = float(parts[1]); power.append(float(parts[2]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if sm:
            # "under load": samples in the upper half of the observed power draw
            thr = 0.5 * (max(power) + min(power)) if power else 0
            loaded = [c for c, p in zip(sm, power) if p >= thr] or sm
            out.update(sm_mhz=statistics.median(loaded), sm_max_mhz=smax, reasons=sorted(reasons), samples=len(sm),
                       power_w_max=max(power))
        return out


def max_over_ranks(values, device, world):
    """Every rank passes its own device-timed durations; all get the element-wise maximum over the ranks
    (the replicas of a multi-GPU run are timed by the slowest one).  One rank: the values themselves."""
    if world <= 1:
        return [float(v) for v in values]
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_throughput(units_per_rank, world, ms_per_step):
    """Aggregate metric of N replicas: the units all ranks processed per second of the slowest rank's step."""
    return world * units_per_rank / (ms_per_step * 1e-3)


def run_ours(args, wl):
    import torch.distributed as dist

    import paper_2512_02541_b200 as P

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                           diag=wl.diag, mean_fill=wl.mean_fill, keep_first_frame=bool(wl.keep_first_frame))
    layer = P.SubsampledGlobalAttention(params, device=dev)
    Q, K, V = inputs.make_qkv(wl, seed=rank, device=dev)
    O = torch.empty_like(Q)
    n_q, M, H, d = wl.n_tokens, layer.M, wl.n_heads, wl.head_dim
    stream = torch.cuda.current_stream(dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(args.warmup):
        layer.forward(Q, K, V, out=O)
    layer.check_status()

    # ---- device-resident timing: K steps, events on the launching stream
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    sampler = ClockSampler(dev) if rank == 0 else None
    time.sleep(0.15 if sampler else 0)
    barrier()
    for i in range(args.steps):
        ev[i][0].record(stream)
        layer.build_kv(K, V)
        ev[i][1].record(stream)
        layer.attend(Q, K, V, out=O)
        ev[i][2].record(stream)
    barrier()
    clocks = sampler.stop() if sampler else None
    layer.check_status()
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    build_ms = [e[0].elapsed_time(e[1]) for e in ev]
    attn_ms = [e[1].elapsed_time(e[2]) for e in ev]

    # ---- outside the timed region: the same tokens through frame attention (Sec. 4.2), for the report
    fe = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    layer.frame_attend(Q, K, V, out=O)
    barrier()
    fe[0].record(stream)
    for _ in range(args.steps):
        layer.frame_attend(Q, K, V, out=O)
    fe[1].record(stream)
    barrier()
    layer.check_status()
    frame_ms = fe[0].elapsed_time(fe[1]) / args.steps

    # ---- outside the timed region: the dense layer (s = 1, both switches off) on the same tokens, the GPU
    #      reference the metric is quoted against
    dense_ms = None
    if wl.sigma != 1 and not args.no_dense:
        dparams = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, 1,
                                diag=0, mean_fill=0)
        dense = P.SubsampledGlobalAttention(dparams, device=dev)
        dense.forward(Q, K, V, out=O)
        barrier()
        de = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        n_dense = 2
        de[0].record(stream)
        for _ in range(n_dense):
            dense.attend(Q, K, V, out=O)
        de[1].record(stream)
        barrier()
        dense.check_status()
        dense_ms = de[0].elapsed_time(de[1]) / n_dense
        del dense

    # ---- end to end through the public API with host buffers
    e2e_steps = max(1, min(args.steps, 5))
    hQ, hK, hV = (t.cpu().pin_memory() for t in (Q, K, V))
    hO = torch.empty_like(hQ).pin_memory()
    dQ, dK, dV = (torch.empty_like(t) for t in (Q, K, V))

    def e2e_step():
        dQ.copy_(hQ, non_blocking=True); dK.copy_(hK, non_blocking=True); dV.copy_(hV, non_blocking=True)
        layer.forward(dQ, dK, dV, out=O)
        hO.copy_(O, non_blocking=True)

    e2e_step()
    barrier()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    s1.record(stream)
    barrier()
    e2e_ms = s0.elapsed_time(s1)

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dev if world > 1 else "cpu", world)

    if rank == 0:
        peaks = _peaks()
        ms_per_step = total_ms / args.steps
        value = whole_job_throughput(n_q, world, ms_per_step)
        flops = 4.0 * n_q * M * H * d
        attn_avg = sum(attn_ms) / len(attn_ms)
        build_avg = sum(build_ms) / len(build_ms)
        achieved_tf = flops / (attn_avg * 1e-3) / 1e12
        long_run = total_ms > 2000.0
        peak_tf = peaks["bf16_tflops_sustained"] if long_run else peaks["bf16_tflops"]
        build_bytes = 2.0 * (n_q + M) * H * d * 2 if wl.mean_fill else 4.0 * M * H * d * 2
        build_gbs = build_bytes / (build_avg * 1e-3) / 1e9
        in_bytes = 3 * Q.numel() * Q.element_size()
        out_bytes = O.numel() * O.element_size()
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "n_frames": wl.n_frames, "grid": [wl.grid_h, wl.grid_w],
                       "n_special": wl.n_special, "heads": H, "head_dim": d, "sigma": wl.sigma, "diag": wl.diag,
                       "mean_fill": wl.mean_fill, "queries": n_q, "compact_keys": M, "l2": "inputs_larger_than_l2",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "tflops": world * flops / (ms_per_step * 1e-3) / 1e12,
            "attn_ms": attn_avg, "attn_ms_min": min(attn_ms), "build_kv_ms": build_avg, "build_kv_ms_min": min(build_ms),
            "attn_queries_per_sec": n_q / (attn_avg * 1e-3),
            "dense_attn_ms": dense_ms,
            "speedup_vs_dense": (dense_ms / attn_avg) if dense_ms else None,
            "frame_attn_ms": frame_ms,
            "frame_attn_tflops": 4.0 * n_q * wl.tokens_per_frame * H * d / (frame_ms * 1e-3) / 1e12,
            "roofline": {"bound": "tensor", "kernel": "global_attn_kernel", "achieved": achieved_tf, "peak": peak_tf,
                         "unit": "TFLOP/s", "frac": achieved_tf / peak_tf,
                         "traffic": NCU_TRAFFIC.get(wl.name, {}).get("global_attn_kernel"),
                         "peak_source": f"{peaks['source']} {'sustained' if long_run else 'burst'} bf16 matmul",
                         "frac_of_nominal_2250": achieved_tf / 2250.0,
                         "flop_per_launch": flops},
            "roofline_build_kv": {"bound": "hbm", "kernel": "build_kv_kernel", "achieved": build_gbs,
                                  "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": build_gbs / peaks["hbm_gbs"],
                                  "traffic": NCU_TRAFFIC.get(wl.name, {}).get("build_kv_kernel"),
                                  "bytes_per_launch": build_bytes,
                                  "peak_source": f"{peaks['source']} copy bandwidth"},
            "e2e": {"value": world * n_q * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": in_bytes,
                    "d2h_bytes_per_step": out_bytes, "steps": e2e_steps},
            "gpu_launches": 3 * args.steps,
            "clocks": clocks,
        }
        if world == 1 and not args.no_cpu_baseline:
            qps, ms, sample = time_oracle(wl, args.cpu_rows, 1, 0)
            line["cpu_baseline"] = {"value": qps, "unit": UNIT, "cores": _threads_used(), "kind": "oracle",
                                    "sample": sample, "ms": ms}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--cpu-rows", type=int, default=4096, help="query rows in the CPU-oracle baseline sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense (s = 1) comparison run")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    wl = inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
