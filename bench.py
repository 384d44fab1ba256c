#!/usr/bin/env python
"""Benchmark of the subsampled global-attention hot path on B200.

One step = one pass of the whole path over one synthetic batch:
``avggt_build_kv`` (K/V compaction + mean-fill reduction) followed by
``avggt_global_attn`` (fused tcgen05 attention).  The default workload is the
largest single-GPU configuration, the VGGT-shaped layer at 800 frames (37x37
patch grid, 5 special tokens, 16 heads x 64, factor 9, diagonal + mean-fill on:
1,099,200 queries x 139,200 compact keys).  After the timed region the other
benchmark configurations (100 and 300 frames, the factor sweep at 333 frames)
are timed with a few launches each and reported in the same JSON line under
``configs``.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

With N > 1 (under torchrun) the frames of the workload are split over the ranks
(``sharded.FrameShardedAttention``: all-gather of the compact K/V, all-reduce of
the mean sums, then local attention), ``"scaling": "strong"``; ``--replicas``
runs N independent copies instead.  ``--impl reference`` times the fp64 CPU
oracle on the host cores on a bounded sample of the same workload.
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
# profiles/; None where no capture covers the workload.  Both kernels are captured on the 30-frame copy of the
# headline layer (profiles/*_vggt_n30_s9.md); their traffic is proportional to the frame count, so the 800-frame
# figures are those captures x 800/30.
_ATTN_N30_S9 = 0.275011072e9 + 0.067811584e9
_BUILD_N30_S9 = 0.168855296e9 + 0.009879808e9
NCU_TRAFFIC = {
    "vggt_n30_s9": {"global_attn_kernel": _ATTN_N30_S9, "build_kv_kernel": _BUILD_N30_S9},
    "vggt_n800_s9": {"global_attn_kernel": _ATTN_N30_S9 * 800 / 30, "build_kv_kernel": _BUILD_N30_S9 * 800 / 30},
}

METRIC = "subsampled_global_attn_queries_per_sec"
UNIT = "queries/s"
DEFAULT_WORKLOAD = "vggt_n800_s9"
# configurations reported under "configs" (a few launches each, outside the timed region)
SWEEP = ("vggt_n100_s4", "vggt_n300_s6", "vggt_n333_s1", "vggt_n333_s2", "vggt_n333_s4", "vggt_n333_s6", "vggt_n333_s9")
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
# query rows in the CPU-oracle sample, the same in the cpu_baseline leg and in the reference arm
CPU_SAMPLE_ROWS = 64


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


def time_oracle(wl, n_rows, steps, warmup, tensors=None, seed=0):
    """Times the oracle (as it stands) on ``n_rows`` sampled query rows per step.

    One step = ``global_attn_blocked`` on the sample, which compacts K/V and takes the mean over the whole
    workload (a cost that does not depend on the sample) and attends for the sampled rows (a cost linear in the
    rows: every row meets all compact keys).  The whole-workload rate is extrapolated accordingly:
    queries/s = N_q / (t_compaction + t_attention(sample) * N_q / n_rows), with the compaction timed once on its
    own.  -> (queries/s, measured ms per step, description of the sample)
    """
    orc, ocfg = _oracle_cfg(wl)
    if tensors is None:
        tensors = inputs.make_qkv(wl, seed=seed, device="cpu")
    Qh, Kh, Vh = (t.float().cpu().numpy() for t in tensors)
    rows = inputs.sample_rows(wl, n_rows).numpy()
    t0 = time.perf_counter()
    orc.build_kv(ocfg, Kh, Vh)
    t_build = time.perf_counter() - t0
    for _ in range(warmup):
        orc.global_attn_blocked(ocfg, Qh, Kh, Vh, rows[:8])
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        orc.global_attn_blocked(ocfg, Qh, Kh, Vh, rows)
        times.append(time.perf_counter() - t0)
    per_step = sum(times) / len(times)
    t_attn = max(per_step - t_build, 1e-9)
    whole = t_build + t_attn * wl.n_tokens / len(rows)
    sample = (f"{len(rows)} stratified query rows x all {wl.n_heads} heads x all compact keys of {wl.name} per step, "
              f"K/V compaction and mean of the whole workload included in every step ({t_build:.2f} s of "
              f"{per_step:.2f} s); rate extrapolated to all {wl.n_tokens} queries (attention cost is linear in the rows)")
    return wl.n_tokens / whole, per_step * 1e3, sample


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    qps, ms, sample = time_oracle(wl, CPU_SAMPLE_ROWS, max(1, args.steps), min(args.warmup, 1))
    line = {
        "impl": "reference", "metric": METRIC, "value": qps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": wl.name, "sample_rows_per_step": CPU_SAMPLE_ROWS},
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
    (a multi-GPU step is timed by its slowest rank).  One rank: the values themselves."""
    if world <= 1:
        return [float(v) for v in values]
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_throughput(units_all_ranks, ms_per_step):
    """Aggregate metric: the units all ranks processed per second of the slowest rank's step."""
    return units_all_ranks / (ms_per_step * 1e-3)


def fractions(tflops, peaks):
    """The three ways the attention rate is quoted: against the nominal dense bf16 peak and against the two
    measured cuBLAS figures (burst: a kernel timed alone; sustained: seconds of back-to-back work under the power cap)."""
    return {"frac_of_nominal_2250": tflops / NOMINAL_BF16_TFLOPS,
            "frac_of_measured_burst": tflops / peaks["bf16_tflops"],
            "frac_of_measured_sustained": tflops / peaks["bf16_tflops_sustained"]}


def build_bytes(n_q, M, H, d, mean_fill):
    """Algorithmic bytes of one compaction launch: every K/V row read once when the mean is taken (else only the
    retained rows), every retained row written once."""
    return 2.0 * (n_q + M) * H * d * 2 if mean_fill else 4.0 * M * H * d * 2


def _layer_for(P, wl, dev, sigma=None, diag=None, mean_fill=None):
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim,
                           wl.sigma if sigma is None else sigma, diag=wl.diag if diag is None else diag,
                           mean_fill=wl.mean_fill if mean_fill is None else mean_fill,
                           keep_first_frame=bool(wl.keep_first_frame))
    return P.SubsampledGlobalAttention(params, device=dev)


def input_logit_stats(wl, Q, K, n=1024):
    """What the synthetic inputs look like to the softmax (harness arithmetic, head 0, patch queries of frame 1):
    scaled logits of a query against its own key, against the key at the same grid position of frame 0 (the
    cross-view correspondence the input recipe plants) and against random other keys."""
    if wl.n_frames < 2 or wl.grid_h * wl.grid_w < 1:
        return None
    L = wl.tokens_per_frame
    g = torch.Generator(device=Q.device).manual_seed(7)
    slots = wl.n_special + torch.randint(0, wl.grid_h * wl.grid_w, (n,), generator=g, device=Q.device)
    rows = L + slots
    q = Q[rows, 0].float()
    scale = wl.head_dim ** -0.5
    own = (q * K[rows, 0].float()).sum(-1) * scale
    same = (q * K[slots, 0].float()).sum(-1) * scale
    other = (q * K[torch.randint(0, wl.n_tokens, (n,), generator=g, device=Q.device), 0].float()).sum(-1) * scale
    return {"own_key_mean": float(own.mean()), "same_position_other_frame_mean": float(same.mean()),
            "other_keys_mean": float(other.mean()), "other_keys_std": float(other.std()), "sampled_queries": n}


def time_config(P, wl, Q, K, V, O, dev, peaks, launches=3):
    """A few launches of the whole path on one configuration (inputs resident): per-kernel times from CUDA events."""
    stream = torch.cuda.current_stream(dev)
    layer = _layer_for(P, wl, dev)
    layer.forward(Q, K, V, out=O)
    layer.check_status()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(launches)]
    for e in ev:
        e[0].record(stream)
        layer.build_kv(K, V)
        e[1].record(stream)
        layer.attend(Q, K, V, out=O)
        e[2].record(stream)
    layer.check_status()
    b_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / launches
    a_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / launches
    n_q, M, H, d = wl.n_tokens, layer.M, wl.n_heads, wl.head_dim
    tf = 4.0 * n_q * M * H * d / (a_ms * 1e-3) / 1e12
    gbs = build_bytes(n_q, M, H, d, wl.mean_fill) / (b_ms * 1e-3) / 1e9
    rec = {"workload": wl.name, "queries": n_q, "compact_keys": M, "sigma": wl.sigma, "launches": launches,
           "attn_ms": a_ms, "build_kv_ms": b_ms, "queries_per_sec": n_q / ((a_ms + b_ms) * 1e-3), "tflops": tf,
           "build_kv_gbs": gbs, "build_kv_frac_of_measured_hbm": gbs / peaks["hbm_gbs"],
           "build_kv_frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS}
    rec.update(fractions(tf, peaks))
    del layer
    return rec


def sweep_configs(P, dev, peaks, skip=()):
    """The benchmark configurations other than the headline one: 100 and 300 frames, and the factor sweep at 333
    frames (one input set, five factors; s = 1 is the dense layer with both switches off)."""
    out = []
    cache_key, tensors = None, None
    for name in SWEEP:
        if name in skip:
            continue
        wl = inputs.WORKLOADS[name]
        if cache_key != wl.n_frames:
            tensors = None
            torch.cuda.empty_cache()
            Q, K, V = inputs.make_qkv(wl, seed=0, device=dev)
            tensors = (Q, K, V, torch.empty_like(Q))
            del Q, K, V
            cache_key = wl.n_frames
        out.append(time_config(P, wl, *tensors, dev, peaks))
    dense = {r["workload"]: r for r in out}.get("vggt_n333_s1")
    if dense:
        for r in out:
            if r["workload"].startswith("vggt_n333_") and r is not dense:
                r["speedup_vs_dense"] = dense["attn_ms"] / r["attn_ms"]
    return out


def run_ours(args, wl):
    import torch.distributed as dist

    import paper_2512_02541_b200 as P
    from paper_2512_02541_b200 import sharded

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    elif args.shard:
        # the frame-sharded path with a group of one rank (no peer, same calls): a check of that path on one GPU
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1, device_id=dev)
    shard_mode = (world > 1 and not args.replicas) or (world == 1 and args.shard)
    stream = torch.cuda.current_stream(dev)
    H, d = wl.n_heads, wl.head_dim

    if shard_mode:
        # the frames of ONE problem split over the ranks: the same seeded tensors everywhere, each rank keeps its rows
        f0, f1 = sharded.shard_frames(wl.n_frames, world, rank)
        Q, K, V = inputs.make_qkv(wl, seed=0, device=dev, frame_range=(f0, f1))
        layer = sharded.FrameShardedAttention(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, H, d, wl.sigma,
                                              diag=wl.diag, mean_fill=wl.mean_fill,
                                              keep_first_frame=bool(wl.keep_first_frame), device=dev)
        M = layer.n_kept_total
        units_all = wl.n_tokens               # strong scaling: the whole problem is the unit count at every N
        n_q_local = Q.shape[0]
    else:
        Q, K, V = inputs.make_qkv(wl, seed=rank, device=dev)
        layer = _layer_for(P, wl, dev)
        M = layer.M
        units_all = world * wl.n_tokens
        n_q_local = wl.n_tokens
    O = torch.empty_like(Q)
    logits = input_logit_stats(wl, Q, K) if (rank == 0 and not shard_mode) else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(args.warmup):
        layer.forward(Q, K, V, out=O)
    layer.check_status()

    # ---- device-resident timing: K steps, events on the launching stream
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    barrier()
    sampler = ClockSampler(dev) if rank == 0 else None
    time.sleep(0.15 if sampler else 0)
    barrier()
    for i in range(args.steps):
        ev[i][0].record(stream)
        layer.build_kv(K, V)
        ev[i][1].record(stream)
        if shard_mode:
            layer.exchange()
        ev[i][2].record(stream)
        layer.attend(Q, K, V, out=O)
        ev[i][3].record(stream)
    barrier()
    clocks = sampler.stop() if sampler else None
    layer.check_status()
    total_ms = ev[0][0].elapsed_time(ev[-1][3])
    build_ms = [e[0].elapsed_time(e[1]) for e in ev]
    exch_ms = [e[1].elapsed_time(e[2]) for e in ev]
    attn_ms = [e[2].elapsed_time(e[3]) for e in ev]

    frame_ms = dense_ms = None
    if not shard_mode:
        # ---- outside the timed region: the same tokens through frame attention (Sec. 4.2), for the report
        fe = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        n_frame = min(args.steps, 5)
        layer.frame_attend(Q, K, V, out=O)
        barrier()
        fe[0].record(stream)
        for _ in range(n_frame):
            layer.frame_attend(Q, K, V, out=O)
        fe[1].record(stream)
        barrier()
        layer.check_status()
        frame_ms = fe[0].elapsed_time(fe[1]) / n_frame

        # ---- outside the timed region: the dense layer (s = 1, both switches off) on the same tokens, the GPU
        #      reference the metric is quoted against.  One launch: at 800 frames it runs for seconds.
        if wl.sigma != 1 and not args.no_dense:
            dense = _layer_for(P, wl, dev, sigma=1, diag=0, mean_fill=0)
            dense.build_kv(K, V)
            barrier()
            de = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            de[0].record(stream)
            dense.attend(Q, K, V, out=O)
            de[1].record(stream)
            barrier()
            dense.check_status()
            dense_ms = de[0].elapsed_time(de[1])
            del dense
            torch.cuda.empty_cache()

    # ---- outside the timed region: the K/V projection with the compaction in its epilogue (model dimension
    #      H * d, random weights), against which the separate compaction pass can be weighed
    proj = None
    if not shard_mode and not args.no_projection:
        C = H * d
        gen = torch.Generator(device=dev).manual_seed(1234)
        X = torch.randn((wl.n_tokens, C), generator=gen, device=dev, dtype=torch.float32).bfloat16()
        Wk = (torch.randn((C, C), generator=gen, device=dev) * C ** -0.5).bfloat16()
        Wv = (torch.randn((C, C), generator=gen, device=dev) * C ** -0.5).bfloat16()
        pws = torch.zeros((P.avggt_project_workspace_bytes(layer.params, C),), dtype=torch.uint8, device=dev)
        Kp, Vp = torch.empty_like(K), torch.empty_like(V)

        def proj_call():
            P.avggt_project_build_kv(layer.params, C, X, Wk, Wv, None, None, Kp, Vp, layer.Kc, layer.Vc, layer.idx,
                                     layer.kmean, layer.vmean, pws, pws.numel(), stream.cuda_stream)

        proj_call()
        barrier()
        P.avggt_check_status(pws)
        pe = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        n_proj = 3
        pe[0].record(stream)
        for _ in range(n_proj):
            proj_call()
        pe[1].record(stream)
        barrier()
        proj_ms = pe[0].elapsed_time(pe[1]) / n_proj
        proj_flops = 2.0 * 2.0 * wl.n_tokens * C * C
        proj = {"ms": proj_ms, "tflops": proj_flops / (proj_ms * 1e-3) / 1e12, "model_dim": C,
                "writes_full_k_v": True}
        del X, Wk, Wv, Kp, Vp, pws
        layer.build_kv(K, V)                      # the layer's compact arrays back to the benchmark's K and V
        torch.cuda.empty_cache()

    # ---- end to end through the public API with host buffers: every step copies the step's Q, K, V from pinned
    #      host memory to the device and the output back
    e2e_steps = max(1, min(args.steps, 3))
    hQ, hK, hV = (t.cpu().pin_memory() for t in (Q, K, V))
    hO = torch.empty_like(hQ).pin_memory()
    dQ, dK, dV = (torch.empty_like(t) for t in (Q, K, V)) if shard_mode else (None, None, None)

    def e2e_step():
        if shard_mode:
            dQ.copy_(hQ, non_blocking=True); dK.copy_(hK, non_blocking=True); dV.copy_(hV, non_blocking=True)
            layer.forward(dQ, dK, dV, out=O)
            hO.copy_(O, non_blocking=True)
        else:
            # the layer's host-buffer entry: K and V first, Q in groups of frames under the attention of the group before
            layer.forward_host(hQ, hK, hV, hO)

    e2e_step()
    barrier()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    s1.record(stream)
    barrier()
    e2e_ms = s0.elapsed_time(s1)
    layer.check_status()
    in_bytes = 3 * Q.numel() * Q.element_size()
    out_bytes = O.numel() * O.element_size()
    cpu_tensors = (hQ, hK, hV) if (world == 1 and not args.no_cpu_baseline) else None
    del dQ, dK, dV, hO, hQ, hK, hV

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dev if world > 1 else "cpu", world)
    exch_avg = max_over_ranks([sum(exch_ms) / len(exch_ms)], dev if world > 1 else "cpu", world)[0]

    if rank == 0:
        peaks = _peaks()
        ms_per_step = total_ms / args.steps
        value = whole_job_throughput(units_all, ms_per_step)
        flops = 4.0 * n_q_local * M * H * d               # of this rank's attention launch
        attn_avg = sum(attn_ms) / len(attn_ms)
        build_avg = sum(build_ms) / len(build_ms)
        achieved_tf = flops / (attn_avg * 1e-3) / 1e12
        # denominator: the burst figure for a kernel timed alone in a short run, the sustained one when the timed
        # region is seconds of back-to-back work under the power cap
        long_run = total_ms > 2000.0
        peak_tf = peaks["bf16_tflops_sustained"] if long_run else peaks["bf16_tflops"]
        M_local = layer.kept[rank] if shard_mode else M
        bbytes = build_bytes(n_q_local, M_local, H, d, wl.mean_fill)
        build_gbs = bbytes / (build_avg * 1e-3) / 1e9
        if shard_mode:
            par, scaling = f"{world} ranks, {wl.n_frames} frames split {[b - a for a, b in layer.ranges]}", "strong"
        elif world > 1:
            par, scaling = "replicas only", "weak"
        else:
            par, scaling = "single GPU", "weak"
        roof = {"bound": "tensor", "kernel": "global_attn_kernel", "achieved": achieved_tf, "peak": peak_tf,
                "unit": "TFLOP/s", "frac": achieved_tf / peak_tf,
                "traffic": NCU_TRAFFIC.get(wl.name, {}).get("global_attn_kernel") if not shard_mode else None,
                "peak_source": f"{peaks['source']} {'sustained' if long_run else 'burst'} bf16 matmul",
                "flop_per_launch": flops}
        roof.update(fractions(achieved_tf, peaks))
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": scaling, "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "n_frames": wl.n_frames, "grid": [wl.grid_h, wl.grid_w],
                       "n_special": wl.n_special, "heads": H, "head_dim": d, "sigma": wl.sigma, "diag": wl.diag,
                       "mean_fill": wl.mean_fill, "queries": wl.n_tokens, "compact_keys": M,
                       "l2": "inputs_larger_than_l2", "parallelism": par, "input_logits": logits},
            "tflops": 4.0 * units_all * M * H * d / (ms_per_step * 1e-3) / 1e12,
            "attn_ms": attn_avg, "attn_ms_min": min(attn_ms), "build_kv_ms": build_avg, "build_kv_ms_min": min(build_ms),
            "exchange_ms": exch_avg if shard_mode else None,
            "attn_queries_per_sec": n_q_local / (attn_avg * 1e-3),
            "dense_attn_ms": dense_ms,
            "speedup_vs_dense": (dense_ms / attn_avg) if dense_ms else None,
            "frame_attn_ms": frame_ms,
            "frame_attn_tflops": (4.0 * n_q_local * wl.tokens_per_frame * H * d / (frame_ms * 1e-3) / 1e12) if frame_ms else None,
            "project_build_kv": proj,
            "roofline": roof,
            "roofline_build_kv": {"bound": "hbm", "kernel": "build_kv_kernel", "achieved": build_gbs,
                                  "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": build_gbs / peaks["hbm_gbs"],
                                  "frac_of_nominal_8000": build_gbs / NOMINAL_HBM_GBS,
                                  "traffic": NCU_TRAFFIC.get(wl.name, {}).get("build_kv_kernel") if not shard_mode else None,
                                  "bytes_per_launch": bbytes,
                                  "peak_source": f"{peaks['source']} copy bandwidth"},
            "e2e": {"value": units_all * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": out_bytes, "steps": e2e_steps},
            "gpu_launches": (5 if shard_mode else 3) * args.steps,
            "clocks": clocks,
        }
        if cpu_tensors is not None:
            qps, ms, sample = time_oracle(wl, CPU_SAMPLE_ROWS, 1, 0, tensors=cpu_tensors)
            line["cpu_baseline"] = {"value": qps, "unit": UNIT, "cores": _threads_used(), "kind": "oracle",
                                    "sample": sample, "ms": ms}
        cpu_tensors = None
        if world == 1 and not args.no_sweep:
            del Q, K, V, O, layer
            torch.cuda.empty_cache()
            line["configs"] = sweep_configs(P, dev, peaks, skip=(wl.name,))
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
    if dist.is_initialized():
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-dense", action="store_true", help="skip the dense (s = 1) comparison run")
    ap.add_argument("--no-sweep", action="store_true", help="skip the per-configuration report")
    ap.add_argument("--no-projection", action="store_true", help="skip the fused projection + compaction timing")
    ap.add_argument("--shard", action="store_true",
                    help="with one GPU: run the frame-sharded path with a one-rank group (checks that path; not the default)")
    ap.add_argument("--replicas", action="store_true",
                    help="with N > 1: N independent copies of the problem instead of one problem split by frames")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    wl = inputs.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
