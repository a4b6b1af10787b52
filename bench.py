"""Benchmark of the MSLT per-stage BERT training step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

One "step" is one pass of the whole hot path (frozen-prefix forward, trainable forward and
backward, MLM head and loss, Adam on the trainable slice) over one synthetic batch.  The path
does not shard: with N > 1 every rank runs an independent replica on its own batch (no
collective on the data path) and the aggregate throughput is reported; started without a
launcher, `--gpus N` starts its N processes itself.

Prints ONE JSON line (rank 0).  The headline is the BERT-Base stage configuration (9 frozen + 3
trainable layers); at one GPU the line also carries a `configs` record with every stage
configuration timed the same way, the contraction kernel's rate against both measured cuBLAS
figures, and the memory-bound kernels one at a time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2011_13635_b200 import inputs as I  # noqa: E402

METRIC = "sequences/sec per MSLT stage step"
UNIT = "sequences/s"


def measured_peaks():
    """Measured B200 peaks of this machine; the stated earlier measurement if the file is absent."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def step_flops(cfg: I.StageConfig) -> float:
    """Dense floating-point operations of one step (2*M*N*K per contraction)."""
    T, H, S, L, k = cfg.batch * cfg.seq, cfg.hidden, cfg.seq, cfg.layers, cfg.trainable
    R, V = cfg.batch * cfg.pred, cfg.vocab
    fwd_layer = 24.0 * T * H * H + 4.0 * T * S * H
    total = L * fwd_layer + k * 2 * fwd_layer
    if 0 < k < L:
        total -= 6.0 * T * H * H          # no input gradient below the frozen boundary
    total += 2.0 * R * H * H + 2.0 * R * H * V          # head forward
    total += 4.0 * R * H * H + 2.0 * R * H * V          # head backward
    if k == L:
        total += 2.0 * R * H * V                        # decoder weight gradient
    return total


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *exc):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons),
                    samples=len(sm))


def describe(cfg: I.StageConfig) -> dict:
    return dict(workload=f"{cfg.name}: {cfg.layers} layers ({cfg.frozen} frozen + {cfg.trainable} "
                         f"trainable), hidden {cfg.hidden}, heads {cfg.heads}, ffn {cfg.ffn}, vocab "
                         f"{cfg.vocab}, seq {cfg.seq}, batch {cfg.batch} per GPU, {cfg.pred} MLM slots",
                batch_per_gpu=cfg.batch, seq_len=cfg.seq, layers=cfg.layers, frozen=cfg.frozen,
                trainable=cfg.trainable, parallelism="replicas only (no collective)",
                l2="working set of one step (GBs of weights and activations) exceeds the 126 MB L2",
                launch="timed steps are replays of one mslt_step captured in a CUDA graph "
                       "(--no-graph launches them one by one)")


# ------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded sample of the workload
# ------------------------------------------------------------------------------------------------
def oracle_sample(cfg: I.StageConfig, n_seq: int):
    from oracle import mslt_oracle as O      # the one place bench.py may touch oracle/
    small = I.scaled(cfg, batch=n_seq)
    w = I.make_weights(small, variant="bench")
    m = O.MsltOracle(w, small.heads)
    m.set_trainable(small.trainable)
    return m, I.make_batch(small), small


def host_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return int(max(n)) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(cfg: I.StageConfig, n_seq: int, steps: int = 1, warmup: int = 0):
    m, batch, small = oracle_sample(cfg, n_seq)
    for _ in range(warmup):
        m.step(*batch)
    t0 = time.perf_counter()
    for _ in range(steps):
        m.step(*batch)
    dt = time.perf_counter() - t0
    return dict(value=n_seq * steps / dt, unit=UNIT, cores=host_threads(), kind="oracle",
                sample=f"{steps} step(s) of the float64 numpy oracle on {n_seq} of the {cfg.batch} "
                       f"sequences of the batch, full architecture ({dt:.1f} s)"), dt


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_seq = 2
    base, dt = cpu_baseline(cfg, n_seq, steps=args.steps, warmup=args.warmup)
    conf = describe(cfg)
    conf["sample"] = (f"each step is the oracle on {n_seq} of the {cfg.batch} sequences of the batch (full "
                      "architecture); value = those sequences per second")
    conf["launch"] = "numpy float64 on the host cores"
    line = dict(impl="reference", metric=METRIC, value=base["value"], unit=UNIT, n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=1e3 * dt / args.steps,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=conf, cpu_baseline=base,
                e2e=dict(value=base["value"], unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
def make_model(cfg, torch, stream=None):
    from paper_2011_13635_b200.binding import Mslt
    m = Mslt.from_config(cfg, stream=stream, max_trainable=cfg.trainable)
    m.set_params(I.make_weights(cfg, variant="bench"))
    m.mslt_set_trainable(cfg.trainable)
    m.mslt_set_optimizer(**I.ADAM_DEFAULTS)
    return m


def capture_step(m, dev, torch):
    """One mslt_step captured into a CUDA graph on the context's stream (after eager warm-up)."""
    g = torch.cuda.CUDAGraph()
    before = m.launch_count
    with torch.cuda.graph(g, stream=m.stream):
        m.mslt_step(*dev, sync=False)
    return g, m.launch_count - before


def time_steps(m, dev, torch, steps, warmup, sync_fn, use_graph=True):
    """(ms of the timed region, kernels launched in it).  The timed steps are replays of one
    captured step unless use_graph is off; events are recorded on the context's stream."""
    with torch.cuda.stream(m.stream):
        for _ in range(warmup):
            m.mslt_step(*dev, sync=False)
        sync_fn()
        graph, per_step = capture_step(m, dev, torch) if use_graph else (None, None)
        sync_fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        before = m.launch_count
        e0.record(m.stream)
        for _ in range(steps):
            if graph is not None:
                graph.replay()
            else:
                m.mslt_step(*dev, sync=False)
        e1.record(m.stream)
        sync_fn()
    launches = per_step * steps if graph is not None else m.launch_count - before
    return e0.elapsed_time(e1), launches, graph


def rank_seed(cfg, rank: int) -> int:
    """Every replica draws its own batch."""
    return I.config_seed(cfg) + 1000 * rank


def aggregate(ms_local: float, batch_per_rank: int, steps: int, world: int, dist=None, device="cpu"):
    """(max over ranks of the timed region in ms, whole-job sequences/s): replicas share nothing, so
    the job is as slow as its slowest rank and processes world * batch sequences per step."""
    import torch
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = float(t.item())
    return ms, batch_per_rank * world * steps / (ms * 1e-3)


# DRAM bytes (read + write) per launch of the contraction kernel from ncu captures of single launches
# of the four forward products of a BERT-Base layer (profiles/gemm_tc_kernel_frozen_layer_shapes_16384.md):
# QKV 47.7 MB, out-proj 53.1 MB, FFN1 73.6 MB, FFN2 144.2 MB; the bench line carries their mean, which
# holds for the BERT-Base configurations only.  None once the kernel changes.
GEMM_DRAM_BYTES_PER_LAUNCH = {"base": 79.7e6}


def gemm_peaks(peaks, clocks):
    """Which measured cuBLAS figure the step's contractions are held against: the burst figure when
    the sampled SM clock stayed near its maximum, the sustained one when it shows the power-capped
    regime (both fractions are printed either way)."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    capped = bool(mhz and mx and mhz < 0.9 * mx)
    return ("sustained" if capped else "burst"), peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]


def measure(cfg, args, torch, dist, world, rank, local, steps, warmup, headline):
    """Times `steps` steps of one configuration on this rank's GPU.  Returns the JSON record of the
    configuration (rank 0 adds the per-kernel passes) and, for the headline, the e2e figures."""
    def sync():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    host = [np.ascontiguousarray(a) for a in I.make_batch(cfg, seed=rank_seed(cfg, rank))]
    if cfg.varlen is None:
        host[1] = None
    pinned = [None if a is None else torch.from_numpy(a).pin_memory() for a in host]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        dev = [None if a is None else a.cuda(non_blocking=True) for a in pinned]
        m = make_model(cfg, torch, stream)
        loss0 = m.mslt_step(*dev)                       # also checks the device status word
    if not np.isfinite(loss0):
        raise RuntimeError("non-finite loss")

    dp = None
    if args.data_parallel:
        # every rank takes its own share of the global batch; the gradients of the trainable slice are
        # all-reduced bucket by bucket while the backward pass goes on (steps run eagerly)
        from paper_2011_13635_b200.data_parallel import DataParallelStep
        dp = DataParallelStep(m, dist if world > 1 else None)
    with ClockSampler(local) as clk:
        if dp is None:
            ms, launches, graph = time_steps(m, dev, torch, steps, warmup, sync, args.graph)
        else:
            graph = None
            with torch.cuda.stream(m.stream):
                for _ in range(warmup):
                    dp.step(*dev, read_loss=False)
                sync()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                before = m.launch_count
                e0.record(m.stream)
                for _ in range(steps):
                    dp.step(*dev, read_loss=False)
                e1.record(m.stream)
                sync()
            ms, launches = e0.elapsed_time(e1), m.launch_count - before
    loss_end = m.mslt_read_loss()
    ms, value = aggregate(ms, cfg.batch, steps, world, dist, "cuda" if world > 1 else "cpu")
    clocks = clk.summary()
    if dp is not None:
        args.dp_note = dict(buckets=len(dp.buckets), gradient_bytes_per_step=dp.bytes_exchanged,
                            of_all_parameters_bytes=4 * sum(int(np.prod(i["shape"])) for i in m.tensors().values()))
    rec = dict(ms_per_step=ms / steps, value=value, unit=UNIT, steps=steps, warmup=warmup,
               gpu_launches=int(launches), launches_per_step=launches / steps, clocks=clocks,
               loss=dict(first=loss0, last=loss_end), workspace_gb=m.workspace_bytes / 1e9,
               param_block_gb=m.param_bytes / 1e9)

    e2e = None
    if headline:
        # end to end: pinned host inputs copied in, loss read back, every step
        sync()
        with torch.cuda.stream(stream):
            t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            for _ in range(steps):
                for d_, p_ in zip(dev, pinned):
                    if d_ is not None:
                        d_.copy_(p_, non_blocking=True)
                if graph is not None:
                    graph.replay()
                    m.mslt_read_loss()
                elif dp is not None:
                    dp.step(*dev)
                else:
                    m.mslt_step(*dev)
            t1.record(stream)
            sync()
        _, e2e_value = aggregate(t0.elapsed_time(t1), cfg.batch, steps, world, dist, "cuda" if world > 1 else "cpu")
        e2e = dict(value=e2e_value, unit=UNIT,
                   h2d_bytes_per_step=int(sum(a.nbytes for a in host if a is not None)),
                   d2h_bytes_per_step=16)
    del graph

    if rank == 0:
        peaks = measured_peaks()
        # per-kernel pass: the same steps again with an event pair around every launch
        m.mslt_set_timing(2)
        m.mslt_get_kernel_profile()
        n_prof = max(1, min(steps, 5))
        with torch.cuda.stream(stream):
            for _ in range(n_prof):
                m.mslt_step(*dev, sync=False)
        torch.cuda.synchronize()
        prof = m.mslt_get_kernel_profile()
        rec["phases_ms"] = m.mslt_get_timings()
        m.mslt_set_timing(0)
        lin, att = prof["linear"], prof["attention"]
        lin_tflops = lin["work"] / (lin["ms"] * 1e-3) / 1e12 if lin["ms"] > 0 else 0.0
        if cfg.dtype == "bf16":
            regime, burst, sustained = gemm_peaks(peaks, clocks)
            peak = burst if regime == "burst" else sustained
            rec["roofline"] = dict(
                bound="tensor", kernel="gemm_tc_kernel (linear-layer products of the step)",
                achieved=lin_tflops, peak=peak, unit="TFLOP/s", frac=lin_tflops / peak,
                traffic=GEMM_DRAM_BYTES_PER_LAUNCH.get("base") if cfg.hidden == 768 and cfg.batch * cfg.seq == 16384 else None,
                peak_source=f"{peaks['source']}: cuBLAS bf16 8192^3, {regime} figure (median SM clock "
                            f"{clocks.get('sm_mhz')} of {clocks.get('sm_max_mhz')} MHz in the timed region)",
                frac_of_burst=lin_tflops / burst, frac_of_sustained=lin_tflops / sustained,
                peak_burst=burst, peak_sustained=sustained,
                launches_per_step=lin["launches"] / n_prof,
                avg_launch_us=1e3 * lin["ms"] / max(lin["launches"], 1),
                launch_us_x_sm_mhz=(1e3 * lin["ms"] / max(lin["launches"], 1)) * (clocks.get("sm_mhz") or 0.0),
                flops_per_step=lin["work"] / n_prof,
                share_of_step_time=lin["ms"] / n_prof / (ms / steps))
        else:
            rec["roofline"] = dict(bound="alu", kernel="gemm_simt_kernel", achieved=lin_tflops, peak=None,
                                   unit="TFLOP/s", frac=None, traffic=None,
                                   note="fp32 CUDA-core path of the small configuration: launch-bound")
        # attention: fused kernels (HBM-bound) where they apply, batched products otherwise
        rec["attention"] = dict(
            tflops=att["work"] / (att["ms"] * 1e-3) / 1e12 if att["ms"] > 0 else 0.0,
            ms_per_step=att["ms"] / n_prof, launches_per_step=att["launches"] / n_prof)
        rec["hbm_kernels"] = {
            k: dict(gbs=v["work"] / (v["ms"] * 1e-3) / 1e9,
                    frac_of_measured_copy=v["work"] / (v["ms"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    ms_per_step=v["ms"] / n_prof, launches_per_step=v["launches"] / n_prof)
            for k, v in prof.items() if k not in ("linear", "attention") and v["ms"] > 0}
        rec["step_tflops"] = step_flops(cfg) / (ms / steps * 1e-3) / 1e12
    m.close()
    del m
    torch.cuda.empty_cache()
    return rec, e2e


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    rec, e2e = measure(cfg, args, torch, dist, world, rank, local, args.steps, args.warmup, True)
    line = dict(metric=METRIC, value=rec["value"], unit=UNIT, n_gpus=world, steps=args.steps,
                warmup=args.warmup, ms_per_step=rec["ms_per_step"], higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype=cfg.dtype, data="synthetic", config=describe(cfg), e2e=e2e,
                gpu_launches=rec["gpu_launches"], clocks=rec["clocks"], loss=rec["loss"])
    if args.data_parallel:
        line["config"]["parallelism"] = (f"data parallel over {world} GPU(s): all-reduce (NCCL) of the trainable "
                                         "gradient slice only, bucket by bucket behind the backward pass")
        line["config"]["launch"] = "eager launches (the exchange hooks run on the host)"
        line["data_parallel"] = getattr(args, "dp_note", None)
    if rank == 0:
        for k in ("roofline", "attention", "phases_ms", "hbm_kernels", "step_tflops", "workspace_gb", "param_block_gb"):
            if k in rec:
                line[k] = rec[k]
        peaks = measured_peaks()
        if world == 1 and args.all_configs and not args.data_parallel:
            # every stage configuration, timed the same way (fewer steps); spec ratio from the two
            # BERT-Base ones
            short = max(10, args.steps // 4)
            per = {cfg.name: rec}
            for name in ("tiny", "base_stage", "base_full", "large_stage", "large_long"):
                if name in per:
                    continue
                per[name], _ = measure(I.CONFIGS[name], args, torch, dist, world, rank, local, short, 3, False)
            line["configs"] = {
                n: dict(ms_per_step=r["ms_per_step"], sequences_per_s=r["value"], steps=r["steps"],
                        launches_per_step=r["launches_per_step"], clocks=r["clocks"],
                        gemm_tflops=r["roofline"]["achieved"],
                        gemm_frac_of_burst=r["roofline"].get("frac_of_burst"),
                        gemm_frac_of_sustained=r["roofline"].get("frac_of_sustained"),
                        attention_ms=r["attention"]["ms_per_step"], phases_ms=r["phases_ms"],
                        step_tflops=r["step_tflops"], workspace_gb=r["workspace_gb"],
                        hbm_kernels={k: round(v["frac_of_measured_copy"], 3) for k, v in r["hbm_kernels"].items()})
                for n, r in per.items()}
            if "base_stage" in per and "base_full" in per:
                a, b = per["base_stage"]["ms_per_step"], per["base_full"]["ms_per_step"]
                line["stage_vs_full"] = dict(
                    staged_ms=a, full_ms=b, ratio=a / b,
                    note="step time of 9 frozen + 3 trainable layers over all 12 trainable, same shapes, "
                         "data and seed, one GPU, no communication")
        if world == 1 and cfg.dtype == "bf16" and cfg.seq <= 512 and args.isolated:
            # the memory-bound kernels one at a time, back to back on rotating buffers larger than L2:
            # no event pair per launch, so short kernels are not understated as in hbm_kernels
            from paper_2011_13635_b200 import op_bench
            with ClockSampler(local) as clk2:
                recs = op_bench.main(["--rows", str(cfg.batch * cfg.seq), "--hidden", str(cfg.hidden), "--ffn", str(cfg.ffn),
                                      "--heads", str(cfg.heads), "--seq", str(cfg.seq), "--batch", str(cfg.batch),
                                      "--iters", "20", "--only", "attention,ln,colsum,ce"], emit=None)
            line["hbm_kernels_alone"] = {
                r["kernel"]: dict(us=r["us"], gbs=r["gbs"], frac_of_measured_copy=r["gbs"] / peaks["hbm_gbs"],
                                  dram_bytes_ncu=HBM_DRAM_BYTES_NCU.get(r["kernel"]) if cfg.name.startswith("base") else None)
                for r in recs}
            line["hbm_kernels_alone"]["clocks"] = clk2.summary()
            torch.cuda.empty_cache()
        if world == 1:
            line["cpu_baseline"], _ = cpu_baseline(cfg, args.cpu_seqs)
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# DRAM bytes per launch of the memory-bound kernels at the op_bench sizes, from one-kernel ncu captures
# (profiles/memory_bound_kernels_base_16384.md); keys are op_bench's kernel names; read + write, outputs
# that were still in L2 at kernel end are not in the write counter.
HBM_DRAM_BYTES_NCU = {"layernorm": 25.2e6, "layernorm_bwd": 50.7e6, "colsum_hidden": 25.2e6, "colsum_ffn": 101.3e6,
                      "cross_entropy(sync)": 436.6e6, "attention_fused": 79.0e6,
                      "attention_fused_with_probs": 98.9e6, "attention_fused_backward": 191.3e6}


# ------------------------------------------------------------------------------------------------
# N replicas on N GPUs when started as a plain `python bench.py --gpus N`
# ------------------------------------------------------------------------------------------------
def free_port() -> int:
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def launch_replicas(n: int, argv):
    """Starts n copies of this script, one per GPU (RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* set as a
    launcher would), waits for them and returns the worst exit code.  Rank 0 prints the JSON line."""
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *argv], env=env))
    return max(abs(p.wait()) for p in procs)


def run_selftest_cpu(args):
    """The launcher and the aggregation without a GPU: every rank pretends its timed region took
    10 * (rank + 1) ms and the ranks meet over gloo."""
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo", init_method=f"tcp://{os.environ['MASTER_ADDR']}:{os.environ['MASTER_PORT']}",
                                rank=rank, world_size=world)
    cfg = I.CONFIGS[args.config]
    ms, value = aggregate(10.0 * (rank + 1), cfg.batch, args.steps, world, dist, "cpu")
    if rank == 0:
        print(json.dumps(dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps,
                              ms_per_step=ms / args.steps, selftest="cpu")))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="base_stage", choices=sorted(I.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-seqs", type=int, default=8, help="sequences in the oracle's timed sample")
    ap.add_argument("--no-ratio", "--one-config", dest="all_configs", action="store_false",
                    help="time only the headline configuration (no `configs` record, no staged : full ratio)")
    ap.add_argument("--selftest-cpu", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--data-parallel", action="store_true",
                    help="N workers train ONE model: gradients of the trainable slice are all-reduced (the default "
                         "is N independent replicas)")
    ap.add_argument("--no-isolated", dest="isolated", action="store_false",
                    help="skip the one-kernel-at-a-time bandwidth figures")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="launch every timed step eagerly instead of replaying one captured step")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = I.CONFIGS[args.config]
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # not under a launcher: start the replicas ourselves, one process per GPU
        sys.exit(launch_replicas(args.gpus, sys.argv[1:]))
    if args.selftest_cpu:
        run_selftest_cpu(args)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
