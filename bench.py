#!/usr/bin/env python
"""Benchmark of the Pruned-CTC head-and-loss hot path (Algorithm 1, forward + backward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c4] [--impl ours|reference]

A step is one complete pruned_ctc_fwd_bwd call (subset, stacking, chunked
projection + online LSE, subset log-probs, alignment DP, chunked backward) on one
seeded synthetic batch that stays resident in HBM.  Rank 0 prints one JSON line.
With N > 1 (launched by torch.distributed.run) every rank works on its own batch
of the same shape; the path has no exchange step, so there is no collective in
the timed region (weak scaling).

`--impl reference` times the float64 CPU oracle on the host cores instead, on a
bounded sample of the same workload.
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_33645_b200 import workloads as wl  # noqa: E402

METRIC = "pruned_ctc_fwd_bwd_frames_per_s"
UNIT = "frames/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(source="measured", hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]))
    return dict(source="fallback", hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0)


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled every 200 ms while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 200):
        self.gpu = gpu_index
        self.period_ms = int(period_ms)
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", str(self.period_ms),
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        # samples under load: the upper half by power draw
        if sm:
            order = np.argsort(power)[len(power) // 2:]
            load_sm = [sm[i] for i in order]
        else:
            load_sm = []
        return dict(sm_mhz=statistics.median(load_sm) if load_sm else None,
                    sm_max_mhz=max(smax) if smax else None,
                    power_w_max=max(power) if power else None,
                    samples=len(sm), reasons=sorted(reasons))


def rank_seed(cfg, rank: int) -> int:
    """Every rank draws its own utterances: same configuration, different seed."""
    return cfg.seed + 7919 * rank


def reduce_over_ranks(ms: float, frames: float, flops: float, device=None):
    """Whole-job figures: time is the max over ranks, frames and FLOPs are summed.

    Works on any initialised process group (NCCL on the GPU machine, gloo in the CPU tests); without
    one it returns its arguments.
    """
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms, frames, flops
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    s = torch.tensor([frames, flops], dtype=torch.float64, device=device)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    return float(t[0].item()), float(s[0].item()), float(s[1].item())


def _traced_call(binding, hidden, W, bias_dev, targets, il, tl, batch, res, trace, call):
    binding.pruned_ctc_fwd_bwd(hidden, W, bias_dev, targets, il, tl, batch.blank, workspace=res["workspace"], out=res,
                               trace=trace, **call)
    return trace


def time_config(binding, torch, dev, cfg, beam, steps, warmup, peaks, frozen_head=False, promise_k=False):
    """Device-resident timing of one configuration with the protocol of the headline run: inputs in HBM,
    `warmup` untimed calls, `steps` timed calls between two CUDA events on the launching stream.
    frozen_head: dW is skipped (6 M D V FLOPs).  promise_k: max_K = the number of selected classes, counted on
    the host as a data loader would."""
    batch = wl.make_batch(cfg)
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    hidden = torch.from_numpy(batch.hidden).to(tdt).to(dev)
    W = torch.from_numpy(batch.W).to(tdt).to(dev)
    targets = torch.from_numpy(batch.targets).to(dev)
    il, tl = batch.input_lengths, batch.target_lengths
    M, D, V, N = batch.M, cfg.D, cfg.V, cfg.N
    dt = binding.PCTC_BF16 if cfg.dtype == "bf16" else binding.PCTC_FP32
    max_K = 0
    if promise_k:
        max_K = 1 + int(np.unique(np.concatenate([batch.targets[n, : tl[n]] for n in range(N)])).size)
    prob = binding.make_problem(N, batch.T, D, V, dt, batch.blank, beam, 0, batch.targets.shape[1], max_K=max_K)
    ws_bytes = binding.workspace_bytes(prob, il, tl)
    chunk, nchunks = binding.chunk_width(prob, il, tl)
    half = binding.make_problem(N, batch.T, D, max(8, V // 2 // 8 * 8), dt, batch.blank, beam, chunk,
                                batch.targets.shape[1], max_K=max_K)
    ws_half = binding.workspace_bytes(half, il, tl)
    kw = dict(beam=beam, skip_dW=frozen_head, max_K=max_K)
    res = binding.pruned_ctc_fwd_bwd(hidden, W, None, targets, il, tl, batch.blank, check_status=True, **kw)
    for _ in range(max(0, warmup - 1)):
        binding.pruned_ctc_fwd_bwd(hidden, W, None, targets, il, tl, batch.blank, workspace=res["workspace"], out=res,
                                   **kw)
    trace = binding.Trace(binding.Trace.capacity_for(V, chunk))
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for s in range(steps):
        binding.pruned_ctc_fwd_bwd(hidden, W, None, targets, il, tl, batch.blank, workspace=res["workspace"], out=res,
                                   trace=trace if s == steps - 1 else None, **kw)
    ev1.record()
    torch.cuda.synchronize()
    if binding.workspace_status(res["workspace"]) != 0:
        raise SystemExit("device status word set while timing " + cfg.name)
    ms = ev0.elapsed_time(ev1) / steps
    dp_ms = sum(t for kind, t in trace.spans() if kind >= 0 and binding.PHASES[kind] == "dp")
    flops = (6.0 if frozen_head else 8.0) * M * D * V
    tfl = flops / (ms * 1e-3) / 1e12
    out = dict(workload=cfg.name, dtype=cfg.dtype, beam=beam, frozen_head=frozen_head, flops_per_step=flops, M_frames=M, K_selected=int(res["K"].item()), D=D, V=V,
               chunk=chunk, steps=steps, warmup=warmup, ms_per_step=round(ms, 4), frames_per_s=round(M / (ms * 1e-3), 1),
               tflops=round(tfl, 2),
               frac_of_bf16_peak=(dict(burst=round(tfl / peaks["bf16_tflops"], 4),
                                       sustained=round(tfl / peaks["bf16_tflops_sustained"], 4))
                                  if cfg.dtype == "bf16" else None),
               dp_ms=round(dp_ms, 4), workspace_bytes=ws_bytes, workspace_bytes_at_half_V=ws_half,
               one_fp32_MxV_array=4 * M * V,
               l2=("inputs larger than L2" if W.numel() * W.element_size() > (126 << 20) else
                   "inputs smaller than L2: L2 flushed by nothing, latency-bound case"))
    del res, hidden, W, targets, trace
    torch.cuda.empty_cache()
    return out


def print_table(path: str) -> int:
    """Markdown rows of the `all_configs` block of a saved bench line."""
    line = None
    with open(path) as f:
        for x in f:
            if x.startswith("{") and '"all_configs"' in x:
                line = json.loads(x)
    if line is None:
        print("no bench line with an all_configs block in", path)
        return 1
    print("| config | M | K | chunk | ms/step | frames/s | TFLOP/s | of measured burst / sustained bf16 peak "
          "| DP ms | workspace (at V/2; one fp32 M x V array) |")
    print("|---|---|---|---|---|---|---|---|---|---|")
    for r in line["all_configs"]:
        if "error" in r:
            print("| %s | failed: %s |" % (r["workload"], r["error"]))
            continue
        name = r["workload"] + (", beam %g" % r["beam"] if r["beam"] else "") + (
            ", frozen head (6MDV)" if r.get("frozen_head") else "")
        fr = r["frac_of_bf16_peak"]
        frac = "n/a (fp32 FMA path)" if fr is None else "%.1f%% / %.1f%%" % (100 * fr["burst"], 100 * fr["sustained"])
        print("| %s | %d | %d | %d | %.3f | %.0fk | %.1f | %s | %.2f | %.2f GB (%.2f GB; %.2f GB) |" % (
            name, r["M_frames"], r["K_selected"], r["chunk"], r["ms_per_step"], r["frames_per_s"] / 1e3, r["tflops"],
            frac, r["dp_ms"], r["workspace_bytes"] / 1e9, r["workspace_bytes_at_half_V"] / 1e9,
            r["one_fp32_MxV_array"] / 1e9))
    return 0


def load_traffic(cfg_name: str, chunk: int):
    """DRAM bytes of the dominant kernel per step for this workload and chunk width, if a capture of it is
    on record (a small JSON written beside the summary of that ncu capture)."""
    path = os.path.join(ROOT, "profiles", "umma_gemm_dram_traffic.json")
    try:
        with open(path) as f:
            table = json.load(f)
    except (OSError, ValueError):
        return None
    for row in table.get("captures", []):
        if row.get("workload") == cfg_name and int(row.get("chunk", -1)) == int(chunk):
            return dict(bytes_per_step=row["bytes_per_step"], launches_per_step=row["launches_per_step"],
                        bytes_per_launch_avg=row["bytes_per_step"] / row["launches_per_step"],
                        source=row.get("source", "ncu dram__bytes_read.sum + dram__bytes_write.sum"))
    return None


def oracle_sample(batch, frames: int):
    """The first `frames` frames of utterance 0 with a proportional prefix of its labels."""
    n = 0
    Tn = int(batch.input_lengths[n])
    f = min(frames, Tn)
    u = max(1, int(batch.target_lengths[n]) * f // Tn // 2)
    return (batch.hidden[n:n + 1, :f].astype(np.float64), batch.targets[n:n + 1, :max(u, 1)],
            np.array([f], dtype=np.int32), np.array([u], dtype=np.int32))


def time_oracle(batch, W64, frames: int):
    from oracle import pruned_ctc_oracle as O
    H, y, il, tl = oracle_sample(batch, frames)
    t0 = time.perf_counter()
    out = O.pruned_ctc_reference(H, W64, None, y, il, tl, batch.blank)
    dt = time.perf_counter() - t0
    assert np.isfinite(out["loss"]).all()
    return dt, int(il[0])


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return len(os.sched_getaffinity(0))


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    batch = wl.make_batch(cfg)
    W64 = batch.W.astype(np.float64)
    total_steps = args.steps + args.warmup
    budget = 150.0 / max(1, total_steps)
    dt8, _ = time_oracle(batch, W64, 8)          # calibration (also the first touch of the BLAS)
    frames = 8
    for cand in (16, 32, 64, 128, 256, 512, 1024, 2048):
        # the per-call cost is a fixed O(V D) part plus a part linear in the frames
        if dt8 * (0.6 + 0.4 * cand / 8.0) <= budget:
            frames = cand
    for _ in range(args.warmup):
        time_oracle(batch, W64, frames)
    times = []
    t_all = time.perf_counter()
    for _ in range(args.steps):
        dt, f = time_oracle(batch, W64, frames)
        times.append(dt)
    total = time.perf_counter() - t_all
    value = frames * args.steps / total
    cores = blas_threads()
    sample = (f"oracle fwd+bwd on the first {frames} frames of utterance 0 of {cfg.name} "
              f"(full V={cfg.V}, D={cfg.D}, full dW); W pre-widened to float64 outside the timed steps")
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=1000.0 * total / args.steps, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=cfg.name, N=cfg.N, D=cfg.D, V=cfg.V, sample_frames=frames),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="c4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--beam", type=float, default=0.0)
    ap.add_argument("--chunk", type=int, default=0)
    ap.add_argument("--vocab", type=int, default=0, help="override V of the configuration (vocabulary sweep)")
    ap.add_argument("--promise-k", action="store_true",
                    help="pass max_K = the number of selected classes, counted on the host as a data loader "
                         "would (default for the g* grid workloads)")
    ap.add_argument("--frozen-head", action="store_true",
                    help="skip dW (the LLM-CTC setting): 6 M D V FLOPs per step instead of 8")
    ap.add_argument("--allreduce-dw", action="store_true",
                    help="data-parallel training step: dW of every step is summed over the ranks, one NCCL "
                         "all-reduce per vocabulary chunk on a communication stream (off by default: the "
                         "head-and-loss path itself has no exchange step)")
    ap.add_argument("--bias", action="store_true", help="give the head a bias (dbias is then part of the step)")
    ap.add_argument("--dense-head", action="store_true",
                    help="also time the three library GEMMs of a dense bf16 head that holds its [M, V] logits "
                         "(forward, dX, dW: 6 M D V FLOPs) on the same shapes, as a yardstick for the time ratio")
    ap.add_argument("--all-configs", dest="all_configs", action="store_true", default=None,
                    help="after the headline region, time every configuration (c1, c2, c3, c4, c5 without a beam "
                         "and at beams 8 and 16) with the same protocol and fewer steps, and report them in an "
                         "`all_configs` block (default: on for the default workload on one GPU)")
    ap.add_argument("--no-all-configs", dest="all_configs", action="store_false")
    ap.add_argument("--all-steps", type=int, default=10, help="timed steps per configuration of --all-configs")
    ap.add_argument("--lib-variant", default="",
                    help="time a measurement build of the library (build.VARIANTS, probe_*): one part of the "
                         "tensor-core kernel is knocked out, so the results are wrong on purpose and the line "
                         "is marked invalid; it shows what the step is bound by")
    ap.add_argument("--clock-ms", type=int, default=200, help="sampling period of the clock record")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-frames", type=int, default=1024)
    ap.add_argument("--table", default="", help="print the all_configs block of a saved bench line as a table and exit")
    args = ap.parse_args()
    if args.table:
        return print_table(args.table)
    cfg = wl.CONFIGS[args.config]
    if args.vocab:
        cfg = wl.reduced(cfg, V=args.vocab, name=f"{cfg.name}-V{args.vocab}")
    if cfg.name.startswith("g"):
        args.promise_k = True

    if args.impl == "reference":
        return run_reference(args, cfg)

    import torch
    from paper_2609_33645_b200 import binding, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU implementation")
    local_dev = local_rank % torch.cuda.device_count()
    torch.cuda.set_device(local_dev)
    dev = torch.device("cuda", local_dev)
    # NCCL over NVLink for the timing reduction; PCTC_BENCH_BACKEND=gloo lets several ranks share one
    # GPU when the multi-rank code path is exercised on a single-GPU machine
    backend = os.environ.get("PCTC_BENCH_BACKEND", "nccl")
    red_dev = dev if backend == "nccl" else None
    if world > 1 or args.allreduce_dw:
        import torch.distributed as dist
        if world == 1:
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", str(29400 + os.getpid() % 500))
            dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
        elif backend == "nccl":
            dist.init_process_group("nccl", device_id=dev)
        else:
            dist.init_process_group(backend)
    if rank == 0:
        build.build()
        if args.lib_variant:
            build.build_variant(args.lib_variant)
    if world > 1:
        dist.barrier()
    if args.lib_variant:
        binding.LIB_PATH = build.variant_path(args.lib_variant)
        if args.lib_variant.startswith("probe_"):
            args.e2e_steps, args.all_configs, args.no_cpu_baseline = 0, False, True
    binding.load()
    peaks = load_peaks()

    # ---- the batch: every rank its own utterances, same shape distribution ----
    batch = wl.make_batch(cfg, seed=rank_seed(cfg, rank), with_bias=args.bias)
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    h_hidden = torch.from_numpy(batch.hidden).to(tdt).pin_memory()
    h_W = torch.from_numpy(batch.W).to(tdt).pin_memory()
    h_targets = torch.from_numpy(batch.targets).pin_memory()
    hidden = h_hidden.to(dev, non_blocking=True)
    W = h_W.to(dev, non_blocking=True)
    targets = h_targets.to(dev, non_blocking=True)
    h_bias = None if batch.bias is None else torch.from_numpy(batch.bias).to(tdt).pin_memory()
    bias_dev = None if h_bias is None else h_bias.to(dev, non_blocking=True)
    il, tl = batch.input_lengths, batch.target_lengths
    M, D, V, N = batch.M, cfg.D, cfg.V, cfg.N
    flops_per_step = (6.0 if args.frozen_head else 8.0) * M * D * V

    max_K_pre = 0
    if args.promise_k:
        max_K_pre = 1 + int(np.unique(np.concatenate([batch.targets[n, : tl[n]] for n in range(N)])).size)
    prob = binding.make_problem(N, batch.T, D, V, binding.PCTC_BF16 if cfg.dtype == "bf16" else binding.PCTC_FP32,
                                batch.blank, args.beam, args.chunk, batch.targets.shape[1], max_K=max_K_pre)
    ws_bytes = binding.workspace_bytes(prob, il, tl)
    chunk, nchunks = binding.chunk_width(prob, il, tl)     # the library's default unless --chunk is given
    call = dict(beam=args.beam, chunk=chunk)
    max_K = 0
    if args.promise_k:
        toks = np.concatenate([batch.targets[n, : tl[n]] for n in range(N)])
        max_K = 1 + int(np.unique(toks).size)
    dev_call = dict(call, skip_dW=args.frozen_head, max_K=max_K)

    res = binding.pruned_ctc_fwd_bwd(hidden, W, bias_dev, targets, il, tl, batch.blank, check_status=True, **dev_call)
    torch.cuda.synchronize()
    if args.lib_variant.startswith("probe_"):
        # a knocked-out store leaves its buffer as it finds it: give the consumers values of the usual size
        # to multiply (all-zero operands would draw less power and flatter the measurement)
        ws = res["workspace"]
        ws[: ws.numel() // 2 * 2].view(torch.bfloat16).normal_(0.0, 1e-5)
        torch.cuda.synchronize()
    for _ in range(max(0, args.warmup - 1)):
        res = binding.pruned_ctc_fwd_bwd(hidden, W, bias_dev, targets, il, tl, batch.blank,
                                         workspace=res["workspace"], out=res, **dev_call)
    torch.cuda.synchronize()

    traces = [binding.Trace(binding.Trace.capacity_for(V, chunk)) for _ in range(args.steps)]
    sum_dW = args.allreduce_dw and not args.frozen_head
    if sum_dW:
        from paper_2609_33645_b200 import data_parallel as dp
        comm = torch.cuda.Stream(dev)
        dw_rows = dp.chunk_rows(V, chunk)
        for _ in range(2):                       # NCCL sets up its channels at the first collective
            dp.allreduce_rows(res["dW"], dw_rows, dp.dw_ready_events(
                _traced_call(binding, hidden, W, bias_dev, targets, il, tl, batch, res, traces[0], dev_call)), comm_stream=comm)
        torch.cuda.synchronize()
    sampler = ClockSampler(local_dev, args.clock_ms)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ev0.record()
    for s in range(args.steps):
        binding.pruned_ctc_fwd_bwd(hidden, W, bias_dev, targets, il, tl, batch.blank, workspace=res["workspace"],
                                   out=res, trace=traces[s], **dev_call)
        if sum_dW:
            dp.allreduce_rows(res["dW"], dw_rows, dp.dw_ready_events(traces[s]), comm_stream=comm)
    ev1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = ev0.elapsed_time(ev1)
    status = binding.workspace_status(res["workspace"])
    if status != 0:
        raise SystemExit(f"device status word {status}: a bounded wait gave up")
    ms_total, frames_all, flops_all = reduce_over_ranks(ms_total, float(M), flops_per_step, red_dev)
    ms_per_step = ms_total / args.steps
    value = frames_all / (ms_per_step * 1e-3)

    # ---- per-phase device time from the event timeline of the same timed steps ----
    phase_ms = {name: 0.0 for name in binding.PHASES}
    phase_cnt = {name: 0 for name in binding.PHASES}
    for tr in traces:
        for kind, ms in tr.spans():
            if kind < 0:
                continue          # gap between the main and the auxiliary stream
            phase_ms[binding.PHASES[kind]] += ms
            phase_cnt[binding.PHASES[kind]] += 1
    for k in phase_ms:
        phase_ms[k] /= args.steps
    gemm_phases = ("lse", "dlogits", "dh", "dw")
    gemm_ms = sum(phase_ms[k] for k in gemm_phases)
    gemm_launches = sum(phase_cnt[k] for k in gemm_phases) // args.steps
    achieved_tflops = flops_per_step / (gemm_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    per_kernel = {}
    split_flops = dict(lse=2.0 * M * D * V, dlogits=2.0 * M * D * V, dh=2.0 * M * D * V, dw=2.0 * M * D * V)
    if args.frozen_head:
        gemm_phases = ("lse", "dlogits", "dh")
        gemm_ms = sum(phase_ms[k] for k in gemm_phases)
        achieved_tflops = flops_per_step / (gemm_ms * 1e-3) / 1e12
    for k in gemm_phases:
        per_kernel[k] = dict(ms=round(phase_ms[k], 4), launches=phase_cnt[k] // args.steps,
                             tflops=round(split_flops[k] / (phase_ms[k] * 1e-3) / 1e12, 2))

    # DRAM bytes of the dominant kernel's launches of one step: from the record of an ncu capture of this
    # workload at this chunk width, if there is one (null otherwise)
    traffic = None
    if not args.vocab and not args.frozen_head and args.beam == 0 and not args.bias:
        traffic = load_traffic(cfg.name, chunk)

    # kernels launched by the library inside the timed region
    dp_launches = 5 if args.beam > 0 else 3      # sweeps (+ best-alignment sweeps, arc flags), label chains, occupancies
    # batch tables (3), subset (3), stacking, gather + Z_U, DP, normaliser + combine, loss, row clean-up, chunks,
    # un-stacking
    launches_per_step = (3 + 3 + 1 + 2 + dp_launches + 2 + 1 + 1 + (2 if args.frozen_head else 3) * nchunks + 1
                        + (nchunks if args.bias else 0))          # + column sums for dbias
    gpu_launches = launches_per_step * args.steps

    # ---- end to end through the host-buffer entry point ----
    e2e = None
    if args.e2e_steps > 0 and not args.frozen_head and not args.bias:
        host_call = dict(beam=args.beam, chunk=args.chunk)     # 0: the host entry point's own default width
        h_res = binding.pruned_ctc_fwd_bwd_host(h_hidden, h_W, None, h_targets, il, tl, batch.blank,
                                                device=dev, **host_call)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.e2e_steps):
            binding.pruned_ctc_fwd_bwd_host(h_hidden, h_W, None, h_targets, il, tl, batch.blank,
                                            scratch=h_res["scratch"], out=h_res, device=dev, **host_call)
        e1.record()
        torch.cuda.synchronize()
        ms_e2e = e0.elapsed_time(e1) / args.e2e_steps
        ms_e2e, _, _ = reduce_over_ranks(ms_e2e, 0.0, 0.0, red_dev)
        h2d = h_hidden.numel() * h_hidden.element_size() + h_W.numel() * h_W.element_size() + h_targets.numel() * 4
        d2h = (N * 4 + h_hidden.numel() * h_hidden.element_size() + h_W.numel() * h_W.element_size()
               + (int(tl.sum()) + 1) * 4 + 4 + h_targets.numel() * 4 + N * 4)
        e2e = dict(value=frames_all / (ms_e2e * 1e-3), unit=UNIT, ms_per_step=ms_e2e,
                   h2d_bytes_per_step=int(h2d), d2h_bytes_per_step=int(d2h), steps=args.e2e_steps,
                   api="pruned_ctc_fwd_bwd_host (pinned host buffers)")
        del h_res
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- peak head-and-loss bytes; the workspace does not depend on M*V ----
    out_bytes = (N * 4 + hidden.numel() * hidden.element_size()
                 + (0 if args.frozen_head else W.numel() * W.element_size()))
    prob_half = binding.make_problem(N, batch.T, D, V // 2 // 8 * 8, prob.dtype, batch.blank, args.beam, chunk,
                                     batch.targets.shape[1], max_K=max_K_pre)
    ws_half = binding.workspace_bytes(prob_half, il, tl)

    # ---- yardstick: a dense head's three library GEMMs with materialised logits (no loss, no softmax) ----
    dense = None
    if args.dense_head and cfg.dtype == "bf16" and rank == 0:
        need = 2 * M * V
        free_b, _ = torch.cuda.mem_get_info(dev)
        if need + (2 << 30) < free_b:
            X2 = hidden.reshape(-1, D)[:M].contiguous()
            Zl = torch.empty((M, V), dtype=torch.bfloat16, device=dev)
            dX2 = torch.empty_like(X2)
            dW2 = torch.empty_like(W)
            def dense_step():
                torch.matmul(X2, W.t(), out=Zl)          # logits, kept
                torch.matmul(Zl, W, out=dX2)             # dX  (Zl stands in for dlogits: same shape and dtype)
                torch.matmul(Zl.t(), X2, out=dW2)        # dW
            for _ in range(3):
                dense_step()
            torch.cuda.synchronize()
            d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            d0.record()
            for _ in range(args.steps):
                dense_step()
            d1.record()
            torch.cuda.synchronize()
            dms = d0.elapsed_time(d1) / args.steps
            dense = dict(ms_per_step=dms, tflops=6.0 * M * D * V / (dms * 1e-3) / 1e12, logits_bytes=need,
                         ratio_this_over_dense=ms_per_step / dms,
                         what="torch.matmul (cuBLAS) forward + dX + dW with a materialised bf16 [M, V] logits "
                              "array; no softmax, no loss: a lower bound for a dense head-and-loss step")
            del Zl, dX2, dW2, X2
            torch.cuda.empty_cache()
        else:
            dense = dict(skipped="the [M, V] logits array does not fit next to the benchmark's buffers")

    # ---- the oracle on the host cores, on a bounded sample ----
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        W64 = batch.W.astype(np.float64)
        dt, frames = time_oracle(batch, W64, args.cpu_frames)
        cpu = dict(value=frames / dt, unit=UNIT, cores=blas_threads(), kind="oracle", seconds=round(dt, 2),
                   sample=(f"oracle fwd+bwd (float64, full V, full dW) on the first {frames} frames of "
                           f"utterance 0 of {cfg.name}"))

    # ---- every configuration, same protocol, fewer steps (the headline stays the default workload) ----
    all_cfg = None
    want_all = args.all_configs
    if want_all is None:
        want_all = (args.config == "c4" and world == 1 and not (args.vocab or args.frozen_head or args.bias
                                                                 or args.allreduce_dw or args.chunk or args.beam))
    K_selected = int(res["K"].item())
    w_gb = W.numel() * W.element_size() / 1e9
    if want_all and world == 1:
        del res, hidden, W, targets, traces
        torch.cuda.empty_cache()
        all_cfg = []
        # the five configurations (c5 also at beams 16 and 8), then two more rows: the frozen-head setting of the
        # paper's LLM-CTC runs on the headline shape, and the smallest workload of the paper's own benchmark grid
        plan = [(n, b, {}) for n, beams in (("c1", (0.0,)), ("c2", (0.0,)), ("c3", (0.0,)), ("c4", (0.0,)),
                                            ("c5", (0.0, 16.0, 8.0))) for b in beams]
        plan += [("c4", 0.0, dict(frozen_head=True)), ("g16k", 0.0, dict(promise_k=True))]
        for name, b, kw in plan:
            try:
                all_cfg.append(time_config(binding, torch, dev, wl.CONFIGS[name], b, args.all_steps, 3, peaks, **kw))
            except Exception as exc:      # the headline line must not be lost to a side measurement
                all_cfg.append(dict(workload=name, beam=b, error=repr(exc)[:300], **kw))
                torch.cuda.empty_cache()

    line = dict(
        metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
        ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype=cfg.dtype, data="synthetic",
        config=dict(workload=cfg.name, N=N, T_range=[cfg.T_lo, cfg.T_hi], D=D, V=V, M_frames=M,
                    K_selected=K_selected, beam=args.beam, chunk=chunk, frozen_head=args.frozen_head, bias=args.bias, max_K=max_K,
                    l2="inputs larger than L2 (W and dW are %.2f GB each)" % w_gb,
                    parallelism=("utterance-sharded data parallel, dW all-reduced per vocabulary chunk (NCCL)"
                                 if sum_dW else "independent utterance batches per GPU, no collective")),
        tflops=flops_all / (ms_per_step * 1e-3) / 1e12,
        frac_of_bf16_peak=dict(burst=flops_all / (ms_per_step * 1e-3) / 1e12 / (peaks["bf16_tflops"] * world),
                               sustained=flops_all / (ms_per_step * 1e-3) / 1e12 / (peak * world),
                               peaks=peaks["source"]),
        flops_per_step=flops_per_step,
        phase_ms={k: round(v, 4) for k, v in phase_ms.items()},
        roofline=dict(bound="tensor", achieved=achieved_tflops, peak=peak, unit="TFLOP/s",
                      frac=achieved_tflops / peak, traffic=traffic,
                      kernel="k_umma_gemm (all fused-epilogue instances: lse, dlogits, dh, dw)",
                      launches_per_step=gemm_launches, ms_per_step=gemm_ms,
                      peak_source="%s bf16_tflops_sustained (kernel timed inside a long step)" % peaks["source"],
                      per_kernel=per_kernel),
        peak_bytes=dict(workspace=ws_bytes, outputs=out_bytes, workspace_at_half_V=ws_half,
                        one_fp32_MxV_array=4 * M * V),
        e2e=e2e, gpu_launches=gpu_launches, clocks=clocks, cpu_baseline=cpu,
    )
    if args.lib_variant.startswith("probe_"):
        line["invalid"] = "measurement build %s: part of the kernel is knocked out, results are wrong" % args.lib_variant
    elif args.lib_variant:
        line["variant"] = args.lib_variant
    if all_cfg is not None:
        line["all_configs"] = all_cfg
    if dense is not None:
        line["dense_head"] = dense
    print(json.dumps(line), flush=True)
    if world > 1 or args.allreduce_dw:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
