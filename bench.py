#!/usr/bin/env python
"""Benchmark of the PCG verification hot path (pcg_verify) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload C5]

One step = one pcg_verify call over one whole batch of the workload: every drafted position's target and draft
row is streamed (softmax statistics, group label, label-group masses, accept test), then per sequence the first
rejection is found and the residual / bonus group and token are drawn.  The default workload is C5 (B=256, K=16,
V=65536, bf16 logits, 16384 groups of top-6 membership), the configuration the headline metric is quoted on.
Inputs are seeded synthetic stand-ins for the paper's TTS logits (see paper_2511_13732_b200/workloads.py).

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank verifies its own batch of the same shape (weak
scaling; sequences are independent, so there is no data-path collective) and the time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2511_13732_b200 import workloads as W  # noqa: E402

METRIC = "verified draft positions/sec"
UNIT = "positions/s"
FALLBACK_HBM_GBS = 6650.0  # used only when MEASURED_PEAKS.json is absent
KERNEL_SOURCES = ("paper_2511_13732_b200/csrc/pcg_kernels.cu", "paper_2511_13732_b200/csrc/pcg_common.cuh")


def kernel_source_hash():
    """sha256 (first 16 hex digits) of the sources of the verification kernels: ties an ncu record to a kernel version."""
    import hashlib

    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic_bytes(workload):
    """dram__bytes_read.sum + dram__bytes_write.sum of one position_kernel launch, from the ncu record kept under
    profiles/ (lines `workload:`, `kernel_source_hash:`, `dram_bytes_read_per_launch:`, `dram_bytes_write_per_launch:`).
    None when there is no record for the workload or the kernels have been edited since it was taken."""
    path = os.path.join(ROOT, "profiles", f"position_kernel_{workload.lower()}_dram_traffic.md")
    try:
        fields = {}
        with open(path) as f:
            for ln in f:
                if ":" in ln and not ln.startswith(" "):
                    k, v = ln.split(":", 1)
                    fields[k.strip().strip("`")] = v.strip().strip("`")
        if fields.get("kernel_source_hash") != kernel_source_hash():
            return None
        return int(fields["dram_bytes_read_per_launch"]) + int(fields["dram_bytes_write_per_launch"])
    except (OSError, KeyError, ValueError):
        return None


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except (OSError, KeyError, ValueError):
        return FALLBACK_HBM_GBS, "fallback"


def hold_device(torch, ms: float) -> float:
    """Enqueues a device-side delay of about `ms` milliseconds on the current stream (torch's spin kernel; nothing
    of it lies inside a timed region).  Returns the delay asked for, 0.0 if the kernel is not available."""
    try:
        khz = torch.cuda.get_device_properties(torch.cuda.current_device()).clock_rate  # kHz
        torch.cuda._sleep(int(ms * khz))
        return ms
    except Exception:
        return 0.0


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period, self.samples, self.reasons = index, period_s, [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None

    def start(self):
        try:
            import pynvml

            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None
            return self
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def _run(self):
        nv = self._nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    bits = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in names.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            pass
    return local_rank


def oracle_leg(cfg, groups, batch, min_seconds=2.0, max_passes=200, timed_outputs=None):
    """Time the CPU oracle, as it stands, with all host cores: whole passes over (a bounded sample of) the batch,
    repeated until about `min_seconds` of wall time (tens of core-seconds of CPU work) have been spent."""
    import oracle

    oracle.build()
    cores = oracle.max_threads()
    B = batch.draft_tokens.shape[0]

    last = {}

    def one_pass(nseq):
        t0 = time.perf_counter()
        last["ref"] = oracle.verify(batch.target_logits[:nseq], batch.draft_logits[:nseq], batch.draft_tokens[:nseq],
                                    groups.group_ptr, groups.group_tok, groups.tok_degree, batch.uniforms[:nseq],
                                    batch.temperature, threads=cores)
        return time.perf_counter() - t0

    probe = max(one_pass(min(B, 8)), 1e-5)  # sizes the sample so that one pass stays below ~min_seconds
    nseq = int(min(B, max(8, min_seconds / (probe / min(B, 8)))))
    passes, spent = 0, 0.0
    while passes < max_passes and (spent < min_seconds or passes < 2):
        spent += one_pass(nseq)
        passes += 1
    evaluated = int((np.minimum(last["ref"].accept_len, cfg.K - 1) + 1).sum())  # positions the oracle really formed
    out = {"value": nseq * cfg.K * passes / spent, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"first {nseq} of {B} sequences of {cfg.name} ({nseq * cfg.K} drafted positions), {passes} "
                     f"passes, {spent:.3f} s wall on {cores} threads (OpenMP over sequences; the oracle stops a "
                     f"sequence at its first rejection, as Algorithm 1 does: it evaluates {evaluated} of the "
                     f"{nseq * cfg.K} positions it is credited with here, so the figure flatters the CPU)",
           "positions_evaluated_per_pass": evaluated,
           "value_counting_evaluated_positions_only": evaluated * passes / spent}
    # the same oracle on ONE thread, on a smaller sample (about a quarter of the time budget)
    n1 = int(max(1, min(nseq, round(nseq * 0.25 * min_seconds / max(spent / passes, 1e-9) / max(cores, 1)))))
    t0 = time.perf_counter()
    oracle.verify(batch.target_logits[:n1], batch.draft_logits[:n1], batch.draft_tokens[:n1], groups.group_ptr,
                  groups.group_tok, groups.tok_degree, batch.uniforms[:n1], batch.temperature, threads=1)
    t1 = time.perf_counter() - t0
    out["single_thread"] = {"value": n1 * cfg.K / t1, "unit": UNIT, "cores": 1,
                            "sample": f"first {n1} sequences, one pass, {t1:.3f} s wall on one thread"}
    if timed_outputs is not None:
        # the oracle's results on that sample against what the timed GPU steps produced, decision by decision
        from oracle.compare import compare_verify

        n, tok, grp = (a[:nseq] for a in timed_outputs)
        cmp = compare_verify(n, tok, grp, last["ref"], band=1e-6)
        out["parity_of_timed_outputs"] = {"sequences": int(nseq), "hard_mismatches": int(cmp.hard),
                                          "excused_within_1e-6": int(cmp.excused)}
    return out


def run_reference(args, cfg, rank):
    """Reference arm: the CPU oracle on the host cores (rank 0 only)."""
    if rank != 0:
        return
    groups = W.make_groups(cfg)
    nseq = min(cfg.B, 64)
    batch = W.make_batch(cfg, B=nseq)
    import oracle

    oracle.build()
    cores = oracle.max_threads()

    def step():
        oracle.verify(batch.target_logits, batch.draft_logits, batch.draft_tokens, groups.group_ptr, groups.group_tok,
                      groups.tok_degree, batch.uniforms, batch.temperature, threads=cores)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = nseq * cfg.K * args.steps / dt
    sample = f"each step = first {nseq} of {cfg.B} sequences of {cfg.name} ({nseq * cfg.K} drafted positions)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def quick_workload(binding, torch, wcfg, peak, steps=300):
    """ms per pcg_verify call (default mode, rotating input copies) and pcg_verify_thinning call of a small workload."""
    groups = W.make_groups(wcfg)
    batch = W.make_batch(wcfg)
    handle = binding.Groups(groups.V, groups.group_ptr, groups.group_tok, groups.tok_degree)

    def dev(a):
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(a).cuda()

    base = (dev(batch.target_logits), dev(batch.draft_logits), dev(batch.draft_tokens), dev(batch.uniforms))
    rotation = [base] + [tuple(t.clone() for t in base) for _ in range(input_copies(wcfg) - 1)]
    B, K, V, M = wcfg.B, wcfg.K, wcfg.V, groups.M
    dt_code = binding.PCG_BF16 if wcfg.dtype == "bf16" else binding.PCG_F32
    esz = 2 if wcfg.dtype == "bf16" else 4
    ws = torch.empty(binding.pcg_verify_workspace_bytes(B, K, V, M, dt_code, 0), dtype=torch.uint8, device="cuda")
    out = (torch.empty(B, dtype=torch.int32, device="cuda"), torch.empty((B, K + 1), dtype=torch.int32, device="cuda"),
           torch.empty((B, K + 1), dtype=torch.int32, device="cuda"), torch.empty(B, dtype=torch.int32, device="cuda"))
    thin_u = torch.from_numpy(W.make_thin_uniforms(wcfg, 32)).cuda()
    thin_ws = torch.empty(binding.pcg_verify_thinning_workspace_bytes(B, K, V, M, dt_code), dtype=torch.uint8, device="cuda")
    thin_out = out + (torch.empty(B, dtype=torch.int32, device="cuda"),)
    res = {"config": workload_config(wcfg)}
    for key in ("verify", "verify_thinning"):
        def one(i):
            a_tl, a_dl, a_x, a_u = rotation[i % len(rotation)]
            if key == "verify":
                binding.pcg_verify(a_tl, a_dl, a_x, handle, a_u, wcfg.temperature, workspace=ws, out=out)
            else:
                binding.pcg_verify_thinning(a_tl, a_dl, a_x, handle, a_u, thin_u, wcfg.temperature, workspace=thin_ws,
                                            out=thin_out)
        for i in range(10):
            one(i)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for i in range(steps):
            one(i)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        gbs = B * (2 * K + 1) * V * esz / (ms * 1e-3) / 1e9
        res[key] = {"ms_per_step": ms, "steps": steps, "value": B * K / (ms * 1e-3), "unit": UNIT,
                    "whole_step_gbs": gbs, "whole_step_frac_of_measured_peak": gbs / peak}
        # the same call captured in a CUDA graph and replayed: the device-side time without the host's launch work
        # (at these sizes the Python caller, not the GPU, paces the plain calls)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            one(0)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            one(0)
        for _ in range(3):
            graph.replay()
        e0.record()
        for _ in range(steps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        res[key]["cuda_graph_replay_ms_per_step"] = e0.elapsed_time(e1) / steps
    handle.close()
    return res


def group_construction_leg(binding, torch, V, reps=2):
    """The one-time group construction (Sec. 2.1) on a seeded clustered table of vocabulary size V, both tensor paths."""
    d_emb = 512 if V >= 32768 else 128
    gen = torch.Generator(device="cuda")
    gen.manual_seed(2511)
    centres = torch.randn((max(1, V // 24), d_emb), device="cuda", generator=gen)
    which = torch.randint(0, max(1, V // 24), (V,), device="cuda", generator=gen)
    table = (centres[which] + 0.35 * torch.randn((V, d_emb), device="cuda", generator=gen)).to(torch.bfloat16)
    res = {"V": V, "d": d_emb, "theta": 0.42}
    for flag, key in ((False, "tcgen05"), (True, "mma_sync")):
        for _ in range(reps):  # the last repetition is reported
            asg = binding.Asg(table, 0.42, mma_sync=flag)
            info = {"similarity_ms": asg.info.similarity_ms, "total_ms": asg.info.total_ms, "groups": asg.info.M,
                    # the full V x V product at 2 flops per multiply-add; the tensor-core form executes about half of it
                    # (the cosine is symmetric: tiles below the diagonal blocks are mirrored, not computed)
                    "tflops_full_matrix_equivalent": 2.0 * V * V * d_emb / (asg.info.similarity_ms * 1e-3) / 1e12}
            asg.close()
        res[key] = info
    return res


L2_BYTES = 126 << 20


def input_copies(cfg):
    """How many rotating copies of the inputs the timed steps walk through: one when a batch alone exceeds the L2,
    else enough for twice the L2 (at most 64)."""
    esz = 4 if cfg.dtype == "f32" else 2
    nbytes = cfg.B * (2 * cfg.K + 1) * cfg.V * esz
    return 1 if nbytes > L2_BYTES else int(min(64, -(-2 * L2_BYTES // nbytes)))


def workload_config(cfg):
    esz = 4 if cfg.dtype == "f32" else 2
    nbytes = cfg.B * (2 * cfg.K + 1) * cfg.V * esz
    copies = input_copies(cfg)
    if copies == 1:
        l2 = "not flushed: each step streams the whole batch, larger than the 126 MB L2"
    elif copies * nbytes > L2_BYTES:
        l2 = (f"not flushed: the timed steps rotate over {copies} copies of the inputs, {copies * nbytes / 2**20:.0f} MB "
              f"in all, larger than the 126 MB L2")
    else:
        l2 = (f"not flushed: the timed steps rotate over {copies} copies of the inputs, only {copies * nbytes / 2**20:.1f} MB "
              f"in all, so the inputs stay in the 126 MB L2 (launch-latency-bound case, not a bandwidth figure)")
    return {"workload": cfg.name, "B": cfg.B, "K": cfg.K, "V": cfg.V, "M": cfg.M, "logits_dtype": cfg.dtype,
            "temperature": cfg.temperature, "membership": f"{cfg.groups} (mean degree {cfg.degree})", "l2": l2}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C5", choices=sorted(W.CONFIGS))
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size B (profiling only)")
    ap.add_argument("--mode", default="default", choices=["default", "dense", "cluster", "batched", "thinning"],
                    help="pcg_verify mode of the timed steps (the headline is 'default'); 'thinning' times "
                         "pcg_verify_thinning (the paper's sampler for the terminal group) instead")
    ap.add_argument("--thin-trials", type=int, default=32, help="trials supplied per sequence to pcg_verify_thinning")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-modes", action="store_true", help="skip the brief timing of the other pcg_verify modes")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the brief timing of the smaller workloads C1-C4")
    ap.add_argument("--only-group-construction", action="store_true",
                    help="run nothing but the one-time group construction (pcg_asg_create) on a seeded clustered table "
                         "of the workload's vocabulary size and print its timing (used for profiling that kernel)")
    args = ap.parse_args()
    cfg = W.CONFIGS[args.workload]
    if args.batch > 0:
        cfg = W.scaled(cfg, B=args.batch, name=f"{cfg.name}[B={args.batch}]")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if args.steps == 2000:
            args.steps = 5
        args.warmup = min(args.warmup, 2)
        run_reference(args, cfg, rank)
        return

    import torch

    from paper_2511_13732_b200 import binding
    from paper_2511_13732_b200.sharding import max_over_ranks, rank_sequences

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    binding.load()
    if args.only_group_construction:
        if rank == 0:
            print(json.dumps({"group_construction": group_construction_leg(binding, torch, cfg.V, reps=3)}), flush=True)
        return

    # ---- inputs: this rank's own batch (sequences rank*B .. rank*B+B-1 of the workload's stream) ----
    groups = W.make_groups(cfg)
    seqs = rank_sequences(cfg.B, rank, world, weak=True)
    batch = W.make_batch(cfg, seqs=seqs)
    handle = binding.Groups(groups.V, groups.group_ptr, groups.group_tok, groups.tok_degree)
    bf16 = cfg.dtype == "bf16"

    def host(a):
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).pin_memory()
        return torch.from_numpy(a).pin_memory()

    h_tl, h_dl, h_x, h_u = host(batch.target_logits), host(batch.draft_logits), host(batch.draft_tokens), host(batch.uniforms)
    tl, dl = h_tl.cuda(non_blocking=True), h_dl.cuda(non_blocking=True)
    if bf16:
        tl, dl = tl.view(torch.bfloat16), dl.view(torch.bfloat16)
    x, u = h_x.cuda(), h_u.cuda()
    B, K, V, M = cfg.B, cfg.K, cfg.V, groups.M
    dt_code = binding.PCG_BF16 if bf16 else binding.PCG_F32
    mode_codes = {"default": binding.VERIFY_DEFAULT, "dense": binding.VERIFY_DENSE,
                  "cluster": binding.VERIFY_CLUSTER_TERMINAL, "batched": binding.VERIFY_BATCHED_TERMINAL}
    thinning = args.mode == "thinning"
    mode = mode_codes.get(args.mode, binding.VERIFY_DEFAULT)
    ws = torch.empty(binding.pcg_verify_workspace_bytes(B, K, V, M, dt_code, mode), dtype=torch.uint8, device="cuda")
    out = (torch.empty(B, dtype=torch.int32, device="cuda"), torch.empty((B, K + 1), dtype=torch.int32, device="cuda"),
           torch.empty((B, K + 1), dtype=torch.int32, device="cuda"), torch.empty(B, dtype=torch.int32, device="cuda"))
    esz = 2 if bf16 else 4
    # pcg_verify_thinning: its own trial uniforms, workspace and a fifth output (trials drawn per sequence)
    thin_u = torch.from_numpy(W.make_thin_uniforms(cfg, args.thin_trials, seqs=seqs)).cuda()
    thin_ws = torch.empty(binding.pcg_verify_thinning_workspace_bytes(B, K, V, M, dt_code), dtype=torch.uint8, device="cuda")
    thin_out = tuple(torch.empty_like(t) for t in out) + (torch.empty(B, dtype=torch.int32, device="cuda"),)

    # small workloads: rotate over several copies of the inputs so that they are not simply served from the L2
    rotation = [(tl, dl, x, u)] + [(tl.clone(), dl.clone(), x.clone(), u.clone()) for _ in range(input_copies(cfg) - 1)]
    turn = [0]

    def thin_step(events=None):
        a_tl, a_dl, a_x, a_u = rotation[turn[0] % len(rotation)]
        turn[0] += 1
        binding.pcg_verify_thinning(a_tl, a_dl, a_x, handle, a_u, thin_u, cfg.temperature, workspace=thin_ws,
                                    out=thin_out, stage_events=events)

    def step(events=None):
        if thinning:
            return thin_step(events)
        a_tl, a_dl, a_x, a_u = rotation[turn[0] % len(rotation)]
        turn[0] += 1
        binding.pcg_verify(a_tl, a_dl, a_x, handle, a_u, cfg.temperature, workspace=ws, out=out, stage_events=events,
                           mode=mode)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(physical_gpu_index(local_rank), period_s=0.002).start()
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # After the barrier the device is idle: without more ado the start event would fire at once and the region
    # would open with the host's latency of issuing the first step (0.1 ms, i.e. 5 us per step of a 20-step run).
    # A short device-side delay ahead of the start event lets the first steps queue up behind it, so that the region
    # holds the device time of K steps, as it does by itself in a long run.
    hold_ms = hold_device(torch, 0.4)
    t_begin.record()
    for i in range(args.steps):
        step()
    t_end.record()
    barrier()
    ms_total = max_over_ranks(t_begin.elapsed_time(t_end), dist)
    ms_step = ms_total / args.steps
    # Stage times: a second, short loop after the timed region, every step carrying the library's three stage events
    # (an event between two kernels costs a drain of the first one, which is why the timed steps carry none).
    STAGE_STEPS = 16
    stage = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(STAGE_STEPS)]
    for evs in stage:
        for e in evs:
            e.record()
    torch.cuda.synchronize()
    for evs in stage:
        step(evs)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    pos_ms = statistics.fmean(e[0].elapsed_time(e[1]) for e in stage)
    term_ms = statistics.fmean(e[1].elapsed_time(e[2]) for e in stage)
    accept_len = (thin_out if thinning else out)[0].cpu().numpy()

    # ---- end to end through the host entry point: pinned host inputs in, host outputs back, every step ----
    arena = torch.empty(binding.pcg_verify_host_arena_bytes(B, K, V, M, dt_code), dtype=torch.uint8, device="cuda")
    h_out = (torch.empty(B, dtype=torch.int32).pin_memory(), torch.empty((B, K + 1), dtype=torch.int32).pin_memory(),
             torch.empty((B, K + 1), dtype=torch.int32).pin_memory(), torch.empty(B, dtype=torch.int32).pin_memory())

    def e2e_step():
        binding.pcg_verify_host(h_tl, h_dl, h_x, handle, h_u, cfg.temperature, arena, h_out)

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist) / args.e2e_steps
    assert np.array_equal(h_out[0].numpy(), accept_len), "host and device entry points disagree"
    h2d = (B * (2 * K + 1) * V * esz) + B * K * 4 + B * (K + 1) * 8
    d2h = B * 4 * 2 + B * (K + 1) * 4 * 2

    # kernels launched by one pcg_verify call (see pcg_verify in csrc/pcg_kernels.cu)
    info = handle.info
    chunk_unit = 256 if (B >= 256 and (64 << 20) // (V * 4) >= 256) else 128 if B >= 128 else 32
    chunk = min(-(-B // chunk_unit) * chunk_unit, max(chunk_unit, ((64 << 20) // (V * 4)) // chunk_unit * chunk_unit))
    batched = 1 + 2 * (-(-B // chunk)) + 1  # position, (transposed operand, sparse product) per chunk, pick
    sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
    default_is_cluster = B * info.slices <= 2 * sm_count  # the library's rule for PCG_VERIFY_DEFAULT
    launches_per_step = {"default": 2 if default_is_cluster else batched, "cluster": 2, "batched": batched,
                         "dense": 2 * 3 + 1 + 1 + 1, "thinning": 2}[args.mode]

    # the other modes, briefly (same inputs, same outputs): context for the headline mode
    other_modes = {}
    if world == 1 and not args.no_other_modes:
        for name, reps in (("cluster", 20), ("batched", 20), ("dense", 3)):
            if name == args.mode:
                continue
            m = mode_codes[name]
            ws_m = torch.empty(binding.pcg_verify_workspace_bytes(B, K, V, M, dt_code, m), dtype=torch.uint8, device="cuda")
            out_m = tuple(torch.empty_like(t) for t in out)
            for _ in range(2):
                binding.pcg_verify(tl, dl, x, handle, u, cfg.temperature, workspace=ws_m, out=out_m, mode=m)
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            m0.record()
            for _ in range(reps):
                binding.pcg_verify(tl, dl, x, handle, u, cfg.temperature, workspace=ws_m, out=out_m, mode=m)
            m1.record()
            torch.cuda.synchronize()
            if thinning:  # other draws for the terminal token: only the accept lengths must agree
                same = torch.equal(thin_out[0], out_m[0])
            else:
                same = all(torch.equal(a_, b_) for a_, b_ in zip(out, out_m))
            other_modes[name] = {"ms_per_step": m0.elapsed_time(m1) / reps, "steps": reps,
                                 ("accept_lengths_equal_to_timed_mode" if thinning else "outputs_equal_to_timed_mode"): bool(same)}
            del ws_m

    # the timed mode once more, captured in a CUDA graph and replayed (launch overhead off the host)
    if world == 1 and not args.no_other_modes:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        reps = 200
        for _ in range(3):
            graph.replay()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        for _ in range(reps):
            graph.replay()
        c1.record()
        torch.cuda.synchronize()
        other_modes["cuda_graph_replay_of_timed_mode"] = {"ms_per_step": c0.elapsed_time(c1) / reps, "steps": reps}

    # the smaller workloads C1-C4, briefly, in the default mode (they are parity-test cases, not the headline; their
    # times are launch-latency bound, see config.l2 of each)
    other_workloads = {}
    if world == 1 and not args.no_other_workloads and not args.no_other_modes and cfg.name == "C5":
        for name in ("C1", "C2", "C3", "C4"):
            other_workloads[name] = quick_workload(binding, torch, W.CONFIGS[name], hbm_peak()[0])

    # the other two entry points of the boundary, briefly: pcg_group_probs on a slice of the target rows, and the
    # one-time group construction on a seeded clustered table of the workload's vocabulary size
    extras = {}
    if world == 1 and not args.no_other_modes:
        rows = min(B * (K + 1), 1024)
        x_rows = tl.reshape(-1, V)[:rows]
        P = binding.pcg_group_probs(x_rows, handle, cfg.temperature)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(5):
            binding.pcg_group_probs(x_rows, handle, cfg.temperature, out=P)
        g1.record()
        torch.cuda.synchronize()
        gp_ms = g0.elapsed_time(g1) / 5
        extras["group_probs"] = {"rows": rows, "ms": gp_ms, "rows_per_s": rows / (gp_ms * 1e-3),
                                 "counted_gbs": rows * (V * esz + M * 4) / (gp_ms * 1e-3) / 1e9,
                                 "row_sum_max_error": float((P.sum(dim=1) - 1).abs().max())}
        # the paper's thinning sampler for the terminal group instead of the enumerated residual
        if not thinning:
            for _ in range(3):
                thin_step()
            reps = 200
            tev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            for e in tev:
                e.record()
            torch.cuda.synchronize()
            q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            q0.record()
            for i in range(reps):
                thin_step(tev if i == reps - 1 else None)
            q1.record()
            torch.cuda.synchronize()
            th_ms = q0.elapsed_time(q1) / reps
            tr = thin_out[4].float()
            extras["verify_thinning"] = {
                "ms_per_step": th_ms, "steps": reps, "value": B * K / (th_ms * 1e-3), "unit": UNIT,
                "whole_step_gbs": B * (2 * K + 1) * V * esz / (th_ms * 1e-3) / 1e9,
                "whole_step_frac_of_measured_peak": B * (2 * K + 1) * V * esz / (th_ms * 1e-3) / 1e9 / hbm_peak()[0],
                "per_sequence_stage_ms_last_step": tev[1].elapsed_time(tev[2]),
                "trials_supplied": args.thin_trials, "trials_mean": float(tr.mean()), "trials_max": int(tr.max()),
                "sequences_exhausted": int((thin_out[3] & binding.FLAG_THINNING_EXHAUSTED).ne(0).sum()),
                "accept_lengths_equal_to_timed_mode": bool(torch.equal(thin_out[0], out[0]))}
        # workload statistics on a sample of drafted positions: how much coarse-graining raises the overlap of the
        # two models (sum_g min(P, Q) against sum_t min(p, q); the former is the group-level acceptance probability)
        ns = min(B, 64)
        t_rows = tl[:ns, 0].contiguous()
        d_rows = dl[:ns, 0].contiguous()
        Pg = binding.pcg_group_probs(t_rows, handle, cfg.temperature)
        Qg = binding.pcg_group_probs(d_rows, handle, cfg.temperature)
        pt = torch.softmax(t_rows.float() / cfg.temperature, dim=1)
        qt = torch.softmax(d_rows.float() / cfg.temperature, dim=1)
        extras["workload_statistics"] = {
            "positions_sampled": ns,
            "group_overlap_sum_min_PQ": float(torch.minimum(Pg, Qg).sum(dim=1).mean()),
            "token_overlap_sum_min_pq": float(torch.minimum(pt, qt).sum(dim=1).mean())}
        extras["group_construction"] = group_construction_leg(binding, torch, V)
    if rank == 0:
        peak, peak_src = hbm_peak()
        alg_bytes = B * K * 2 * V * esz  # per drafted position: one target and one draft row, read once
        achieved = alg_bytes / (pos_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": world * B * K / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(cfg),
            "hbm": {"counted_bytes_per_step": B * (2 * K + 1) * V * esz,
                    "whole_step_gbs": B * (2 * K + 1) * V * esz / (ms_step * 1e-3) / 1e9,
                    "whole_step_frac_of_measured_peak": B * (2 * K + 1) * V * esz / (ms_step * 1e-3) / 1e9 / peak,
                    "whole_step_frac_of_8tbs": B * (2 * K + 1) * V * esz / (ms_step * 1e-3) / 1e9 / 8000.0},
            "roofline": {"bound": "hbm", "kernel": "position_kernel", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "traffic": ncu_traffic_bytes(cfg.name),
                         "traffic_source": f"profiles/position_kernel_{cfg.name.lower()}_dram_traffic.md (null if the "
                                           "kernels were edited after that capture)",
                         "peak_source": peak_src, "algorithmic_bytes_per_launch": alg_bytes,
                         "avg_launch_ms": pos_ms,
                         # the figure the target is stated on: ALL kernels of the call, counted logits bytes / step time
                         "whole_call": {"achieved": B * (2 * K + 1) * V * esz / (ms_step * 1e-3) / 1e9,
                                        "frac": B * (2 * K + 1) * V * esz / (ms_step * 1e-3) / 1e9 / peak,
                                        "counted_bytes_per_step": B * (2 * K + 1) * V * esz, "ms_per_step": ms_step}},
            "timing": {"events": "CUDA events on the launching stream around the K steps",
                       "device_hold_before_start_event_ms": hold_ms,
                       "why": "the device is idle after the barrier; the hold lets the first steps queue up, so the "
                              "region holds K steps of device work and not the host's latency of issuing the first one"},
            "stages_ms": {"per_position_stage": pos_ms, "per_sequence_stage": term_ms,
                          "samples": STAGE_STEPS, "sampled": "on a separate loop of steps after the timed region"},
            "mode": args.mode + (" (per-sequence stage: " + ("cluster" if default_is_cluster else "batched") + ")"
                                 if args.mode == "default" else
                                 f" (pcg_verify_thinning, {args.thin_trials} trials supplied)" if thinning else ""),
            "other_modes": other_modes,
            "other_workloads": other_workloads,
            "other_entry_points": extras,
            "e2e": {"value": world * B * K / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": args.e2e_steps,
                    "api": "pcg_verify_host (pinned host tensors)"},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
            "mean_accept_len": float(accept_len.mean()),
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = oracle_leg(
                cfg, groups, batch,
                timed_outputs=None if thinning else tuple(t.cpu().numpy() for t in out[:3]))
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
