#!/usr/bin/env python
"""Benchmark of the FP32 GPT-2 training step (forward + backward + AdamW) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

One JSON line on stdout (rank 0).  `value` is tokens/s with the token batches already in
HBM; `e2e` is the same step driven through the host-buffer entry point (pinned host tokens
copied in, loss read back, every step).  `roofline` describes the dominant kernel, timed
with CUDA events on the launching stream; `cpu_baseline` is the float64 oracle on the
host cores on a bounded sample.  With N > 1 every rank runs an independent replica (the
path does not shard: one GPU, no collectives); the ranks only share a barrier and the
max-over-ranks time.  `--impl reference` times the CPU oracle itself.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import seeded_inputs as si  # noqa: E402

METRIC = "GPT-2 124M FP32 train tokens/s on 1 B200"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
TF32_OVER_BF16 = 0.5          # nominal dense ratio (1.1 / 2.25 PFLOP/s)
MMA_PER_PRODUCT = 3.0         # 3xTF32: three tensor-core products per FP32 product
GEMM_PROFILE = os.path.join(ROOT, "profiles", "gemm_tc_kernel_gpt2small_block.txt")


def ncu_qkv_gemm_dram_bytes():
    """dram__bytes_read.sum + dram__bytes_write.sum of the forward QKV GEMM launch (the first kernel of
    the committed ncu summary), in bytes; None if the summary is missing or unreadable."""
    try:
        total, seen = 0.0, 0
        with open(GEMM_PROFILE) as f:
            for line in f:
                parts = line.split()
                if len(parts) >= 3 and parts[0] in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
                    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}[parts[2]]
                    total += float(parts[1]) * scale
                    seen += 1
                    if seen == 2:
                        return total
    except (OSError, KeyError, ValueError):
        pass
    return None


_RESULT_OUT = None


def claim_stdout():
    """Standard output carries exactly one JSON line.  Libraries underneath write there too (NCCL prints
    its version banner on the first communicator), so file descriptor 1 is pointed at standard error
    for the rest of the process and the result goes to a private copy of the original descriptor."""
    global _RESULT_OUT
    if _RESULT_OUT is None:
        sys.stdout.flush()
        _RESULT_OUT = os.fdopen(os.dup(1), "w")
        os.dup2(2, 1)


def emit(line: dict):
    out = _RESULT_OUT if _RESULT_OUT is not None else sys.stdout
    out.write(json.dumps(line) + "\n")
    out.flush()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_step_seconds(cfg, seq_len, seed):
    """One forward + backward + AdamW of the oracle on ONE sequence of `seq_len` tokens."""
    import oracle
    c = dict(cfg)
    c["seq_len"] = seq_len
    m = oracle.Model(c)
    m.set_params(si.init_params(c, seed))
    tok, tgt = si.tokens_for(c, seed, 1)
    hp = si.ADAMW
    t0 = time.perf_counter()
    m.loss_and_grad(tok, tgt)
    m.adamw_step(hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], hp["grad_clip"])
    dt = time.perf_counter() - t0
    return dt, oracle.num_threads(), m


def run_reference(args, cfg):
    """The CPU oracle as the reference arm: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    total_steps = args.steps + args.warmup
    allowance = 150.0 / max(1, total_steps)
    # calibrate on a 64-token sequence, then pick the longest sample that fits the per-step allowance
    dt64, cores, _ = oracle_step_seconds(cfg, 64, 1)
    seq = 64
    while seq * 2 <= cfg["seq_len"] and dt64 * (seq * 2 / 64.0) * 1.3 < allowance:
        seq *= 2
    c = dict(cfg)
    c["seq_len"] = seq
    m = oracle.Model(c)
    m.set_params(si.init_params(c, 2))
    hp = si.ADAMW
    times = []
    for step in range(total_steps):
        tok, tgt = si.tokens_for(c, 100 + step, 1)
        t0 = time.perf_counter()
        m.loss_and_grad(tok, tgt)
        m.adamw_step(hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], hp["grad_clip"])
        if step >= args.warmup:
            times.append(time.perf_counter() - t0)
    ms = 1e3 * float(np.mean(times))
    value = seq / (ms / 1e3)
    sample = f"1 sequence of {seq} tokens per step (of B={cfg['batch']} x T={cfg['seq_len']}), full model, fwd+bwd+AdamW"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg["name"], "sample": sample},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    emit(line)


class RankSync:
    """What the replicas share: a barrier and the max-over-ranks of a locally measured time.
    `dist` is torch.distributed (already initialised) or None for a single rank; `device` is where
    the reduction tensor lives ("cuda" under NCCL, "cpu" under gloo)."""

    def __init__(self, dist=None, device="cuda"):
        self.dist, self.device = dist, device

    def _sync_device(self):
        if self.device != "cpu":
            import torch
            torch.cuda.synchronize()

    def barrier(self):
        self._sync_device()
        if self.dist is not None:
            self.dist.barrier()
        self._sync_device()

    def max(self, x: float) -> float:
        if self.dist is None:
            return float(x)
        import torch
        t = torch.tensor([x], dtype=torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Replicas only: every rank processes its own batch in the (max-over-ranks) step time."""
    return tokens_per_rank_step * world / (ms_per_step / 1e3)


def run_ours(args, cfg):
    import torch
    from paper_2606_24780_b200 import binding as b

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    elif args.ddp:
        import socket
        import torch.distributed as dist
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                                device_id=torch.device(f"cuda:{local}"))

    B, T = cfg["batch"], cfg["seq_len"]
    model = b.Model(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], T, cfg["vocab_size"],
                    cfg["padded_vocab_size"], B, flags=(b.BT_FLAG_RECOMPUTE_LN if args.recompute_ln else 0) |
                    (b.BT_FLAG_LOGITS_IN_PLACE if args.logits_in_place else 0) |
                    (b.BT_FLAG_RECOMPUTE_GELU if args.recompute_gelu else 0),
                    device=f"cuda:{local}")
    model.init(1234 + rank)
    if args.ddp:
        # Algorithm 1 instead of independent replicas: identical start weights from rank 0, then every
        # backward pass averages the gradients bucket by bucket on a second stream (NCCL through
        # torch.distributed; the library only orders the two streams with events)
        torch.cuda.synchronize()
        dist.broadcast(model.arena(0), src=0)
        comm_stream = torch.cuda.Stream()
        model.ddp_attach(lambda buf, bucket: dist.all_reduce(buf, op=dist.ReduceOp.AVG), comm_stream)
    opt = b.make_adamw(**si.ADAMW)
    n_batches = 4
    batches = [si.tokens_for(cfg, 10 * rank + i) for i in range(n_batches)]
    dev_batches = [(torch.as_tensor(t).cuda(), torch.as_tensor(g).cuda()) for t, g in batches]
    pin_batches = [(torch.as_tensor(t).pin_memory(), torch.as_tensor(g).pin_memory()) for t, g in batches]

    sync = RankSync(dist, "cuda")
    barrier, max_over_ranks = sync.barrier, sync.max

    for i in range(max(3, args.warmup)):
        tk, tg = dev_batches[i % n_batches]
        model.train_step(tk, tg, opt, want_loss=False)
    loss0 = b.bt_get_loss(model.h)

    # ---- timed region: K steps, tokens resident in HBM, CUDA events on the launching stream
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    l0 = b.bt_launch_count(model.h)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for i in range(args.steps):
        tk, tg = dev_batches[i % n_batches]
        model.train_step(tk, tg, opt, want_loss=False)
    ev1.record()
    barrier()
    launches = b.bt_launch_count(model.h) - l0
    clocks = sampler.stop()
    ms_total = max_over_ranks(ev0.elapsed_time(ev1))
    ms_per_step = ms_total / args.steps
    value = whole_job_tokens_per_s(B * T, world, ms_per_step)
    loss1 = b.bt_get_loss(model.h)

    # ---- end to end: host (pinned) tokens in, loss out, every step
    # (timed on the device as well: the events bracket the copies, the kernels and the idle gaps
    # the per-step loss read-back leaves on the stream)
    barrier()
    ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev2.record()
    for i in range(args.steps):
        tk, tg = pin_batches[i % n_batches]
        model.train_step_host(tk, tg, opt, want_loss=True)
    ev3.record()
    barrier()
    e2e_ms = max_over_ranks(ev2.elapsed_time(ev3)) / args.steps
    e2e_value = whole_job_tokens_per_s(B * T, world, e2e_ms)

    # ---- per-kernel event timing over a further K steps (events around every launch group)
    b.bt_profile_enable(model.h, 1)
    for i in range(args.steps):
        tk, tg = dev_batches[i % n_batches]
        model.train_step(tk, tg, opt, want_loss=False)
    kernels = {}
    for cat in range(b.bt_profile_num_categories()):
        ms, n, fl, by = b.bt_profile_read(model.h, cat)
        if n:
            kernels[b.bt_profile_category_name(cat)] = {
                "ms_per_step": ms / args.steps, "launch_groups_per_step": n / args.steps,
                "tflops": (fl / (ms * 1e-3) / 1e12) if ms > 0 else None,
                "gbs": (by / (ms * 1e-3) / 1e9) if ms > 0 else None}
    b.bt_profile_enable(model.h, 0)

    # the tensor pipe's own rate: clocks per 128 x 256 x 8 TF32 MMA on every SM (run after the timed regions)
    _, probe_clk, _ = b.bt_probe_tf32_mma_rate(torch.cuda.get_device_properties(local).multi_processor_count, 4000)
    mac_per_clk_sm = 128 * 256 * 8 / probe_clk
    n_sms = torch.cuda.get_device_properties(local).multi_processor_count

    peaks, peak_kind = load_peaks()
    tf32x3_peak = peaks["bf16_tflops_sustained"] * TF32_OVER_BF16 / MMA_PER_PRODUCT
    gemm = {k: v for k, v in kernels.items() if k.startswith("gemm_")}
    gemm_ms = sum(v["ms_per_step"] for v in gemm.values())
    gemm_flops = sum(v["tflops"] * v["ms_per_step"] for v in gemm.values())  # TFLOP/s * ms
    achieved = gemm_flops / gemm_ms if gemm_ms > 0 else 0.0
    roofline = {"bound": "tensor", "kernel": "gemm_tc_kernel / gemm_tc2_kernel (forward, dX and dW products, 3xTF32)", "achieved": achieved,
                "peak": tf32x3_peak, "unit": "TFLOP/s", "frac": achieved / tf32x3_peak,
                "peak_kind": f"{peak_kind} bf16 sustained x {TF32_OVER_BF16} (tf32) / {MMA_PER_PRODUCT:g} (3xTF32)",
                "share_of_step": gemm_ms / sum(v["ms_per_step"] for v in kernels.values()),
                # DRAM bytes of ONE launch of the forward QKV GEMM (8192 x 2304 x 768) from the committed
                # ncu capture under profiles/ (dram__bytes_read.sum + dram__bytes_write.sum), beside
                # its algorithmic bytes 8(MK + NK) + 4MN; other launches scale with their own sizes
                "traffic": ncu_qkv_gemm_dram_bytes(), "traffic_launch": "gemm forward qkv, M=8192 N=2304 K=768",
                "traffic_algorithmic": 8.0 * (8192 * 768 + 2304 * 768) + 4.0 * 8192 * 2304}
    # the same achieved rate against the pipe's own measured peak at the clock this run held:
    # (MAC per clock per SM from the probe) x 2 x SMs x median sampled SM clock / 3
    if clocks.get("sm_mhz"):
        clock_peak = mac_per_clk_sm * 2.0 * n_sms * clocks["sm_mhz"] * 1e6 / 1e12 / MMA_PER_PRODUCT
        roofline["tf32_probe"] = {"clocks_per_mma_128x256x8": probe_clk, "mac_per_clk_per_sm": mac_per_clk_sm,
                                  "peak_3xtf32_at_sampled_clock": clock_peak}
        roofline["frac_clock_scaled"] = achieved / clock_peak
        for v in kernels.values():
            v["mcycles"] = v["ms_per_step"] * clocks["sm_mhz"] / 1e3      # millions of SM clocks per step

    flop_per_token = si_flops_per_token(cfg)
    step_frac = value / world * flop_per_token / 1e12 / tf32x3_peak

    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 (3xTF32 tensor-core products, FP32 accumulate)", "data": "synthetic",
        "config": {"workload": cfg["name"], "n_layers": cfg["n_layers"], "d_model": cfg["d_model"],
                   "n_heads": cfg["n_heads"], "seq_len": T, "batch_per_gpu": B, "vocab": cfg["vocab_size"],
                   "padded_vocab": cfg["padded_vocab_size"], "tokens": "Zipf(1.1), seeded",
                   "parallelism": (f"ddp{world}: bucketed gradient all-reduce (Algorithm 1)" if args.ddp else
                                   "replicas only" if world > 1 else "1 GPU"),
                   "l2": "working set per step (>10 GB) exceeds L2; no explicit flush",
                   "layernorm_outputs": "recomputed in the backward pass" if args.recompute_ln else "kept",
                   "logits": "overwritten by their gradient" if args.logits_in_place else "kept",
                   "gelu_outputs": "recomputed in the backward pass" if args.recompute_gelu else "kept",
                   "workspace_gib": model.workspace_bytes / 2 ** 30,
                   "workspace_parts_gib": {k: v / 2 ** 30 for k, v in b.bt_workspace_parts(model.cfg).items()}},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": 2 * B * T * 4 * world, "d2h_bytes_per_step": 4 * world},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "step_model_tflops": value / world * flop_per_token / 1e12,
        "step_frac_of_3xtf32_peak": step_frac,
        "kernels": kernels,
        "loss_first_last": [loss0, loss1],
    }

    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            # bounded oracle sample (10 - 30 s of CPU work): one sequence of the same workload, as long
            # as fits; the time of a half-length sequence predicts the full one (attention grows with
            # the square of the length, the rest linearly: at most 4x)
            seq = max(64, T // 2)
            dt, cores, _ = oracle_step_seconds(cfg, seq, 2)
            while seq * 2 <= T and dt * 3.0 < 30.0:
                seq *= 2
                dt, cores, _ = oracle_step_seconds(cfg, seq, 2)
            line["cpu_baseline"] = {"value": seq / dt, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                                    "sample": f"1 sequence of {seq} tokens, full model, fwd+bwd+AdamW, {dt:.1f} s"}
        emit(line)
    model.close()
    if dist is not None:
        dist.destroy_process_group()


def si_flops_per_token(cfg):
    """Model FLOPs per token of one training step (GEMMs fwd + 2x bwd, causal attention fwd + 2.5x bwd)."""
    L, C, T, Vp = cfg["n_layers"], cfg["d_model"], cfg["seq_len"], cfg["padded_vocab_size"]
    F = 4 * C
    gemm_f = L * 2 * (C * 3 * C + C * C + 2 * C * F) + 2 * C * Vp
    attn_f = L * 4 * C * (T + 1) / 2.0
    return 3 * gemm_f + 3.5 * attn_f


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--recompute-ln", action="store_true",
                    help="BT_FLAG_RECOMPUTE_LN: smaller workspace, the LayerNorm forward runs again in the backward pass")
    ap.add_argument("--recompute-gelu", action="store_true",
                    help="BT_FLAG_RECOMPUTE_GELU: the GELU output planes are formed again in the backward pass")
    ap.add_argument("--logits-in-place", action="store_true",
                    help="BT_FLAG_LOGITS_IN_PLACE: the logit gradient's hi plane overwrites the logits")
    ap.add_argument("--ddp", action="store_true",
                    help="average the gradients over the ranks (bucketed all-reduce overlapped with the backward "
                         "pass) instead of running independent replicas")
    args = ap.parse_args()
    cfg = si.config(args.config)
    claim_stdout()
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
