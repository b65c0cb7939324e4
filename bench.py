#!/usr/bin/env python
"""Benchmark of the residual-VQ hot path on B200.

One step = one pass of the whole path over one batch of the key-cache workload
(4096 tokens x 8 KV heads x 128 bf16 channels, strided groups of 32, depth 8,
1024 codes per stage): prepare codebooks -> encode (with the batch's EMA
statistics) -> decode [-> all-reduce of the statistics over ranks] -> EMA apply.  Prints one JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (torchrun) every rank runs the same batch shape on its own vectors
(weak scaling); the only exchange is the all-reduce of the EMA statistics.
`--impl reference` times the CPU oracle on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import rvq_synth  # noqa: E402

def workload_name(tokens):
    return f"key_cache: {tokens} tokens x 8 heads x 128 bf16, strided groups of 32, R=8, K=1024"


# dram__bytes_read.sum + dram__bytes_write.sum of one encode launch on the default workload, from the ncu
# capture summarised in profiles/encode_tensor_key_cache.md (x 8.4 MB, codebooks and operand image 3.3 MB;
# the 2.2 MB of outputs stay in L2).  Reported only for the workload and kernel it was taken on.
ENCODE_DRAM_TRAFFIC = {4096: 11688960}
METRIC = "RVQ hot path (encode+decode+EMA update) head vectors per second"
UNIT = "Mvectors/s"
L2_FLUSH_BYTES = 256 << 20


def algorithmic_numbers(w):
    """Per-step algorithmic work of each phase (bytes and flops), from the shapes."""
    n, G, R, K, gd, d = w.n, w.groups, w.depth, w.codebook_size, w.group_dim, w.dim
    code_b = (G * R * w.code_bits + 31) // 32 * 4
    return {
        "encode_flops": 2.0 * gd * K * R * G * n,
        "encode_bytes": n * (d * 2 + code_b + 2),
        "decode_bytes": n * (code_b + 2 + d * 2),
        "ema_bytes": n * (d * 2 + code_b) + 2 * R * K * (gd + 1) * 4,
    }


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi during the timed region."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- CPU oracle arm

def oracle_step(w, oracle, n_sample):
    """The whole path on the CPU oracle over the first n_sample vectors; returns seconds."""
    x = w.x[:n_sample].astype(np.float64)
    cb = w.codebooks.astype(np.float64)
    t0 = time.perf_counter()
    enc = oracle.encode(x, cb, w.group_dim, w.layout)
    oracle.decode(enc["codes"], enc["std_bits"], cb, w.dim, w.layout, out_dtype=oracle.BF16)
    oracle.ema_update(x, enc["codes"], cb, np.ones(cb.shape[:2]), cb.copy(), w.decay, w.eps, w.layout)
    return time.perf_counter() - t0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = rvq_synth.key_cache(tokens=args.tokens)
    # a bounded sample per step, sized from a calibration run so that all K steps take about 90 s
    t_cal = min(oracle_step(w, oracle, 512) for _ in range(max(1, args.warmup)))
    n_sample = int(min(w.n, max(64, 90.0 / max(1, args.steps) / (t_cal / 512))))
    times = [oracle_step(w, oracle, n_sample) for _ in range(args.steps)]
    t = sum(times)
    value = n_sample * args.steps / t / 1e6
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": workload_name(args.tokens), "sample": f"first {n_sample} of {w.n} head vectors per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": f"first {n_sample} of {w.n} head vectors per step, {args.steps} steps"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- CUDA arm

def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2410_15704_b200 as rvq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # every rank works on its own seeded batch of the same shape (weak scaling)
    w = rvq_synth.key_cache(tokens=args.tokens, seed=1002 + rank)
    base = rvq_synth.key_cache(tokens=8, seed=1002)      # shared initial codebooks
    w.codebooks = base.codebooks
    cfg = rvq.make_config(w.dim, w.group_dim, w.layout, w.depth, w.codebook_size, w.code_bits, rvq.BF16, 0)
    n, R, K, gd = w.n, w.depth, w.codebook_size, w.group_dim
    alg = algorithmic_numbers(w)

    b = rvq.alloc_buffers(cfg, n, w.codebooks)
    x_host = torch.from_numpy(w.x_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
    x_dev = x_host.cuda()
    recon = torch.empty(n, w.dim, dtype=torch.bfloat16, device="cuda")
    ema_count = torch.ones(R, K, device="cuda")
    ema_sum = b.codebooks.clone()
    stats = torch.empty(R * K * (gd + 1), device="cuda")      # batch counts then batch sums, one all-reduce
    bcount, bsum = stats[:R * K], stats[R * K:]
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    codes_host = torch.empty_like(b.codes, device="cpu").pin_memory()
    std_host = torch.empty_like(b.std, device="cpu").pin_memory()
    recon_host = torch.empty_like(recon, device="cpu").pin_memory()
    cb0 = b.codebooks.clone()

    phases = ("prepare", "encode", "decode", "ema")
    ev = {p: [] for p in phases}

    def step(x, timed=False, out=None):
        codes, std, rec = out if out is not None else (b.codes, b.std, recon)
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(5)] if timed else None
        if timed: marks[0].record()
        rvq.rvq_prepare_codebooks(cfg, b.codebooks, b.prepared)
        if timed: marks[1].record()
        # encode and, in the same pass, this batch's EMA statistics
        rvq.rvq_encode_stats(cfg, x, n, w.dim, b.codebooks, b.prepared, codes, std, bcount, bsum,
                             b.workspace, b.workspace_bytes, b.status)
        if timed: marks[2].record()
        rvq.rvq_decode(cfg, codes, std, n, b.codebooks, b.prepared, rec, w.dim, b.status)
        if timed: marks[3].record()
        if world > 1:
            dist.all_reduce(stats)          # counts and sums share one buffer: a single collective
        rvq.rvq_ema_apply(cfg, bcount, bsum, b.codebooks, ema_count, ema_sum, w.decay, w.eps)
        if timed: marks[4].record()
        return marks

    def reset_state():
        b.codebooks.copy_(cb0); ema_sum.copy_(cb0); ema_count.fill_(1.0)

    def timed_loop(steps):
        """K device-resident steps; L2 flushed (untimed) before each; returns per-step ms list."""
        starts, ends, marks_all = [], [], []
        for _ in range(steps):
            flush.fill_(1)
            s_, e_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s_.record()
            marks_all.append(step(x_dev, timed=True))
            e_.record()
            starts.append(s_); ends.append(e_)
        torch.cuda.synchronize()
        ms = [s_.elapsed_time(e_) for s_, e_ in zip(starts, ends)]
        for m in marks_all:
            for i, p in enumerate(phases):
                ev[p].append(m[i].elapsed_time(m[i + 1]))
        return ms

    # End to end: every step copies its input in from pinned host memory and its codes, deviations and
    # reconstruction back out.  The copies run on streams of their own and the device buffers are doubled,
    # so step k's copy-out and step k+1's copy-in overlap step k+1's / step k's kernels (the codebooks
    # still pass from one step to the next: the kernels themselves stay in order on one stream).
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    x_slot = [x_dev, torch.empty_like(x_dev)]
    out_slot = [(b.codes, b.std, recon),
                (torch.empty_like(b.codes), torch.empty_like(b.std), torch.empty_like(recon))]

    def e2e_loop(steps):
        """K pipelined end-to-end steps; returns the total ms from the first copy-in to the last copy-out."""
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        done_k = [None, None]        # kernels of the step that last used slot i
        out_k = [None, None]         # copy-out of the step that last used slot i
        t0.record(main)
        s_in.wait_stream(main)
        s_out.wait_stream(main)
        for k in range(steps):
            i = k & 1
            with torch.cuda.stream(s_in):
                if done_k[i] is not None:
                    s_in.wait_event(done_k[i])                 # the kernels that read this input slot
                x_slot[i].copy_(x_host, non_blocking=True)
                arrived = torch.cuda.Event()
                arrived.record(s_in)
            main.wait_event(arrived)
            if out_k[i] is not None:
                main.wait_event(out_k[i])                      # this output slot has been copied out
            step(x_slot[i], out=out_slot[i])
            done_k[i] = torch.cuda.Event()
            done_k[i].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(done_k[i])
                codes_host.copy_(out_slot[i][0], non_blocking=True)
                std_host.copy_(out_slot[i][1], non_blocking=True)
                recon_host.copy_(out_slot[i][2], non_blocking=True)
                out_k[i] = torch.cuda.Event()
                out_k[i].record(s_out)
        main.wait_stream(s_out)
        main.wait_stream(s_in)
        t1.record(main)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(v):
        if world == 1:
            return v
        t = torch.tensor([v], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    # warm-up
    reset_state()
    for _ in range(max(3, args.warmup)):
        flush.fill_(1)
        step(x_dev)
    barrier()

    # device-resident timing
    reset_state()
    sampler = ClockSampler(local)
    launches0 = rvq.rvq_launch_count()
    barrier()
    if rank == 0:
        sampler.start()
    t_wall = time.perf_counter()
    ms = timed_loop(args.steps)
    barrier()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop() if rank == 0 else None
    launches = rvq.rvq_launch_count() - launches0
    total_ms = max_over_ranks(sum(ms))
    st = rvq.read_status(b.status)

    # end to end: pinned host input copied in, codes + std + reconstruction copied out, every step
    reset_state()
    e2e_loop(3)
    barrier()
    e2e_ms = max_over_ranks(e2e_loop(args.steps))
    barrier()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    enc_ms = statistics.mean(ev["encode"])
    dec_ms = statistics.mean(ev["decode"])
    ema_ms = statistics.mean(ev["ema"])
    enc_tflops = alg["encode_flops"] / (enc_ms * 1e-3) / 1e12
    tensor_peak = peaks["bf16_tflops"]          # burst: the encode kernel runs alone in a ~ms step
    line = {
        "metric": METRIC, "value": n * world * args.steps / (total_ms * 1e-3) / 1e6, "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 (f16 tensor-core operands, f32 accumulate)", "data": "synthetic",
        "config": {"workload": workload_name(args.tokens), "vectors_per_gpu": n, "l2": "flushed (256 MB write) before every timed step",
                   "timing": "CUDA events around each step on the launch stream, summed over K steps"},
        "phases": {
            "encode": {"ms": enc_ms, "Mvectors/s": n / enc_ms / 1e3, "TFLOP/s": enc_tflops,
                       "note": "encode kernel with fused EMA statistics, plus two memsets and a count conversion"},
            "decode": {"ms": dec_ms, "GB/s": alg["decode_bytes"] / dec_ms / 1e6,
                       "frac_hbm": alg["decode_bytes"] / dec_ms / 1e6 / peaks["hbm_gbs"]},
            "ema_apply": {"ms": ema_ms, "note": "statistics are accumulated inside the encode kernel"},
            "prepare": {"ms": statistics.mean(ev["prepare"])},
        },
        "roofline": {"kernel": "encode", "bound": "tensor", "achieved": enc_tflops, "peak": tensor_peak,
                     "unit": "TFLOP/s", "frac": enc_tflops / tensor_peak, "traffic": ENCODE_DRAM_TRAFFIC.get(args.tokens),
                     "peak_source": f"{peaks['source']} bf16 burst x1 (f16 operands, same rate)"},
        "e2e": {"value": n * world * args.steps / (e2e_ms * 1e-3) / 1e6, "unit": UNIT,
                "h2d_bytes_per_step": x_host.numel() * 2,
                "d2h_bytes_per_step": codes_host.numel() + std_host.numel() * 2 + recon_host.numel() * 2,
                "note": "copies on their own streams with doubled device buffers: they overlap the neighbouring "
                        "steps' kernels; L2 is not flushed in this loop (the input arrives from the host every step)"},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "device_status": st,
        "wall_s_timed_region": t_wall,
    }

    if world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        # the oracle as it stands on the host cores: whole batches until about 10 s have passed
        t, reps, n_cpu = 0.0, 0, min(n, 32768)
        while t < 10.0 and reps < 12:
            t += oracle_step(w, oracle, n_cpu)
            reps += 1
        line["cpu_baseline"] = {"value": n_cpu * reps / t / 1e6, "unit": UNIT, "cores": oracle.threads(),
                                "kind": "oracle",
                                "sample": f"{reps} steps over the first {n_cpu} of {n} head vectors ({t:.1f} s)"}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tokens", type=int, default=4096,
                    help="tokens per GPU of the key-cache recipe (default: the quoted workload, 4096)")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args)
    else:
        args.steps = 3000 if args.steps is None else args.steps
        args.warmup = 5 if args.warmup is None else args.warmup
        run_ours(args)


if __name__ == "__main__":
    main()
