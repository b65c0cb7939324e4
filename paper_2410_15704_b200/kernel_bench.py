#!/usr/bin/env python
"""Per-kernel timings of the residual-VQ library on one GPU, one JSON line per case.

  python paper_2410_15704_b200/kernel_bench.py encode key_cache:4096 value_cache:32768 tiny:4096
  python paper_2410_15704_b200/kernel_bench.py decode decode_bandwidth:131072
  python paper_2410_15704_b200/kernel_bench.py decode_rope decode_bandwidth:131072
  python paper_2410_15704_b200/kernel_bench.py attention decode_bandwidth:131072
  python paper_2410_15704_b200/kernel_bench.py ema ema_learning:131072
  python paper_2410_15704_b200/kernel_bench.py learn_step ema_learning:131072
  python paper_2410_15704_b200/kernel_bench.py kmeans ema_learning:131072 --iterations 10
  python paper_2410_15704_b200/kernel_bench.py encode ablation:32768 --shape 128,32,6,1024

A case is `<workload>:<tokens>` (workload names of `rvq_synth`; `tiny:<n>` takes a vector count).  Each
launch is timed with CUDA events on the launching stream after three warm-up launches; before every timed
launch a 256 MB buffer is written so that nothing of the inputs is left in L2.  `--reps N` launches are timed
and the median and the best are printed.  Encode reports useful flops (2·group_dim·K·R·G per vector)
against the dense bf16 peak, decode and EMA report algorithmic bytes against the copy bandwidth; both peaks
come from MEASURED_PEAKS.json beside the package when it exists.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

import paper_2410_15704_b200 as rvq  # noqa: E402
import rvq_synth  # noqa: E402


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p["hbm_gbs"], p["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


def make(spec, **kw):
    name, count = spec.split(":")
    w = rvq_synth.tiny(int(count)) if name == "tiny" else rvq_synth.WORKLOADS[name](int(count), **kw)
    return name, w


def timed(fn, reps, flush):
    for _ in range(3):
        fn()
    ts = []
    for _ in range(reps):
        flush.fill_(1)
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        fn()
        e.record()
        torch.cuda.synchronize()
        ts.append(s.elapsed_time(e))
    return statistics.median(ts), min(ts)


def config_of(w, bits=None):
    dt = {"f32": rvq.F32, "bf16": rvq.BF16, "f16": rvq.F16}
    return rvq.make_config(w.dim, w.group_dim, w.layout, w.depth, w.codebook_size,
                           w.code_bits if bits is None else bits, dt[w.out_dtype if w.x is None else w.x_dtype], 0)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kernel", choices=["encode", "encode_stats", "encode_exact", "decode", "decode_rope", "attention", "ema",
                                       "learn_step", "kmeans"])
    ap.add_argument("--iterations", type=int, default=10, help="Lloyd iterations per stage (kmeans)")
    ap.add_argument("--shape", default=None,
                    help="dim,group_dim,depth,codes[,layout] of the `ablation` workload, e.g. 128,32,6,1024")
    ap.add_argument("--codes", type=int, default=None, help="codes per stage, for workloads that take a size")
    ap.add_argument("cases", nargs="+")
    ap.add_argument("--reps", type=int, default=10)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("kernel_bench.py needs a CUDA device: there is no CPU fallback")
    hbm, tensor, src = peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    for spec in args.cases:
        if args.kernel == "attention":
            runs = [make(spec, layout=1)]
        elif args.kernel in ("decode", "decode_rope") and spec.startswith("decode_bandwidth"):
            runs = [make(spec, layout=0), make(spec, layout=1)]
        elif spec.startswith("ablation") and args.shape:
            f = [int(t) for t in args.shape.split(",")]
            runs = [make(spec, dim=f[0], group_dim=f[1], depth=f[2], size=f[3], layout=f[4] if len(f) > 4 else 0)]
        elif args.codes:
            runs = [make(spec, size=args.codes)]
        else:
            runs = [make(spec)]
        for name, w in runs:
            n, G, R, K, gd = w.n, w.groups, w.depth, w.codebook_size, w.group_dim
            code_b = (G * R * w.code_bits + 31) // 32 * 4
            line = {"kernel": args.kernel, "workload": name, "vectors": n, "dim": w.dim, "group_dim": gd, "K": K, "R": R,
                    "layout": "strided" if w.layout else "contiguous", "code_bits": w.code_bits}
            if args.kernel == "attention":
                # one new token (32 query heads, 8 kv heads) over a cache of n / 8 tokens: the workload's codes as
                # keys on strided groups (half-split rotary pairs, position = token index), the same codes read as
                # values on contiguous groups
                tokens = n // 8
                cfg_k = rvq.make_config(w.dim, gd, rvq_synth.STRIDED, R, K, w.code_bits, rvq.BF16, 0)
                cfg_v = rvq.make_config(w.dim, gd, rvq_synth.CONTIGUOUS, R, K, w.code_bits, rvq.BF16, 0)
                b = rvq.alloc_buffers(cfg_k, n, w.codebooks)
                b.codes.view(torch.int16)[: n * G * R].copy_(
                    torch.from_numpy(w.codes.astype(np.uint16).view(np.int16).reshape(-1)))
                b.std.copy_(torch.from_numpy(w.std_bits.view(np.int16)))
                q = torch.from_numpy(np.random.default_rng(1).normal(size=(32, w.dim)).astype(np.float32)).cuda()
                table = torch.empty(tokens, w.dim // 2, 2, device="cuda")
                rvq.rvq_rope_table(w.dim, 500000.0, tokens, table)
                ws_bytes = rvq.rvq_attention_workspace_bytes(tokens, 32)
                ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
                out = torch.empty(32, w.dim, device="cuda")
                med, best = timed(lambda: rvq.rvq_attention_decode(cfg_k, cfg_v, q, 32, b.codes, b.std, b.codes, b.std, tokens,
                                                                   8, b.codebooks, b.codebooks, None, table, tokens,
                                                                   rvq.ROPE_HALVES, float(w.dim) ** -0.5, out, ws, ws_bytes,
                                                                   b.status), args.reps, flush)
                nbytes = 2 * n * (code_b + 2) + tokens * (w.dim // 2) * 8          # both caches' codes and deviations, the table
                line.update(tokens=tokens, ms_median=med, ms_best=best, cached_vectors_per_s=2 * n / med / 1e3, bytes=nbytes,
                            GBps=nbytes / med / 1e6, frac_hbm=nbytes / med / 1e6 / hbm, peak=hbm, peak_source=src,
                            decoded_bytes_never_written=2 * n * w.dim * 2)
                line.update(rvq.read_status(b.status))
                print(json.dumps(line), flush=True)
                continue
            if args.kernel in ("decode", "decode_rope"):
                cfg = config_of(w)
                b = rvq.alloc_buffers(cfg, n, w.codebooks)
                tdt = rvq.TORCH_DTYPE[cfg.x_dtype]
                if getattr(w, "codes", None) is not None:
                    codes, std_bits = w.codes, w.std_bits
                else:   # a workload without stored codes: encode it first
                    x = torch.from_numpy(w.x).to(tdt).cuda()
                    rvq.rvq_encode(cfg, x, n, w.dim, b.codebooks, b.prepared, b.codes, b.std,
                                   b.workspace, b.workspace_bytes, b.status)
                    codes = std_bits = None
                if codes is not None:
                    cfg = config_of(w, bits=16)
                    code_b = G * R * 2
                    b = rvq.alloc_buffers(cfg, n, w.codebooks)
                    b.codes.view(torch.int16)[: n * G * R].copy_(
                        torch.from_numpy(codes.astype(np.uint16).view(np.int16).reshape(-1)))
                    b.std.copy_(torch.from_numpy(std_bits.view(np.int16)))
                out = torch.empty(n, w.dim, dtype=tdt, device="cuda")
                if args.kernel == "decode_rope":
                    # one position per token (all its heads), 128K context, Llama-3's base, half-split pairs
                    tokens, max_pos = n // w.heads, 131072
                    table = torch.empty(max_pos, w.dim // 2, 2, device="cuda")
                    rvq.rvq_rope_table(w.dim, 500000.0, max_pos, table)
                    pos = (torch.arange(tokens, device="cuda", dtype=torch.int32) % max_pos).contiguous()
                    med, best = timed(lambda: rvq.rvq_decode_rope(cfg, b.codes, b.std, n, b.codebooks, b.prepared, pos, w.heads,
                                                                  table, max_pos, rvq.ROPE_HALVES, out, w.dim,
                                                                  b.status), args.reps, flush)
                    extra = w.dim // 2 * 8 // w.heads + 4 // w.heads      # a table row and a position per token
                else:
                    med, best = timed(lambda: rvq.rvq_decode(cfg, b.codes, b.std, n, b.codebooks, b.prepared, out,
                                                             w.dim, b.status), args.reps, flush)
                    extra = 0
                nbytes = n * (code_b + 2 + w.dim * out.element_size() + extra)
                line.update(ms_median=med, ms_best=best, bytes=nbytes, GBps=nbytes / med / 1e6,
                            frac_hbm=nbytes / med / 1e6 / hbm, peak=hbm, peak_source=src)
            else:
                cfg = config_of(w)
                b = rvq.alloc_buffers(cfg, n, w.codebooks)
                x = torch.from_numpy(w.x).to(rvq.TORCH_DTYPE[cfg.x_dtype]).cuda()
                bc = torch.empty(R, K, device="cuda")
                bs = torch.empty(R, K, gd, device="cuda")
                if args.kernel == "learn_step":
                    cb0 = b.codebooks.clone()
                    ema_n, ema_m = torch.ones(R, K, device="cuda"), b.codebooks.clone()
                    fn = lambda: rvq.rvq_learn_step(cfg, x, n, w.dim, b.codebooks, b.prepared, ema_n, ema_m, b.codes,
                                                    b.std, w.decay, w.eps, b.workspace, b.workspace_bytes, b.status)
                elif args.kernel == "kmeans":
                    seeds = torch.from_numpy(np.stack([rvq_synth.randint(rvq_synth.stream_seed(w.seed, f"seed rows {r}"),
                                                                         K, n * G) for r in range(R)])).cuda()
                    nbytes = rvq.rvq_kmeans_workspace_bytes(cfg, n)
                    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
                    fn = lambda: rvq.rvq_kmeans_init(cfg, x, n, w.dim, seeds, args.iterations, b.codebooks, b.prepared,
                                                     ws, nbytes, b.status)
                elif args.kernel == "encode":
                    fn = lambda: rvq.rvq_encode(cfg, x, n, w.dim, b.codebooks, b.prepared, b.codes, b.std,
                                                b.workspace, b.workspace_bytes, b.status)
                elif args.kernel == "encode_exact":
                    fn = lambda: rvq.rvq_encode_exact(cfg, x, n, w.dim, b.codebooks, b.prepared, b.codes, b.std,
                                                      b.status)
                elif args.kernel == "encode_stats":
                    fn = lambda: rvq.rvq_encode_stats(cfg, x, n, w.dim, b.codebooks, b.prepared, b.codes, b.std,
                                                      bc, bs, b.workspace, b.workspace_bytes, b.status)
                else:
                    rvq.rvq_encode(cfg, x, n, w.dim, b.codebooks, b.prepared, b.codes, b.std,
                                   b.workspace, b.workspace_bytes, b.status)
                    fn = lambda: rvq.rvq_ema_stats(cfg, x, n, w.dim, b.codes, b.codebooks, bc, bs,
                                                   b.workspace, b.workspace_bytes, b.status)
                med, best = timed(fn, args.reps if args.kernel != "kmeans" else min(args.reps, 3), flush)
                if args.kernel == "kmeans":
                    # assignments made: every iteration of every stage, plus one per stage but the last
                    sweeps = R * args.iterations + R - 1
                    flops = 2.0 * gd * K * G * n * sweeps
                    line.update(ms_median=med, ms_best=best, iterations=args.iterations, assignment_passes=sweeps,
                                useful_TFLOPs=flops / med / 1e9, frac_tensor=flops / med / 1e9 / tensor,
                                peak=tensor, peak_source=src, workspace_bytes=nbytes,
                                wait_timeouts=rvq.read_status(b.status)["wait_timeouts"])
                elif args.kernel == "ema":
                    nbytes = n * (w.dim * x.element_size() + code_b) + 2 * R * K * (gd + 1) * 4
                    line.update(ms_median=med, ms_best=best, bytes=nbytes, GBps=nbytes / med / 1e6,
                                frac_hbm=nbytes / med / 1e6 / hbm, peak=hbm, peak_source=src)
                else:
                    flops = 2.0 * gd * K * R * G * n
                    st = rvq.read_status(b.status)
                    line.update(ms_median=med, ms_best=best, Mvectors_per_s=n / med / 1e3,
                                useful_TFLOPs=flops / med / 1e9, frac_tensor=flops / med / 1e9 / tensor,
                                peak=tensor, peak_source=src,
                                rescored_rows_per_launch=st["rescored_rows"] // (args.reps + 3),
                                exhaustive_rows=st["exhaustive_rows"], wait_timeouts=st["wait_timeouts"])
            print(json.dumps(line), flush=True)
            del b
            torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
