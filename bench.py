#!/usr/bin/env python
"""Benchmark of the ECQ-SGD gradient codec on B200.

One *step* is one pass of the whole hot path over one batch of synthetic
gradients: the fused encode of all W simulated workers (compensate, per-bucket
max-abs, stochastic rounding, accumulator update, bit-pack; one batched launch
of the encode kernel) followed by one fused decode-mean over the W messages.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
    python bench.py --impl reference      # the CPU oracle on a bounded sample

Prints ONE JSON line.  ``value`` is algorithmic GB/s of the whole step with
inputs resident in HBM; ``e2e`` is the same metric through ``ecq_step_host``
with host buffers (copies inside the timed region); ``roofline`` describes the
dominant kernel (the tiled encode) against the measured HBM copy rate;
``cpu_baseline`` is the oracle timed on the host cores on a bounded sample.
With N > 1 every rank runs an independent replica (the path has no exchange
step on one node); the reported time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_1806_08054_b200 import workloads as wl  # noqa: E402

METRIC = "codec_step_throughput"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes per entry of the batched tiled encode kernel from an ncu capture of the default
# workload's own launch (dram__bytes_read.sum + dram__bytes_write.sum = 141,431,158,016 bytes
# over 11,310,497,792 entries; see profiles/encode_tiled_kernel.md), keyed by (bucket, levels).
# Traffic grows in proportion to the entries of a launch.  Set an entry to None when the
# kernel changes.
NCU_DRAM_BYTES_PER_ENTRY = {(512, 4): 141431376025 / 11310497792}


def code_bits(s: int) -> int:
    return (2 * s).bit_length()


def step_bytes(w: wl.Workload):
    """Algorithmic bytes of one step: (encode per launch, decode)."""
    r = code_bits(w.s)
    nb = -(-w.d // w.bucket)
    words = -(-w.d * r // 32)
    enc = 12 * w.d + 4 * words + 4 * nb          # g, h read; h write; codes, scales write
    dec = w.W * (4 * words + 4 * nb) + 4 * w.d   # W messages read; mean written
    return enc, dec


def hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while timing."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower() == "active":
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    return rank, local, world


def max_over_ranks(values, world):
    """Element-wise maximum of a list of floats over all ranks."""
    if world == 1:
        return list(values)
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor(values, dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def cpu_oracle_sample(w: wl.Workload, sample_elems: int, sample_workers: int):
    """Time the oracle, as it stands, on a bounded sample of the workload."""
    import numpy as np
    import oracle
    n = min(sample_elems, w.d) // w.bucket * w.bucket or w.d
    Ws = min(sample_workers, w.W)
    gs = [wl.gradient(wl.scaled(w, n), p, 0, "cpu").numpy() for p in range(Ws)]
    hs = [np.zeros(n, np.float32) for _ in range(Ws)]
    t0 = time.perf_counter()
    msgs = [oracle.encode(gs[p], hs[p], bucket=w.bucket, s=w.s, alpha=w.alpha, beta=w.beta,
                          seed=wl.CODEC_SEED, worker=p, step=0) for p in range(Ws)]
    oracle.decode_mean([m[0] for m in msgs], [m[1] for m in msgs], n=n, bucket=w.bucket, s=w.s)
    dt = time.perf_counter() - t0
    sw = wl.Workload(w.name, w.index, Ws, n, w.bucket, w.s, w.alpha, w.beta, 1, w.kind)
    enc, dec = step_bytes(sw)
    return {"value": (Ws * enc + dec) / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": "%d workers x first %d entries of %s, 1 step (encode+decode), %.1f s"
                      % (Ws, n, w.name, dt),
            "elements_per_s": Ws * n / dt}, dt


def entropy_coded_message(ctx, codes, counts_host, w):
    """Huffman-code one worker's message with the library's coder (outside the timed step):
    message size and the time of the coder's launches."""
    import paper_1806_08054_b200 as ecq
    lengths = ecq.ecq_huffman_lengths(ctx, counts_host)
    cap = ecq.ecq_huffman_stream_bound(ctx, counts_host, lengths)
    n_chunks = ecq.ecq_huffman_chunks(ctx)
    tables = torch.zeros(ecq.ECQ_HUFFMAN_TABLE_BYTES, dtype=torch.uint8, device="cuda")
    stream = torch.zeros(cap, dtype=torch.int32, device="cuda")
    offsets = torch.zeros(n_chunks + 1, dtype=torch.int32, device="cuda")
    quarters = torch.zeros(3 * n_chunks, dtype=torch.int16, device="cuda")
    back = torch.zeros_like(codes)
    ecq.ecq_huffman_tables(ctx, lengths, tables)

    def timed(fn, reps=5):
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    enc_ms = timed(lambda: ecq.ecq_huffman_encode(ctx, tables, codes, stream, offsets, quarters))
    dec_ms = timed(lambda: ecq.ecq_huffman_decode(ctx, tables, stream, offsets, quarters, back))
    if not torch.equal(back, codes):
        raise SystemExit("entropy-coded message does not decode to the codes")
    words = int(offsets[-1].item()) & 0xFFFFFFFF
    nb = -(-w.d // w.bucket)
    bits = 32.0 * words + 32.0 * (n_chunks + 1) + 48.0 * n_chunks + 4.0 * len(lengths) + 32.0 * nb
    return {"bits_per_entry": bits / w.d, "compression": 32.0 * w.d / bits,
            "payload_bits_per_entry": sum(c * l for c, l in zip(counts_host, lengths)) / w.d,
            "encode_ms": enc_ms, "decode_ms": dec_ms,
            "encode_entries_per_s": w.d / (enc_ms * 1e-3), "decode_entries_per_s": w.d / (dec_ms * 1e-3),
            "includes": "stream, chunk offsets, quarter marks, 4-bit code lengths, fp32 scales"}


def run_reference(args, w):
    rank, _, world = dist_env()
    if rank != 0:
        return
    Ws = 2
    times, last = [], None
    for i in range(args.warmup + args.steps):
        cb, dt = cpu_oracle_sample(w, args.ref_elems, Ws)
        if i >= args.warmup:
            times.append(dt)
            last = cb
    n = min(args.ref_elems, w.d) // w.bucket * w.bucket or w.d
    Ws = min(Ws, w.W)
    sw = wl.Workload(w.name, w.index, Ws, n, w.bucket, w.s, w.alpha, w.beta, 1, w.kind)
    enc, dec = step_bytes(sw)
    total = sum(times)
    value = (Ws * enc + dec) * len(times) / total / 1e9
    last["value"] = value
    vals = times
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * total / len(vals), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "W": w.W, "d": w.d, "bucket": w.bucket, "s": w.s,
                       "note": "CPU oracle, single thread, bounded sample per step"},
            "cpu_baseline": last,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="lm_350m", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--bucket", type=int, default=0)
    ap.add_argument("--levels", type=int, default=0)
    ap.add_argument("--workers", type=int, default=0, help="override W (smaller runs)")
    ap.add_argument("--decode-kernel", default="auto", choices=["auto", "warp", "ring"],
                    help="receiver kernel (ecq_set_decode_plan); auto = the library's choice")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-elems", type=int, default=1 << 25)
    ap.add_argument("--ref-elems", type=int, default=1 << 22)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    w = wl.WORKLOADS[args.workload]
    if args.bucket or args.levels:
        w = wl.with_codec(w, args.bucket or w.bucket, args.levels or w.s)
    if args.workers:
        w = wl.Workload(w.name, w.index, args.workers, w.d, w.bucket, w.s, w.alpha, w.beta,
                        w.steps, w.kind, w.layers)

    if args.impl == "reference":
        run_reference(args, w)
        return

    import paper_1806_08054_b200 as ecq
    rank, local, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the codec has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    warmup = max(args.warmup, 3)

    d, W = w.d, w.W
    ctx = ecq.ecq_create(d, w.bucket, w.s, w.alpha, w.beta, wl.CODEC_SEED)
    ecq.ecq_set_decode_plan(ctx, {"auto": ecq.ECQ_DECODE_AUTO, "warp": ecq.ECQ_DECODE_WARP,
                                  "ring": ecq.ECQ_DECODE_RING}[args.decode_kernel], 0)
    r = ecq.ecq_code_bits(ctx)
    nw, nb = ecq.ecq_codes_words(ctx), ecq.ecq_num_buckets(ctx)
    enc_bytes, dec_bytes = step_bytes(w)

    # device-resident state and inputs
    err = torch.zeros(W * d, device="cuda")
    codes = [torch.zeros(nw, dtype=torch.int32, device="cuda") for _ in range(W)]
    scales = [torch.zeros(nb, device="cuda") for _ in range(W)]
    out = torch.zeros(d, device="cuda")
    ws_bytes = 0 if args.no_e2e else ecq.ecq_step_host_workspace_bytes(ctx, W)
    free, _ = torch.cuda.mem_get_info()
    G = int(max(1, min(W, (free - ws_bytes - (4 << 30)) // (d * 4 * 2))))
    grads = [wl.gradient(w, p + 1000 * rank, 0, "cuda") for p in range(G)]
    torch.cuda.synchronize()

    errs = [err[p * d:(p + 1) * d] for p in range(W)]
    grad_list = [grads[p % G] for p in range(W)]

    def step(t):
        # all W workers' encodes as one batched launch, then the decode-mean
        ecq.ecq_encode_batch(ctx, t, grad_list, errs, codes, scales)
        ev_mid = torch.cuda.Event(enable_timing=True)
        ev_mid.record()
        ecq.ecq_decode_mean(ctx, codes, scales, out)
        return ev_mid

    for t in range(warmup):
        step(t)
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ecq.ecq_launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    mids = []
    torch.cuda.synchronize()
    ev[0].record()
    for t in range(args.steps):
        mids.append(step(warmup + t))
        ev[t + 1].record()
    torch.cuda.synchronize()
    launches = ecq.ecq_launch_count() - launches0
    if world > 1:
        dist.barrier()
    total_ms = ev[0].elapsed_time(ev[-1])
    enc_ms = sum(ev[t].elapsed_time(mids[t]) for t in range(args.steps))
    dec_ms = sum(mids[t].elapsed_time(ev[t + 1]) for t in range(args.steps))
    # level statistics of worker 0's last message (outside the timed region)
    counts = torch.zeros(2 * w.s + 1, dtype=torch.int64, device="cuda")
    ecq.ecq_code_histogram(ctx, codes[0], counts)
    counts_host = counts.cpu().tolist()
    entropy_bits = ecq.ecq_entropy_bound_bits(counts_host)
    huffman = entropy_coded_message(ctx, codes[0], counts_host, w) if w.s <= 2047 else None
    status = ecq.ecq_status(ctx)
    if status != ecq.ECQ_OK:
        raise SystemExit("codec status %d: %s" % (status, ecq.binding.strerror(status)))
    total_ms, enc_ms, dec_ms = max_over_ranks([total_ms, enc_ms, dec_ms], world)
    clocks = sampler.stop() if rank == 0 else None

    # end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        Gh = min(G, 2)
        hosts = [grads[p].cpu().pin_memory() for p in range(Gh)]
        out_host = torch.empty(d).pin_memory()
        host_list = [hosts[p % Gh] for p in range(W)]
        err.zero_()
        ecq.ecq_step_host(ctx, 0, host_list, err, ws, out_host)       # warm-up
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for t in range(args.e2e_steps):
            ecq.ecq_step_host(ctx, 1 + t, host_list, err, ws, out_host)
        e1.record()
        torch.cuda.synchronize()
        (e2e_ms,) = max_over_ranks([e0.elapsed_time(e1)], world)
        e2e = {"value": world * (W * enc_bytes + dec_bytes) * args.e2e_steps / (e2e_ms * 1e-3) / 1e9,
               "unit": UNIT, "h2d_bytes_per_step": W * d * 4, "d2h_bytes_per_step": d * 4,
               "ms_per_step": e2e_ms / args.e2e_steps, "steps": args.e2e_steps,
               "host_gradient_buffers": Gh}
        del ws

    if rank == 0:
        peak, how = hbm_peak()
        step_b = W * enc_bytes + dec_bytes
        value = world * step_b * args.steps / (total_ms * 1e-3) / 1e9
        enc_gbs = enc_bytes * W * args.steps / (enc_ms * 1e-3) / 1e9
        dec_gbs = dec_bytes * args.steps / (dec_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": warmup, "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "W": W, "d": d, "bucket": w.bucket, "s": w.s,
                       "code_bits": r, "alpha": w.alpha, "beta": w.beta,
                       "distinct_gradient_buffers": G,
                       "l2": ("inputs larger than L2 (%.1f GB touched per step)" % (step_b / 1e9)
                              if step_b > 4 * 126e6 else
                              "L2-resident workload (%.2f GB per step, 126 MB L2, no flush): "
                              "launch-bound, reported for completeness only" % (step_b / 1e9)),
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "elements_per_s": world * W * d * args.steps / (total_ms * 1e-3),
            "encode": {"GB/s": enc_gbs, "elements_per_s": W * d * args.steps / (enc_ms * 1e-3),
                       "ms_per_launch": enc_ms / args.steps, "workers_per_launch": W,
                       "frac_of_measured_copy": enc_gbs / peak,
                       "frac_of_nominal_8TBs": enc_gbs / NOMINAL_HBM_GBS},
            "decode": {"GB/s": dec_gbs, "outputs_per_s": d * args.steps / (dec_ms * 1e-3),
                       "ms_per_launch": dec_ms / args.steps,
                       "frac_of_measured_copy": dec_gbs / peak,
                       "frac_of_nominal_8TBs": dec_gbs / NOMINAL_HBM_GBS},
            "roofline": {"kernel": "encode_tiled_kernel", "bound": "hbm", "achieved": enc_gbs,
                         "peak": peak, "peak_source": "of " + how, "unit": "GB/s",
                         "frac": enc_gbs / peak,
                         "traffic": (NCU_DRAM_BYTES_PER_ENTRY[(w.bucket, w.s)] * W * d
                                     if NCU_DRAM_BYTES_PER_ENTRY.get((w.bucket, w.s)) else None),
                         "algorithmic_bytes_per_launch": W * enc_bytes},
            "message": {"fixed_bits_per_entry": r + 32.0 / w.bucket,
                        "compression_fixed": 32.0 / (r + 32.0 / w.bucket),
                        "entropy_bound_bits_per_entry": (entropy_bits + 32.0 * nb) / d,
                        "compression_entropy_bound": 32.0 * d / (entropy_bits + 32.0 * nb),
                        "huffman": huffman,
                        "note": "worker 0, last timed step; the paper's Table 1 ratios are "
                                "entropy-coded on other workloads (context only)"},
            # the decode kernel's own bound: one logic instruction per code on the ALU pipe
            # (16 lanes per clock per SM sub-partition)
            "decode_roofline": {"kernel": "decode kernel (%s)" % args.decode_kernel, "bound": "alu",
                                "achieved": W * d * args.steps / (dec_ms * 1e-3) / 1e12,
                                "peak": 148 * 4 * 16 * 1.965e9 / 1e12, "unit": "Tcodes/s",
                                "frac": (W * d * args.steps / (dec_ms * 1e-3)) / (148 * 4 * 16 * 1.965e9),
                                "peak_source": "derived: 148 SMs x 4 x 16 lanes x 1.965 GHz, "
                                               "1 logic op per code"},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if e2e:
            line["e2e"] = e2e
        if world == 1 and not args.no_cpu:
            line["cpu_baseline"], _ = cpu_oracle_sample(w, args.cpu_elems, 4)
        print(json.dumps(line))
    ecq.ecq_destroy(ctx)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
