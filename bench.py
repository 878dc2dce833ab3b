#!/usr/bin/env python
"""Benchmark of the batched AED decoder: output tokens/s and RTFx on synthetic Canary-style workloads.

    python bench.py --gpus 1 --steps 5 --warmup 3                 # this library
    python bench.py --impl reference --steps 2 --warmup 1         # the CPU checker, as a baseline

One "step" is one pass of the whole hot path over one batch: cross-K/V precompute followed by greedy
decoding of every utterance to its forced length.  Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2503_05931_b200 import workloads as wl   # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


# Bytes per element of the cross-attention K/V store when it is not the workload's dtype (--cross-kv e4m3: 1).
CROSS_KV_BYTES = None


def step_bytes_and_flops(w):
    """Algorithmic bytes and flops of greedy decoding, step by step (weights once per step, each active row's
    own self and cross K/V once per layer), and of the cross-K/V precompute."""
    m = w.model
    e = 2 if w.dtype == "bf16" else 4
    NL, d, F, V, de = m["n_layers"], m["d_model"], m["d_ffn"], m["vocab"], m["d_enc"]
    step_params = NL * (4 * d * d + 2 * d * d + 2 * d * F) + V * d
    T, L = w.enc_lens.astype(np.int64), w.dec_lens.astype(np.int64)
    ec = CROSS_KV_BYTES or e
    per_step = []
    for s in range(int(L.max())):
        act = L > s
        n = int(act.sum())
        kv_pos = int((T[act] + s + 1).sum())
        kv_bytes = NL * 2 * d * (ec * int(T[act].sum()) + e * int((act.sum()) * (s + 1)))
        per_step.append((e * step_params + kv_bytes, 2 * n * step_params + 4 * d * NL * kv_pos, n))
    total_T = int(T.sum())
    pre_flops = 2 * total_T * de * NL * 2 * d
    pre_bytes = e * (total_T * de + NL * 2 * d * de) + ec * total_T * NL * 2 * d
    return per_step, pre_bytes, pre_flops, step_params


def family_bytes(family, w):
    """Algorithmic bytes one whole pass (precompute + greedy decode) moves in the launches of a kernel family."""
    m = w.model
    e = 2 if w.dtype == "bf16" else 4
    NL, d, F, V, de = m["n_layers"], m["d_model"], m["d_ffn"], m["vocab"], m["d_enc"]
    T, L = w.enc_lens.astype(np.int64), w.dec_lens.astype(np.int64)
    steps = int(L.max())
    per_layer_weights = {"gemm_qkv": 3 * d * d, "gemm_o": d * d, "gemm_qc": d * d, "gemm_oc": d * d,
                         "gemm_ff1": d * F, "gemm_ff2": d * F, "ffn": 2 * d * F}
    if family in per_layer_weights:
        return e * per_layer_weights[family] * NL * steps
    if family == "gemm_vocab":
        return e * V * d * steps
    if family == "attn_cross":
        return sum((CROSS_KV_BYTES or e) * NL * 2 * d * int(T[L > s].sum()) for s in range(steps))
    if family == "attn_self":
        return sum(e * NL * 2 * d * int((L > s).sum()) * (s + 1) for s in range(steps))
    if family == "precompute_cross_kv":
        total_T = int(T.sum())
        return e * (total_T * de + NL * 2 * d * de) + (CROSS_KV_BYTES or e) * total_T * NL * 2 * d
    return None


# Which kernel a launch family runs (the library times launches per call site; the projections of a layer are
# five or six call sites of one kernel).
KERNEL_OF_FAMILY = {
    "gemm_qkv": "step_gemm_kernel", "gemm_o": "step_gemm_kernel", "gemm_qc": "step_gemm_kernel",
    "gemm_oc": "step_gemm_kernel", "gemm_ff1": "step_gemm_kernel", "gemm_ff2": "step_gemm_kernel",
    "attn_self": "attn_fused_kernel", "attn_cross": "attn_fused_kernel", "attn_combine": "attn_combine_kernel",
    "gemm_vocab": "tc_gemm_kernel", "precompute_cross_kv": "crosskv_gemm_kernel", "layernorm": "layernorm_planes_kernel",
    "embed": "embed_kernel", "bookkeeping": "build_active/finish_step",
}

# DRAM bytes per algorithmic byte of a kernel, from the ncu captures summarised under profiles/ (dram__bytes_read.sum +
# dram__bytes_write.sum of the captured launches over their algorithmic bytes).  An entry is removed when its kernel
# changes, which turns the reported traffic back into null.
NCU_TRAFFIC_RATIO = {
    # five launches of one layer at 128 rows (cfg3): 73.68 MB read for 29.36 MB of layer weights; the launches also read
    # the composite cross-query matrix (2.1 MB), the fp32 activation rows, and each prefetches the next layer's matrices
    # of its kind into L2, which under the profiler's serialised replay is a second DRAM read
    "step_gemm_kernel": 2.51,
    # the five launches at 16 and at 4 rows (cfg2): 63.24 MB and 62.97 MB read
    "step_gemv_staged_kernel": 2.15,
    "step_gemv_kernel": 2.14,
    # self + cross attention of one layer at 64 rows: 0.84 + 31.05 MB for 0.52 + 30.49 MB of K/V
    "attn_fused_kernel": 1.03,
    # vocabulary projection: 33.85 MB for the 33.55 MB output matrix (tcgen05 kernel; 33.79 MB in the few-row kernel)
    "tc_gemm_kernel": 1.01,
    "vocab_gemv_kernel": 1.01,
    # cross-K/V of 7444 frames: 117.2 MB read + 677.2 MB written for 847.7 MB (part of the output is still in L2 at exit)
    "crosskv_gemm_kernel": 0.94,
}


def roofline_seconds(w, peaks):
    per_step, pre_bytes, pre_flops, _ = step_bytes_and_flops(w)
    bw, fl = peaks["hbm_gbs"] * 1e9, peaks["bf16_tflops_sustained"] * 1e12
    dec = sum(max(b / bw, f / fl) for b, f, _ in per_step)
    pre = max(pre_bytes / bw, pre_flops / fl)
    return dec, pre


def reduce_over_ranks(total_ms: float, n_tok: float, n_frames: float, device: str, world: int):
    """Whole-job figures of a weak-scaling run: the slowest rank's time, tokens and frames summed over ranks.
    Ranks decode independent batches, so these two reductions are the only communication of the benchmark."""
    if world <= 1:
        return total_ms, n_tok, n_frames
    import torch
    import torch.distributed as dist
    t = torch.tensor([total_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor([n_tok, n_frames], dtype=torch.float64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return float(t.item()), float(c[0].item()), float(c[1].item())


def rank_seed(workload: str, rank: int) -> int:
    """Every rank draws its own batch from the same distribution."""
    return wl.BASE_SEED + wl._CONFIG_INDEX[workload] + 1000 * rank


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu_index)], stdout=self.file,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.file:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons), "samples": len(sm)}


def run_reference(args):
    """The CPU checker, as it stands (fp32 build, OpenMP over utterances), on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import aed_oracle as orc
    w = wl.make_workload(args.workload)
    cores = os.cpu_count() or 1
    rng = np.random.default_rng(1)
    short = np.flatnonzero(w.dec_lens <= 24)
    rows = sorted(int(r) for r in rng.choice(short, size=min(len(short), max(2, cores // 2)), replace=False))
    sub = w.subset(rows)
    model = orc.Model(w.model, w.weights, ln_eps=w.ln_eps)
    n_tok = int(sub.dec_lens.sum())
    times, threads = [], 1
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        out = orc.decode_batch(model, sub.enc, sub.enc_lens, sub.dec_lens, bos=w.bos_id, precision="f32")
        dt = time.perf_counter() - t0
        threads = out["threads"]
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = n_tok * len(times) / total
    sample = f"{len(rows)} utterances of {w.name} with at most 24 output tokens ({n_tok} tokens, {int(sub.enc_lens.sum())} frames) per step"
    line = {
        "impl": "reference", "metric": "decoder output tokens/s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, **w.model, "batch": w.batch, "weights": w.dtype, "sample": sample},
        "rtfx": float(sub.enc_lens.sum()) * wl.FRAME_SECONDS * len(times) / total,
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def cpu_baseline(w, budget_tokens: int = 0):
    """Time the CPU checker (fp32 build) on a bounded sample of the same workload."""
    from oracle import aed_oracle as orc
    cores = os.cpu_count() or 1
    rng = np.random.default_rng(2)
    rows = sorted(int(r) for r in rng.choice(w.batch, size=min(w.batch, cores), replace=False))
    sub = w.subset(rows)
    model = orc.Model(w.model, w.weights, ln_eps=w.ln_eps)
    t0 = time.perf_counter()
    out = orc.decode_batch(model, sub.enc, sub.enc_lens, sub.dec_lens, bos=w.bos_id, precision="f32")
    dt = time.perf_counter() - t0
    n_tok = int(sub.dec_lens.sum())
    return {"value": n_tok / dt, "unit": "tokens/s", "cores": int(out["threads"]), "kind": "oracle",
            "sample": f"{len(rows)} randomly chosen utterances of {w.name} ({n_tok} tokens, {int(sub.enc_lens.sum())} "
                      f"encoder frames), precompute + greedy decode, fp32 build, {dt:.1f} s",
            "rtfx": float(sub.enc_lens.sum()) * wl.FRAME_SECONDS / dt}


def run_stream(args):
    """cfg5: the same 4096 utterances decoded as random batches of 128, as 2D buckets on (encoder length, output
    length) (8 x 4 quantile bins with a 64k frame+token budget per batch; the paper's 30 x 2 bins), and through 128
    continuously refilled slots in random arrival order.  Reports padding fractions, tokens/s and RTFx of every arm in
    one JSON line (value = the 8 x 4 bucketed arm)."""
    import torch
    from paper_2503_05931_b200 import binding, bucketing

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    device = "cuda:0"
    torch.cuda.set_device(0)
    w = wl.make_workload("cfg5")
    peaks = load_peaks()
    rng = np.random.default_rng(5)
    # the paper's configuration: 30 duration bins of equal cumulative duration x 2 token sub-bins, estimated on a
    # separate sample of the same law, flexible allocation (nothing that fits any bucket is dropped)
    _, est_enc, est_dec = wl.draw_lengths(np.random.default_rng(wl.BASE_SEED + 500), 20000, "lognormal")
    dur_bounds, tok_bounds = bucketing.estimate_bins_2d(est_enc, est_dec, 30, 2)
    sizes = bucketing.bucket_batch_sizes(dur_bounds, tok_bounds)
    paper_batches, dropped = bucketing.bucket_batches(w.enc_lens, w.dec_lens, dur_bounds, tok_bounds, sizes, "flexible")
    paper_batches += [dropped[i:i + 128] for i in range(0, len(dropped), 128)]      # every arm decodes all utterances
    arms = {"random128": bucketing.random_batches(w.batch, 128, rng),
            "bucketed8x4": bucketing.bucket_batches_2d(w.enc_lens, w.dec_lens),
            "bucketed30x2": paper_batches}
    all_batches = [b for bs in arms.values() for b in bs]
    slot_counts = (128, 256)
    dec = binding.Decoder(w.model, w.weights, w.dtype, max_batch=max(max(slot_counts), max(len(b) for b in all_batches)),
                          max_total_enc_frames=max(max(slot_counts) * int(w.enc_lens.max()), max(int(w.enc_lens[b].sum()) for b in all_batches)),
                          max_enc_len=int(w.enc_lens.max()), max_dec_len=int(w.dec_lens.max()), bos_id=w.bos_id,
                          eos_id=w.eos_id, ln_eps=w.ln_eps, device=device)
    enc_all = torch.from_numpy(w.enc).to(device).to(dec.tdtype)
    off = w.enc_offsets
    toks = torch.empty((dec.max_batch, dec.max_dec_len), dtype=torch.int32, device=device)
    lens = torch.empty(dec.max_batch, dtype=torch.int32, device=device)
    result = {}
    for name, batches in arms.items():
        packed = [torch.cat([enc_all[off[u]:off[u + 1]] for u in b]) for b in batches]      # resident before timing
        def run_arm():
            for b, enc in zip(batches, packed):
                dec.precompute_cross_kv(enc, w.enc_lens[b])
                dec.greedy_decode(w.dec_lens[b], toks, lens)
        run_arm()                                   # warm-up: captures the step graphs of this arm
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = dec.launch_count()
        e0.record()
        for _ in range(args.steps):
            run_arm()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        pad_enc, pad_dec = bucketing.padding_fractions(w.enc_lens, w.dec_lens, batches)
        roof = 0.0
        for b in batches:
            sub = w.subset_lengths(b)
            d_s, p_s = roofline_seconds(sub, peaks)
            roof += d_s + p_s
        result[name] = {"batches": len(batches), "pad_enc": pad_enc, "pad_dec": pad_dec, "ms": ms,
                        "tokens_per_s": float(w.dec_lens.sum()) / (ms * 1e-3), "rtfx": w.audio_seconds / (ms * 1e-3),
                        "roofline_ms": 1e3 * roof, "roofline_frac": 1e3 * roof / ms,
                        "gpu_launches": int((dec.launch_count() - launches0) / args.steps)}
        del packed
    # continuous batching: no sorting by lengths that a server does not know; a slot is refilled when its utterance ends
    arrival = np.random.default_rng(6).permutation(w.batch)
    host_toks = torch.empty((w.batch, dec.max_dec_len), dtype=torch.int32).pin_memory()
    host_lens = torch.zeros(w.batch, dtype=torch.int32).pin_memory()
    per_step, pre_bytes, pre_flops, step_params = step_bytes_and_flops(w)
    e = 2 if w.dtype == "bf16" else 4
    bw, fl = peaks["hbm_gbs"] * 1e9, peaks["bf16_tflops_sustained"] * 1e12
    kv_bytes = sum(b - e * step_params for b, _, _ in per_step)
    for slots in slot_counts:
        stats = {}
        def run_slots():
            _, _, steps, row_steps = dec.decode_stream(enc_all, w.enc_lens, w.dec_lens, slots, order=arrival, tokens_out=host_toks,
                                                       out_lens=host_lens)
            stats.update({"steps": steps, "row_steps": row_steps})
        run_slots()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = dec.launch_count()
        e0.record()
        for _ in range(args.steps):
            run_slots()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        assert np.array_equal(host_lens.numpy(), w.dec_lens)
        # roofline of this schedule: the step weights once per issued step, every (utterance, position)'s K/V once, and
        # the precompute of every utterance
        roof = (stats["steps"] * e * step_params + kv_bytes) / bw + max(pre_bytes / bw, pre_flops / fl)
        result[f"slots{slots}"] = {"slots": slots, "steps": stats["steps"], "occupancy": stats["row_steps"] / (stats["steps"] * slots),
                                   "ms": ms, "tokens_per_s": float(w.dec_lens.sum()) / (ms * 1e-3), "rtfx": w.audio_seconds / (ms * 1e-3),
                                   "roofline_ms": 1e3 * roof, "roofline_frac": 1e3 * roof / ms,
                                   "gpu_launches": int((dec.launch_count() - launches0) / args.steps)}
    dec.sync_status()
    dec.close()
    best = result["bucketed8x4"]
    line = {"metric": "decoder output tokens/s", "value": best["tokens_per_s"], "unit": "tokens/s", "n_gpus": 1,
            "steps": args.steps, "warmup": 1, "ms_per_step": best["ms"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "cfg5", **w.model, "utterances": w.batch, "step": "one pass over the whole stream",
                       "l2": "inputs larger than L2"},
            "rtfx": best["rtfx"], "arms": result, "gpu_launches": best["gpu_launches"]}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=list(wl.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-profile", action="store_true")
    ap.add_argument("--clip-batch", type=int, default=0,
                    help="keep only this many utterances, those with the longest outputs (profiling captures of the few-row kernels)")
    ap.add_argument("--cross-kv", default="dtype", choices=["dtype", "e4m3"],
                    help="storage of the cross-attention K/V: the workload's dtype (the measured configuration) or 8-bit E4M3")
    ap.add_argument("--clip-len", type=int, default=0,
                    help="shorten every forced output length to at most this many tokens (profiling captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.cross_kv == "e4m3":
        global CROSS_KV_BYTES
        CROSS_KV_BYTES = 1

    if args.impl == "reference":
        run_reference(args)
        return
    if args.workload == "cfg5":
        run_stream(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2503_05931_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(device))

    # Every rank decodes its own batch of the same distribution (utterances are independent: no collective
    # on the data path, weak scaling).
    w = wl.make_workload(args.workload, seed=rank_seed(args.workload, rank))
    if args.clip_batch > 0:
        keep = np.sort(np.argsort(-w.dec_lens, kind="stable")[:args.clip_batch])
        w = w.subset(keep)
    if args.clip_len > 0:
        w.dec_lens = np.minimum(w.dec_lens, args.clip_len).astype(np.int32)
    peaks = load_peaks()
    dec = binding.decoder_for_workload(w, device=device, cross_kv_e4m3=args.cross_kv == "e4m3")
    enc_host = torch.from_numpy(w.enc).to(dec.tdtype).pin_memory()
    enc_dev = enc_host.to(device)
    B, Lmax = w.batch, int(w.dec_lens.max())
    toks_dev = torch.empty((B, Lmax), dtype=torch.int32, device=device)
    lens_dev = torch.empty(B, dtype=torch.int32, device=device)
    toks_host = torch.empty((B, Lmax), dtype=torch.int32).pin_memory()
    lens_host = torch.empty(B, dtype=torch.int32).pin_memory()
    n_tok = int(w.dec_lens.sum())

    def one_pass(from_host: bool):
        src = enc_dev
        if from_host:
            src = enc_host.to(device, non_blocking=True)
        dec.precompute_cross_kv(src, w.enc_lens)
        dec.greedy_decode(w.dec_lens, toks_dev, lens_dev)
        if from_host:
            toks_host.copy_(toks_dev, non_blocking=True)
            lens_host.copy_(lens_dev, non_blocking=True)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(from_host: bool, steps: int):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        barrier()
        ev[0].record()
        for i in range(steps):
            one_pass(from_host)
            ev[i + 1].record()
        barrier()
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        total_ms = ev[0].elapsed_time(ev[steps])
        return total_ms, per

    for _ in range(max(args.warmup, 3)):
        one_pass(False)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = dec.launch_count()
    total_ms, per = timed(False, args.steps)
    launches = dec.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    one_pass(True)
    e2e_ms, _ = timed(True, args.steps)
    dec.sync_status()

    e2e_ms, _, _ = reduce_over_ranks(e2e_ms, 0.0, 0.0, device, world)
    total_ms, total_tokens, total_frames = reduce_over_ranks(total_ms, float(n_tok), float(w.enc_lens.sum()), device, world)
    value = total_tokens * args.steps / (total_ms * 1e-3)
    e2e_value = total_tokens * args.steps / (e2e_ms * 1e-3)
    rtfx = total_frames * wl.FRAME_SECONDS * args.steps / (total_ms * 1e-3)

    if rank == 0:
        dec_s, pre_s = roofline_seconds(w, peaks)
        ms_per_step = total_ms / args.steps
        h2d = int(enc_host.numel() * enc_host.element_size())
        d2h = int(toks_host.numel() * 4 + lens_host.numel() * 4)
        line = {
            "metric": "decoder output tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": w.name, **w.model, "batch_per_gpu": w.batch, "total_enc_frames": int(w.enc_lens.sum()),
                       "total_out_tokens": n_tok, "decode_steps": Lmax, "clip_len": args.clip_len, "clip_batch": args.clip_batch,
                       "cross_kv_store": "e4m3" if args.cross_kv == "e4m3" else w.dtype,
                       "l2": "inputs larger than L2 (weights + K/V stores stream every decode step)",
                       "step": "cross-K/V precompute + greedy decode of one batch"},
            "rtfx": rtfx,
            "step_roofline": {"roofline_ms": 1e3 * (dec_s + pre_s), "frac": 1e3 * (dec_s + pre_s) / ms_per_step,
                              "peaks": peaks["source"], "hbm_gbs": peaks["hbm_gbs"],
                              "bf16_tflops": peaks["bf16_tflops_sustained"]},
            "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if not args.no_profile:
            line["roofline"] = profile_dominant_kernel(dec, w, one_pass, peaks, ms_per_step)
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(w)
        print(json.dumps(line), flush=True)
    dec.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def profile_dominant_kernel(dec, w, one_pass, peaks, ms_per_step):
    """Roofline figure of the kernel that takes the largest share of device time.

    Shares come from one extra pass with CUDA events around every launch on the library's stream (no graph replay in
    that pass), summed per kernel, not per call site.  The kernel's time inside the measured (graphed, overlapped)
    pass is taken as share x measured pass time: launches overlap under programmatic dependent launch, so a per-launch
    duration of the measured configuration only exists in that sense.  ``avg_us_ungraphed`` is the plain event
    figure of the extra pass, which includes the host launch gap."""
    prof = dec.profile_pass(one_pass)
    if not prof:
        return None
    total = sum(v["ms"] for v in prof.values())
    kernels = {}
    m = w.model
    e = 2 if w.dtype == "bf16" else 4
    d, F = m["d_model"], m["d_ffn"]
    # bytes of weights one launch of a projection call site reads (what the layer's definition contains)
    site_weights = {"gemm_qkv": 3 * d * d, "gemm_o": d * d, "gemm_qc": d * d, "gemm_oc": d * d, "gemm_ff1": d * F, "gemm_ff2": d * F}
    for fam, v in prof.items():
        base, _, variant = fam.partition("@")                  # "gemm_qkv@gemv_staged": call site and the kernel that ran it
        kernel = {"gemv": "step_gemv_kernel", "gemv_staged": "step_gemv_staged_kernel"}.get(variant, KERNEL_OF_FAMILY.get(base, base))
        if base == "gemm_vocab" and variant:
            kernel = "vocab_gemv_kernel"                       # final LayerNorm + vocabulary projection of steps with few rows
        k = kernels.setdefault(kernel, {"ms": 0.0, "launches": 0, "bytes": 0.0, "families": []})
        k["ms"] += v["ms"]; k["launches"] += v["launches"]; k["families"].append(fam)
        if base in site_weights:
            per_launch_w = site_weights[base]
            # steps of at most 128 rows: the cross-attention query matrix is read by the launch that reads Wqkv
            if base == "gemm_qkv" and not any(f.partition("@")[0] == "gemm_qc" for f in prof):
                per_launch_w += d * d
            k["bytes"] += e * per_launch_w * v["launches"]
        else:
            k["bytes"] += family_bytes(base, w) or 0.0
    top = max(kernels, key=lambda k: kernels[k]["ms"])
    info = kernels[top]
    share = info["ms"] / total
    in_graph_ms = share * ms_per_step
    per_launch = info["bytes"] / max(info["launches"], 1)
    achieved = info["bytes"] / (in_graph_ms * 1e-3) / 1e9 if info["bytes"] else None
    ratio = NCU_TRAFFIC_RATIO.get(top)
    family_shares = {}
    for fam, v in prof.items():
        base = fam.partition("@")[0]
        family_shares[base] = family_shares.get(base, 0.0) + v["ms"] / total
    return {"bound": "hbm", "kernel": top, "families": sorted(info["families"]), "achieved": achieved,
            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": (achieved / peaks["hbm_gbs"]) if achieved else None,
            "traffic": ratio * per_launch if (ratio and per_launch) else None,
            "traffic_unit": "bytes per launch (ncu capture of one layer's launches, scaled by algorithmic bytes)",
            "algorithmic_bytes_per_launch": per_launch or None,
            "launches": info["launches"], "share_of_device_time": round(share, 4),
            "avg_us": 1e3 * in_graph_ms / max(info["launches"], 1),
            "avg_us_ungraphed": 1e3 * info["ms"] / max(info["launches"], 1),
            "peak_source": peaks["source"],
            "shares": {k: round(v["ms"] / total, 4) for k, v in sorted(kernels.items(), key=lambda kv: -kv[1]["ms"])},
            "family_shares": {k: round(v, 4) for k, v in family_shares.items()}}


if __name__ == "__main__":
    main()
