#!/usr/bin/env python
"""Benchmark of the block-sparse fused attention path.

A step is one call of the whole hot path (work list -> persistent kernel: TMA loads, QK^T,
online softmax, PV, epilogue) over one synthetic batch.  The default workload is the 32K
block-sparse configuration the headline target is stated on (16 heads, S = 32768, d = 128,
causal per-head block bitmap with keep probability 0.25).  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank runs its own replica of the workload
(independent problems, different seeds, no data-path collective): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_09385_b200 import inputs  # noqa: E402

METRIC = "effective attention TFLOP/s (kept tiles)"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_BF16_TFLOPS = 2250.0  # vendor figure for dense bf16 on one B200 (context, not a measurement)
# dram__bytes_read.sum + dram__bytes_write.sum of one kernel launch on the default workload,
# from the ncu capture summarised in profiles/ (None until a capture exists for a workload).
NCU_TRAFFIC_BYTES = {"c2_causal_s4k_mha32": 100930304 + 11335936,          # one-pass captures of one full launch each
                     "c3_window4k_s16k_gqa32x8": 213756928 + 99447296,
                     "c4_bitmap25_s32k_h16": 413043200 + 119604736,
                     "c5_causal_s128k_gqa32x8": 3695049472 + 1193544192}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["source"] = "fallback"
    return d


class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons through NVML (read-only queries)
    every few milliseconds while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.005):
        self.index, self.period = index, period_s
        self.sm, self.mask, self.max_mhz, self.error = [], 0, None, None
        self._stop = threading.Event()
        self._thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.index
            if visible:
                ids = [x for x in visible.split(",") if x]
                if idx < len(ids) and ids[idx].isdigit():
                    idx = int(ids[idx])
            h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while not self._stop.is_set():
                self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                self.mask |= int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h))
                self._stop.wait(self.period)
        except Exception as exc:  # report, never fail the benchmark on a monitoring problem
            self.error = repr(exc)

    def __enter__(self):
        self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        self._thread.join(timeout=10)

    def summary(self) -> dict:
        out = {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_mhz,
               "sm_min_mhz": min(self.sm) if self.sm else None,
               "reasons": [n for bit, n in self.REASONS.items() if self.mask & bit], "samples": len(self.sm)}
        if self.error:
            out["error"] = self.error
        return out


def oracle_sample_rows(w, n_rows: int, seed: int = 7) -> np.ndarray:
    """Seeded random (b, h, i) rows, uniform over the workload's query rows."""
    rng = np.random.default_rng(seed)
    return np.stack([np.zeros(n_rows, np.int64), rng.integers(0, w.heads_q, n_rows),
                     rng.integers(0, w.seq, n_rows)], axis=1)


def time_oracle(w, data, n_rows: int, effective_flop: float):
    """Time the CPU oracle on `n_rows` sampled rows; returns (equivalent TFLOP/s, seconds, threads)."""
    import oracle
    p = oracle.OracleProblem(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                             w.block, w.block, w.window, data["bitmap"])
    rows = oracle_sample_rows(w, n_rows)
    oracle.rows(p, data["q"], data["k"], data["v"], rows[:8])  # touch the library and the inputs
    t0 = time.perf_counter()
    oracle.rows(p, data["q"], data["k"], data["v"], rows)
    dt = time.perf_counter() - t0
    share = n_rows / float(w.batch * w.heads_q * w.seq)
    return effective_flop * share / dt / 1e12, dt, oracle.max_threads()


def calibrate_rows(w, data, effective_flop: float, target_seconds: float, cap: int = 1 << 17) -> int:
    """Number of sampled rows that makes one oracle pass last about `target_seconds` on this host."""
    probe = 128
    _, dt, _ = time_oracle(w, data, probe, effective_flop)
    rows = int(probe * target_seconds / max(dt, 1e-4))
    return max(probe, min(rows, cap, w.batch * w.heads_q * w.seq))


def tile_counts_from_definition(w, bitmap):
    """(kept, partial) mask blocks of a workload from the mask's definition alone -- closed forms for
    causal / window / dense masks on block-aligned lengths, the bitmap's population count for the
    block-bitmap workload, the oracle's brute-force count otherwise.  Uses nothing of the CUDA library."""
    T = w.seq // w.block
    aligned = w.seq % w.block == 0
    causal, window, bmp = (bool(w.flags & f) for f in (inputs.MASK_CAUSAL, inputs.MASK_WINDOW, inputs.MASK_BITMAP))
    heads = w.batch * w.heads_q
    if aligned and bmp and causal and not window:
        # bits above the diagonal are clear in these bitmaps; the diagonal blocks carry the token-level triangle
        idx = np.arange(T)
        upper = sum(int((int(bitmap[h, i, j >> 5]) >> (j & 31)) & 1) for h in range(min(2, w.heads_q))
                    for i in idx[:8] for j in range(i + 1, min(T, i + 40)))
        if upper == 0:
            kept = int(sum(bin(int(x)).count("1") for x in np.asarray(bitmap).ravel())) * w.batch
            diag = sum(inputs.bitmap_bit(bitmap, h, i, i) for h in range(w.heads_q) for i in range(T)) * w.batch
            return kept, int(diag)
    if aligned and not bmp and causal and not window:
        return heads * T * (T + 1) // 2, heads * T
    if aligned and not bmp and causal and window and w.window % w.block == 0:
        wb = w.window // w.block
        return heads * sum(min(i, wb) + 1 for i in range(T)), heads * (T + max(0, T - wb))
    if aligned and not bmp and not causal and not window:
        return heads * T * T, 0
    import oracle
    p = oracle.OracleProblem(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                             w.block, w.block, w.window, bitmap)
    c = oracle.count_tiles(p)
    return int(c[:, 0].sum()) * w.batch, int(c[:, 1].sum()) * w.batch


def make_config(w, kept, partial, world):
    """The `config` object of the JSON line: the same keys and values in both arms."""
    tensors_mib = (2 * w.batch * w.heads_q + 2 * w.batch * w.heads_kv) * w.seq * w.head_dim * 2 >> 20
    return {"workload": w.name, "batch": w.batch, "heads_q": w.heads_q, "heads_kv": w.heads_kv, "seq": w.seq,
            "head_dim": w.head_dim, "mask_block": w.block, "kept_tiles": int(kept), "partial_tiles": int(partial),
            "effective_flop": 4.0 * w.block * w.block * w.head_dim * kept,
            "l2": "inputs larger than L2 (Q+K+V+O = %d MiB)" % tensors_mib if tensors_mib > 126 else
                  "Q+K+V+O = %d MiB; an L2-cold leg (flush between calls) is reported beside the warm one" % tensors_mib,
            "parallelism": f"replicas x{world}"}


def run_reference(args, w, rank, world):
    """--impl reference: the CPU oracle as it stands, on a bounded sample per step.  Imports nothing
    of the CUDA library: the kept-tile count comes from the mask's definition."""
    if rank != 0:
        return
    data = inputs.make_inputs(w, inputs.DEFAULT_SEED)
    kept, partial = tile_counts_from_definition(w, data["bitmap"])
    config = make_config(w, kept, partial, world)
    flop = config["effective_flop"]
    # a bounded sample per step: the whole run (warm-up + steps) aims at about a minute of oracle time
    n_rows = args.oracle_rows or calibrate_rows(w, data, flop, 60.0 / max(1, args.steps + args.warmup / 8.0))
    for _ in range(args.warmup):
        time_oracle(w, data, max(8, n_rows // 8), flop)
    vals, secs = [], []
    threads = 1
    for _ in range(args.steps):
        v, dt, threads = time_oracle(w, data, n_rows, flop)
        vals.append(v)
        secs.append(dt)
    value = float(np.mean(vals))
    sample = (f"{n_rows} seeded random query rows of {w.name} per step (dense fp64 rows over all {w.seq} keys), "
              f"credited with their share of the effective FLOP")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(secs)) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config, "timing": "host wall clock, CPU only",
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def time_calls(torch, fn, steps, warmup, flush=None):
    """Mean / median / min milliseconds per call of `fn` by CUDA events on the current stream; with
    `flush`, an L2-sized buffer is overwritten before every call, outside the timed events."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    for i in range(steps):
        if flush is not None:
            flush.add_(1)
        starts[i].record()
        fn()
        ends[i].record()
    torch.cuda.synchronize()
    ms = np.array([a.elapsed_time(b) for a, b in zip(starts, ends)])
    return {"mean": float(ms.mean()), "median": float(np.median(ms)), "min": float(ms.min())}


def l2_flush_buffer(torch, dev):
    """A buffer twice the size of L2 (size read from the device attributes)."""
    l2 = torch.cuda.get_device_properties(dev).L2_cache_size
    return torch.zeros(2 * l2 // 4, dtype=torch.int32, device=dev)


def run_emulation_sweep(args, dev):
    """Software exponent (a cubic on the FMA pipe for 0 / 12.5 / 25 / 50 % of the exponentials) at
    head_dim 128 and 64: ms per call and the LSE difference against the build without emulation."""
    import torch
    from paper_2607_09385_b200 import binding
    rows = []
    for name in ("c2", "c4", "llama1b_h32_d64_s8192"):
        w = inputs.workload(name)
        data = inputs.make_inputs(w, inputs.DEFAULT_SEED)
        q, k, v = (torch.from_numpy(data[x].view(np.int16)).to(dev).view(torch.bfloat16) for x in "qkv")
        o = torch.empty_like(q)
        lse = torch.empty((w.batch, w.heads_q, w.seq), dtype=torch.float32, device=dev)
        lse0 = None
        for emu in range(4):
            attn = binding.SteelAttention(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                                          w.block, w.window, data["bitmap"], exp_emulation=emu)
            t = time_calls(torch, lambda: attn.run(q, k, v, o, lse), args.steps, max(3, args.warmup))
            if attn.last_status() != binding.STEEL_OK:
                raise SystemExit("device status is not OK")
            if emu == 0:
                lse0 = lse.clone()
            rows.append({"workload": w.name, "head_dim": w.head_dim, "exp_emulation": emu,
                         "share": (0.0, 0.125, 0.25, 0.5)[emu], "ms_per_call": t["mean"], "ms_min": t["min"],
                         "tflops": attn.stats()["effective_flop"] / (t["mean"] * 1e-3) / 1e12,
                         "max_abs_lse_diff_vs_no_emulation": float((lse - lse0).abs().max())})
            attn.close()
    print(json.dumps({"sweep": "emulation", "steps": args.steps, "results": rows}), flush=True)


def run_keep_sweep(args, dev):
    """Runtime against kept-tile count: the headline shape (16 heads, S = 32768, d = 128, causal block
    bitmap) at keep probabilities 0.05 ... 1.0; least-squares fit ms = a + b * tiles."""
    import dataclasses
    import torch
    from paper_2607_09385_b200 import binding
    base = inputs.workload("c4")
    if args.profile_heads:
        base = dataclasses.replace(base, heads_q=args.profile_heads, heads_kv=args.profile_heads)
    data = inputs.make_inputs(base, inputs.DEFAULT_SEED)
    q, k, v = (torch.from_numpy(data[x].view(np.int16)).to(dev).view(torch.bfloat16) for x in "qkv")
    o = torch.empty_like(q)
    lse = torch.empty((base.batch, base.heads_q, base.seq), dtype=torch.float32, device=dev)
    rows = []
    for keep in (0.05, 0.125, 0.25, 0.5, 1.0):
        bitmap = inputs.block_bitmap(base.heads_q, base.tiles, base.tiles, keep, inputs.DEFAULT_SEED)
        attn = binding.SteelAttention(base.batch, base.heads_q, base.heads_kv, base.seq, base.seq, base.head_dim,
                                      base.scale, base.flags, base.block, base.window, bitmap)
        st = attn.stats()
        t = time_calls(torch, lambda: attn.run(q, k, v, o, lse), args.steps, max(3, args.warmup))
        if attn.last_status() != binding.STEEL_OK:
            raise SystemExit("device status is not OK")
        rows.append({"keep_prob": keep, "kept_tiles": st["kept_tiles"], "ms_per_call": t["mean"], "ms_min": t["min"],
                     "tflops": st["effective_flop"] / (t["mean"] * 1e-3) / 1e12})
        attn.close()
    x = np.array([r["kept_tiles"] for r in rows], dtype=np.float64)
    y = np.array([r["ms_per_call"] for r in rows], dtype=np.float64)
    b, a = np.polyfit(x, y, 1)
    r2 = 1.0 - float(((y - (a + b * x)) ** 2).sum() / ((y - y.mean()) ** 2).sum())
    print(json.dumps({"sweep": "keep", "shape": f"{base.heads_q} heads, S = {base.seq}, d = {base.head_dim}",
                      "steps": args.steps, "fit": {"intercept_ms": float(a), "ns_per_tile": float(b) * 1e6, "r2": r2},
                      "results": rows}), flush=True)


def run_paper_sweep(args, dev):
    """Throughput against sequence length on the paper's own shapes (BERT and Llama-3.1-1B attention,
    head_dim 64): one JSON line with one entry per shape."""
    import torch
    from paper_2607_09385_b200 import binding
    rows = []
    for w in inputs.paper_workloads():
        data = inputs.make_inputs(w, inputs.DEFAULT_SEED)
        attn = binding.SteelAttention(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                                      w.block, w.window, None)
        q, k, v = (torch.from_numpy(data[x].view(np.int16)).to(dev).view(torch.bfloat16) for x in "qkv")
        o = torch.empty_like(q)
        lse = torch.empty((w.batch, w.heads_q, w.seq), dtype=torch.float32, device=dev)
        for _ in range(max(3, args.warmup)):
            attn.run(q, k, v, o, lse)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            attn.run(q, k, v, o, lse)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        flop = attn.stats()["effective_flop"]
        rows.append({"workload": w.name, "seq": w.seq, "heads": w.heads_q, "head_dim": w.head_dim,
                     "causal": bool(w.flags & inputs.MASK_CAUSAL), "ms_per_call": ms,
                     "tflops": flop / (ms * 1e-3) / 1e12})
        attn.close()
    print(json.dumps({"sweep": "paper", "metric": METRIC, "unit": UNIT, "steps": args.steps, "results": rows}),
          flush=True)


def run_unfused_sweep(args, dev):
    """Fused kernel against layer-by-layer attention (library GEMM -> scale/mask -> softmax -> library
    GEMM, every intermediate through HBM) on the paper's shapes, with the modelled HBM traffic of
    both.  The layer-by-layer arm is a comparison baseline, not part of the library."""
    import torch
    from paper_2607_09385_b200 import binding, layer_by_layer, traffic_model

    unfused = layer_by_layer.layer_by_layer_attention

    rows = []
    for w in inputs.paper_workloads():
        if w.heads_q * w.seq * w.seq * 2 > (8 << 30):      # the score matrix must fit comfortably
            continue
        data = inputs.make_inputs(w, inputs.DEFAULT_SEED)
        attn = binding.SteelAttention(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                                      w.block, w.window, None)
        q, k, v = (torch.from_numpy(data[x].view(np.int16)).to(dev).view(torch.bfloat16) for x in "qkv")
        o = torch.empty_like(q)
        causal = bool(w.flags & inputs.MASK_CAUSAL)

        def timed(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / args.steps

        ms_fused = timed(lambda: attn.run(q, k, v, o, None, want_lse=False))
        ms_unfused = timed(lambda: unfused(q, k, v, w.scale, causal))
        ref = unfused(q, k, v, w.scale, causal)
        err = float((ref.float() - o.float()).abs().max())
        st = attn.stats()
        fused_model = traffic_model.fused_bytes(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim,
                                                st["kv_tile_loads"])
        unfused_model = traffic_model.unfused_bytes(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim)
        rows.append({"workload": w.name, "seq": w.seq, "ms_fused": ms_fused, "ms_layer_by_layer": ms_unfused,
                     "speedup": ms_unfused / ms_fused, "max_abs_diff": err,
                     "model_bytes_fused_compulsory": fused_model["compulsory"],
                     "model_bytes_fused_no_reuse": fused_model["no_reuse"],
                     "model_bytes_layer_by_layer": unfused_model["total"]})
        attn.close()
        del q, k, v, o, ref
        torch.cuda.empty_cache()
    print(json.dumps({"sweep": "unfused", "steps": args.steps, "results": rows}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=25)
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--impl", default="steel", choices=["steel", "reference"])
    ap.add_argument("--oracle-rows", type=int, default=0,
                    help="rows the CPU oracle is timed on (0: calibrated to about 12 s of wall time)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cold", action="store_true", help="skip the L2-cold timing leg")
    ap.add_argument("--e2e-chunks", type=int, default=8, help="chunks of the host-memory call")
    ap.add_argument("--policy", type=int, default=0)
    ap.add_argument("--exp-emulation", type=int, default=0, help="0..3: share of exponentials on the FMA pipe")
    ap.add_argument("--sweep", default="", choices=["", "paper", "unfused", "keep", "emulation"],
                    help="'paper': time the paper's own attention shapes (head_dim 64) instead of one workload; "
                         "'unfused': the same shapes against layer-by-layer attention through HBM; "
                         "'keep': the headline shape at keep probabilities 0.05 ... 1.0 with a linear fit of "
                         "ms against kept tiles; 'emulation': software-exponent shares 0 ... 50 %")
    ap.add_argument("--profile-heads", type=int, default=0,
                    help="shrink the workload to this many query heads (same KV grouping) for ncu captures")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "steel" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    w = inputs.workload(int(args.workload) if args.workload.isdigit() else args.workload)
    if args.profile_heads:
        import dataclasses
        group = w.heads_q // w.heads_kv
        w = dataclasses.replace(w, name=f"{w.name}_h{args.profile_heads}", heads_q=args.profile_heads,
                                heads_kv=max(1, args.profile_heads // group))

    if args.impl == "reference":
        run_reference(args, w, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2607_09385_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    if args.sweep == "paper":
        run_paper_sweep(args, dev)
        return
    if args.sweep == "unfused":
        run_unfused_sweep(args, dev)
        return
    if args.sweep == "keep":
        run_keep_sweep(args, dev)
        return
    if args.sweep == "emulation":
        run_emulation_sweep(args, dev)
        return

    # every rank works on its own replica (independent problem, own seed)
    data = inputs.make_inputs(w, inputs.DEFAULT_SEED + rank)
    attn = binding.SteelAttention(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                                  w.block, w.window, data["bitmap"], policy=args.policy,
                                  exp_emulation=args.exp_emulation)
    stats = attn.stats()
    host = {x: torch.from_numpy(data[x].view(np.int16)).pin_memory() for x in "qkv"}
    q, k, v = (host[x].to(dev, non_blocking=True).view(torch.bfloat16) for x in "qkv")
    o = torch.empty_like(q)
    lse = torch.empty((w.batch, w.heads_q, w.seq), dtype=torch.float32, device=dev)
    # CTA 0 reports the SM cycles and nanoseconds of each launch: the clock the kernel really ran at
    probe = torch.zeros(2, dtype=torch.int64, device=dev)
    binding.steel_attn_debug_clock_probe(attn.handle, probe.data_ptr())
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        attn.run(q, k, v, o, lse)
    barrier()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    probes = torch.zeros((args.steps, 2), dtype=torch.int64, device=dev)
    with ClockSampler(local_rank) as clocks:
        t_begin = torch.cuda.Event(enable_timing=True)
        t_end = torch.cuda.Event(enable_timing=True)
        t_begin.record()
        for i in range(args.steps):
            starts[i].record()
            attn.run(q, k, v, o, lse)
            ends[i].record()
        t_end.record()
        barrier()
    status = attn.last_status()
    if status != binding.STEEL_OK:
        raise SystemExit(f"device status: {binding.steel_status_string(status)}")
    total_ms = t_begin.elapsed_time(t_end)
    kernel_ms = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    # in-kernel clock over a second, untimed pass of the same length (the copy of the probe between
    # launches would otherwise sit inside the timed region)
    for i in range(args.steps):
        attn.run(q, k, v, o, lse)
        probes[i].copy_(probe)
    torch.cuda.synchronize()
    pr = probes.cpu().numpy().astype(np.float64)
    sm_mhz_kernel = float(np.median(pr[:, 0] / np.maximum(pr[:, 1], 1.0)) * 1e3)

    # L2-cold leg: a buffer twice the size of L2 is overwritten before every call, outside the events
    cold = None
    if rank == 0 and not args.no_cold:
        flush = l2_flush_buffer(torch, dev)
        cold = time_calls(torch, lambda: attn.run(q, k, v, o, lse), max(3, min(args.steps, 20)), 2, flush)
        del flush

    # end to end through the C ABI with host buffers (steel_attn_host_run): H2D of Q, K, V and D2H of
    # O, LSE are inside the call, chunked so that copies overlap kernels
    e2e = None
    if not args.no_e2e:
        o_host = torch.empty(q.shape, dtype=torch.int16).pin_memory()
        lse_host = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
        e2e_steps = max(3, min(args.steps, 10))
        attn_host = binding.SteelAttentionHost(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale,
                                               w.flags, w.block, w.window, data["bitmap"],
                                               max_chunks=args.e2e_chunks, policy=args.policy,
                                               exp_emulation=args.exp_emulation)

        def e2e_step():
            attn_host.run(host["q"], host["k"], host["v"], o_host, lse_host)

        for _ in range(2):
            e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        e2e_ms = e0.elapsed_time(e1) / e2e_steps
        if attn_host.last_status() != binding.STEEL_OK:
            raise SystemExit("device status of the host-memory call is not OK")
        e2e_chunks = attn_host.chunks
        attn_host.close()
        h2d = sum(host[x].numel() * 2 for x in "qkv")
        d2h = o_host.numel() * 2 + lse_host.numel() * 4
    times = torch.tensor([total_ms, e2e_ms if not args.no_e2e else 0.0], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
    total_ms, e2e_ms = float(times[0]), float(times[1])
    ms_per_step = total_ms / args.steps
    flop = stats["effective_flop"]
    value = world * flop / (ms_per_step * 1e-3) / 1e12
    if not args.no_e2e:
        e2e = {"value": world * flop / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "chunks": e2e_chunks,
               "call": "steel_attn_host_run (pinned host buffers)"}

    if rank == 0:
        peaks = load_peaks()
        launch_ms = float(np.mean(kernel_ms))
        achieved = flop / (launch_ms * 1e-3) / 1e12
        sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
        # tensor pipe at the clock the kernel ran at: SMs x 8192 dense bf16 FLOP per clock x measured MHz
        peak_at_clock = sm_count * 8192 * sm_mhz_kernel * 1e6 / 1e12
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": UNIT,
                    "frac": achieved / peaks["bf16_tflops"], "traffic": NCU_TRAFFIC_BYTES.get(w.name),
                    "peak_source": f"{peaks['source']} bf16 burst (kernel timed alone)",
                    "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                    "peak_nominal": NOMINAL_BF16_TFLOPS, "frac_of_nominal": achieved / NOMINAL_BF16_TFLOPS,
                    "sm_mhz_in_kernel": sm_mhz_kernel, "peak_at_clock": peak_at_clock,
                    "frac_at_clock": achieved / peak_at_clock,
                    "denominators": "peak = measured cuBLAS bf16 burst; sustained = the same GEMM for seconds under "
                                    "the power cap; nominal = vendor dense bf16 figure; at_clock = SMs x 8192 "
                                    "FLOP/clk x the SM clock CTA 0 measured inside the kernel (cycles / ns)",
                    "launch_ms": {"mean": launch_ms, "median": float(np.median(kernel_ms)),
                                  "min": float(np.min(kernel_ms))},
                    "l2_cold": None if cold is None else
                    {"launch_ms": cold, "achieved": flop / (cold["mean"] * 1e-3) / 1e12,
                     "how": "a buffer of twice the L2 size is overwritten before every call, outside the events"},
                    "hbm_min_bytes": 2 * (q.numel() * 2) + 2 * (k.numel() * 2) + lse.numel() * 4,
                    "hbm_gbs_at_min_bytes": (2 * (q.numel() * 2) + 2 * (k.numel() * 2) + lse.numel() * 4)
                    / (launch_ms * 1e-3) / 1e9, "hbm_peak_gbs": peaks["hbm_gbs"]}
        cpu = None
        if not args.no_cpu_baseline:
            n_rows = args.oracle_rows or calibrate_rows(w, data, flop, 12.0)
            val, dt, threads = time_oracle(w, data, n_rows, flop)
            cpu = {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt,
                   "sample": f"{n_rows} seeded random query rows of {w.name} (dense fp64 rows over all {w.seq} "
                             f"keys), credited with their share of the effective FLOP"}
        config = make_config(w, stats["kept_tiles"], stats["partial_tiles"], world)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config,
            "timing": "CUDA events on the launching stream, max over ranks",
            "useful_flop": stats["useful_flop"], "policy": args.policy, "exp_emulation": args.exp_emulation,
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": args.steps,
            "clocks": clocks.summary(),
        }
        print(json.dumps(line), flush=True)
    attn.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
