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
# dram__bytes_read.sum + dram__bytes_write.sum of one kernel launch on the default workload,
# from the ncu capture summarised in profiles/ (None until a capture exists for a workload).
NCU_TRAFFIC_BYTES = {"c2_causal_s4k_mha32": 143.90e6 + 12.46e6,                 # one-pass captures of a full launch
                     "c3_window4k_s16k_gqa32x8": 213.86e6 + 98.80e6,
                     "c4_bitmap25_s32k_h16": 4 * (141.451008e6 + 16.546048e6),  # 4 x the 4-head capture
                     "c5_causal_s128k_gqa32x8": 3.38e9 + 1.08e9}              # one-pass capture of a full launch


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


def plan_stats(w, bitmap):
    from paper_2607_09385_b200 import binding
    params, _keep = binding.make_params(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale,
                                        w.flags, w.block, w.block, w.window, bitmap)
    st, stats, _ = binding.steel_attn_plan_host(params)
    assert st == 0
    return stats


def run_reference(args, w, rank, world):
    """--impl reference: the CPU oracle as it stands, on a bounded sample per step."""
    if rank != 0:
        return
    data = inputs.make_inputs(w, inputs.DEFAULT_SEED)
    stats = plan_stats(w, data["bitmap"])
    # a bounded sample per step: the whole run (warm-up + steps) aims at about a minute of oracle time
    n_rows = args.oracle_rows or calibrate_rows(w, data, stats["effective_flop"],
                                                60.0 / max(1, args.steps + args.warmup / 8.0))
    for _ in range(args.warmup):
        time_oracle(w, data, max(8, n_rows // 8), stats["effective_flop"])
    vals, secs = [], []
    threads = 1
    for _ in range(args.steps):
        v, dt, threads = time_oracle(w, data, n_rows, stats["effective_flop"])
        vals.append(v)
        secs.append(dt)
    value = float(np.mean(vals))
    sample = f"{n_rows} seeded random query rows of {w.name} per step (dense fp64 rows over all {w.seq} keys)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(secs)) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "timing": "host wall clock, CPU only"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


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
    from paper_2607_09385_b200 import binding, traffic_model

    def unfused(q, k, v, scale, causal):
        a = torch.matmul(q, k.transpose(-1, -2))
        a = a * scale
        if causal:
            s = q.shape[-2]
            a = a.masked_fill(torch.ones(s, s, dtype=torch.bool, device=q.device).triu(1), float("-inf"))
        p = torch.softmax(a, dim=-1, dtype=torch.float32).to(torch.bfloat16)
        return torch.matmul(p, v)

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
    ap.add_argument("--e2e-chunks", type=int, default=8, help="chunks of the host-memory call")
    ap.add_argument("--policy", type=int, default=0)
    ap.add_argument("--sweep", default="", choices=["", "paper", "unfused"],
                    help="'paper': time the paper's own attention shapes (head_dim 64) instead of one workload; "
                         "'unfused': the same shapes against layer-by-layer attention through HBM")
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

    # every rank works on its own replica (independent problem, own seed)
    data = inputs.make_inputs(w, inputs.DEFAULT_SEED + rank)
    binding.steel_attn_set_policy(args.policy)
    attn = binding.SteelAttention(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale, w.flags,
                                  w.block, w.window, data["bitmap"])
    stats = attn.stats()
    host = {x: torch.from_numpy(data[x].view(np.int16)).pin_memory() for x in "qkv"}
    q, k, v = (host[x].to(dev, non_blocking=True).view(torch.bfloat16) for x in "qkv")
    o = torch.empty_like(q)
    lse = torch.empty((w.batch, w.heads_q, w.seq), dtype=torch.float32, device=dev)
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

    # end to end through the C ABI with host buffers (steel_attn_host_run): H2D of Q, K, V and D2H of
    # O, LSE are inside the call, chunked so that copies overlap kernels
    e2e = None
    if not args.no_e2e:
        o_host = torch.empty(q.shape, dtype=torch.int16).pin_memory()
        lse_host = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
        e2e_steps = max(3, min(args.steps, 10))
        attn_host = binding.SteelAttentionHost(w.batch, w.heads_q, w.heads_kv, w.seq, w.seq, w.head_dim, w.scale,
                                               w.flags, w.block, w.window, data["bitmap"],
                                               max_chunks=args.e2e_chunks)

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
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": UNIT,
                    "frac": achieved / peaks["bf16_tflops"], "traffic": NCU_TRAFFIC_BYTES.get(w.name),
                    "peak_source": f"{peaks['source']} bf16 burst (kernel timed alone)",
                    "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                    "launch_ms": {"mean": launch_ms, "median": float(np.median(kernel_ms)),
                                  "min": float(np.min(kernel_ms))},
                    "hbm_min_bytes": 2 * (q.numel() * 2) + 2 * (k.numel() * 2) + lse.numel() * 4}
        cpu = None
        if not args.no_cpu_baseline:
            n_rows = args.oracle_rows or calibrate_rows(w, data, flop, 12.0)
            val, dt, threads = time_oracle(w, data, n_rows, flop)
            cpu = {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt,
                   "sample": f"{n_rows} seeded random query rows of {w.name} "
                             f"(dense fp64 rows over all {w.seq} keys), scaled by rows/total rows"}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "batch": w.batch, "heads_q": w.heads_q, "heads_kv": w.heads_kv,
                       "seq": w.seq, "head_dim": w.head_dim, "mask_block": w.block,
                       "kept_tiles": stats["kept_tiles"], "partial_tiles": stats["partial_tiles"],
                       "effective_flop": flop, "useful_flop": stats["useful_flop"], "policy": args.policy,
                       "l2": "inputs larger than L2 (Q+K+V+O = %d MiB)" % ((2 * q.numel() + 2 * k.numel()) * 2 >> 20),
                       "parallelism": f"replicas x{world}"},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": args.steps,
            "clocks": clocks.summary(),
        }
        print(json.dumps(line), flush=True)
    attn.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
