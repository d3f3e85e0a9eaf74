#!/usr/bin/env python
"""Benchmark of the elastic-KV attention hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ekv|reference]

One "step" = one pass of the hot path over one batch of the Llama-3-8B-shaped decode workload
(benchmark configs[1]): ekv_write_kv of the 256 new K/V rows through the slot mapping, then
ekv_attn_decode (split pass + combine pass) of 256 sequences with context lengths U[1024, 8192]
whose blocks are randomly permuted over the pool.  value = algorithmic bytes of the step / time.
Multi-GPU runs are independent replicas (one pool per rank, no collective on the data path): under
torchrun the ranks come from the environment; started plainly with --gpus N > 1 this script starts the
N ranks itself.

The JSON line also carries: roofline (decode kernels, timed live with CUDA events), e2e (same
step through host buffers), cpu_baseline (the CPU oracle on this machine's host cores), and two side
measurements of the other hot-path rows: prefill-chunk TFLOP/s and grow/shrink ms.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import ekv_inputs as I  # noqa: E402

METRIC = "decode-attn HBM GB/s (% peak); prefill-chunk TFLOP/s (% peak); grow/shrink ms"
UNIT = "GB/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM bytes (read + write) per algorithmic byte of the decode split kernel: dram__bytes_read.sum +
# dram__bytes_write.sum of one ncu capture of a 32-sequence slice of this workload (623.65 MB read, 4.77 MB
# written, 622.92 MB algorithmic).  The traffic is proportional to the KV bytes read, so the full launch is
# that ratio times its algorithmic bytes.  The capture has to be retaken whenever decode_split_kernel changes.
DECODE_SPLIT_DRAM_TRAFFIC_RATIO = (623.649792 + 4.772352) / 622.920860


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------- clocks


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons of one GPU in the background; every sample is
    stamped with the host clock so that the ones taken DURING a region can be picked out."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        # nvidia-smi numbers the GPUs of the machine, CUDA the visible ones: address the device by its UUID
        try:
            self.index = "GPU-" + str(torch.cuda.get_device_properties(index).uuid)
        except Exception:
            self.index = str(index)
        self.rows, self.proc = [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [c.strip() for c in line.split(",")]))

    def wait_for_samples(self, n=1, timeout=3.0):
        t0 = time.perf_counter()
        while len(self.rows) < n and time.perf_counter() - t0 < timeout and self.proc:
            time.sleep(0.01)

    def __exit__(self, *exc):
        if self.proc:
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self, t0, t1):
        """Median SM clock and throttle reasons over the samples stamped inside [t0, t1]."""
        sm, mx, reasons = [], [], set()
        for (t, r) in self.rows:
            if not (t0 <= t <= t1):
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(self.NAMES, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- workload


class DecodeWorkload:
    """configs[1] resident on one GPU: pool filled by the seeded generator, tables, lengths, inputs."""

    def __init__(self, cfg: I.Config, device: torch.device, batch: int | None = None):
        import paper_2608_23658_b200 as ekv
        self.ekv, self.cfg, self.shape, self.dev = ekv, cfg, cfg.shape, device
        s = cfg.shape
        self.lengths = I.decode_lengths(cfg, batch)
        self.B = len(self.lengths)
        need = int(I.blocks_for(self.lengths, s.block_size).sum())
        pool_blocks = int(need * 1.1) + 64
        self.pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim,
                             base_blocks=pool_blocks, device=device.index or 0)
        live = self.pool.info.live_blocks
        self.tables, _ = I.assign_blocks(cfg.seed, 12, self.lengths, s.block_size, live)
        I.fill_pool_layer_(self.pool.layer_tensor(0), cfg.seed)
        n_q = self.B * s.num_q_heads * s.head_dim
        n_kv = self.B * s.num_kv_heads * s.head_dim
        # host-side (pinned) inputs of one step
        self.h_q = I.normal_bf16(cfg.seed, 3, 0, n_q).view(self.B, s.num_q_heads, s.head_dim).pin_memory()
        self.h_k = I.normal_bf16(cfg.seed, 4, 0, n_kv).view(self.B, s.num_kv_heads, s.head_dim).pin_memory()
        self.h_v = I.normal_bf16(cfg.seed, 5, 0, n_kv).view(self.B, s.num_kv_heads, s.head_dim).pin_memory()
        self.h_slots = I.last_token_slots(self.lengths, self.tables, s.block_size).pin_memory()
        self.h_tables = self.tables.pin_memory()
        self.h_lens = self.lengths.to(torch.int32).pin_memory()
        self.h_out = torch.empty(self.B, s.num_q_heads, s.head_dim, dtype=torch.bfloat16).pin_memory()
        # device-resident copies
        self.q, self.k, self.v = self.h_q.to(device), self.h_k.to(device), self.h_v.to(device)
        self.slots, self.d_tables, self.d_lens = self.h_slots.to(device), self.h_tables.to(device), self.h_lens.to(device)
        self.out = torch.empty_like(self.q)
        self.ws = self.pool.workspace(self.B, int(self.tables.shape[1]) * s.block_size)
        self.scale = 1.0 / math.sqrt(s.head_dim)
        self.decode_bytes = I.decode_algorithmic_bytes(self.lengths, s)
        self.write_bytes = I.write_algorithmic_bytes(self.B, s)
        torch.cuda.synchronize(device)

    def step_resident(self, ev=None):
        p = self.pool
        if ev:
            ev[0].record()
        p.write_kv(0, self.k, self.v, self.slots)
        if ev:
            ev[1].record()
        p.attn_decode(0, self.q, self.d_tables, self.d_lens, self.scale, out=self.out, workspace=self.ws)
        if ev:
            ev[2].record()

    def setup_e2e(self):
        """The end-to-end pipeline: ekv_hoststep_* with two staging sets (copies on the library's own streams)."""
        self.hs = self.ekv.HostStep(self.pool, self.B, int(self.tables.shape[1]), depth=2)
        self.h_outs = [torch.empty_like(self.h_out).pin_memory() for _ in range(2)]
        self.e2e_i = 0

    def step_e2e(self):
        """Same step through HOST buffers, one C-ABI call: every step copies its inputs from pinned host memory,
        runs ekv_write_kv + ekv_attn_decode and copies its result back to the host.  The copies are double-buffered
        against the kernels (the H2D of step i+1 and the D2H of step i-1 overlap the kernels of step i); every byte
        still moves every step."""
        out = self.h_outs[self.e2e_i % 2]
        self.e2e_i += 1
        self.hs.decode(0, self.h_q, self.h_tables, self.h_lens, self.scale, out, h_k=self.h_k, h_v=self.h_v,
                       h_slot_mapping=self.h_slots)

    def finish_e2e(self):
        """Make the current stream wait for every copy still in flight (called inside the timed region)."""
        self.hs.flush()

    def h_out_check(self):
        """Result of the resident path, on the host: the end-to-end path must deliver the same bits."""
        self.step_resident()
        torch.cuda.synchronize(self.dev)
        return self.out.cpu()

    def e2e_bytes(self):
        h2d = sum(t.numel() * t.element_size() for t in (self.h_q, self.h_k, self.h_v, self.h_slots, self.h_tables,
                                                         self.h_lens))
        return h2d, self.h_out.numel() * self.h_out.element_size()

    def close(self):
        if getattr(self, "hs", None) is not None:
            self.hs.close()
            self.hs = None
        self.pool.close()


def max_over_ranks(ms: float, dist, device) -> float:
    """Replicas run independently; the job's time is the slowest rank's (all-reduce MAX of a device-timed value)."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def whole_job_gbs(step_bytes: int, steps: int, ms: float, world: int) -> float:
    """Aggregate throughput of `world` replicas that each moved step_bytes per step."""
    return world * step_bytes * steps / (ms * 1e-3) / 1e9


def timed_loop(fn, steps, device, dist):
    """barrier + sync, K steps between two CUDA events on the current stream, sync + barrier; max over ranks."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(device)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize(device)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize(device)
    ms = max_over_ranks(e0.elapsed_time(e1), dist, device)
    if dist is not None:
        dist.barrier()
    return ms


# ----------------------------------------------------------------------------- side measurements

# idle time before every timed prefill run (the sustained loop that follows each one-shot measurement has none)
PREFILL_IDLE_S = 0.1


def _time_reps(fn, device, reps, warmup=3, idle_s=0.0):
    """ms of `reps` separately timed runs of fn (CUDA events on the current stream), after `warmup` untimed runs.
    idle_s > 0: the device idles that long before every timed run, so that each one is a launch timed alone (what the
    burst matmul peak is) and not the tail of a loop that has run the part into its power cap."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize(device)
    ts = []
    for _ in range(reps):
        if idle_s > 0:
            time.sleep(idle_s)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize(device)
        ts.append(e0.elapsed_time(e1))
    return ts


def measure_prefill(device, peaks, reps=7, prompt_len=None, chunks=None, shape=None, sustained=True):
    """Prefill-chunk TFLOP/s on the configs[2] prompt: 32768 tokens as four 8192-token chunks over
    cached prefixes 0/8k/16k/24k, and as one 32768-token chunk.  Median of `reps` runs, with min and max."""
    import paper_2608_23658_b200 as ekv
    cfg, s = I.C3, shape or I.C3.shape
    Lp = prompt_len or cfg.prompt_len
    nblk = Lp // s.block_size
    pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=nblk + 64,
                    device=device.index or 0)
    try:
        live = pool.info.live_blocks
        table, _ = I.assign_blocks(cfg.seed, 13, torch.tensor([Lp]), s.block_size, live)
        I.fill_pool_layer_(pool.layer_tensor(0), cfg.seed)
        q = I.normal_bf16(cfg.seed, 6, 0, Lp * s.num_q_heads * s.head_dim, device=device).view(Lp, s.num_q_heads, s.head_dim)
        out = torch.empty_like(q)
        d_table = table.to(device)
        scale = 1.0 / math.sqrt(s.head_dim)
        res = {}
        # the one-shot chunk first: it carries the roofline figure, and a part that has just done
        # ~50 ms of dense tensor work runs into its power cap (ms_runs shows the drift within a measurement)
        for chunk in sorted(chunks or cfg.chunk_lens, reverse=True):
            calls = []
            for start in range(0, Lp, chunk):
                cu = torch.tensor([0, chunk], dtype=torch.int32)
                calls.append((q[start:start + chunk], out[start:start + chunk], cu.to(device), cu,
                              torch.tensor([start + chunk], dtype=torch.int32, device=device)))

            def run():
                for (qq, oo, cud, cuh, sl) in calls:
                    pool.attn_prefill_chunk(0, qq, d_table, cud, cuh, sl, scale, out=oo)
            ts = _time_reps(run, device, reps, idle_s=PREFILL_IDLE_S)
            med = statistics.median(ts)
            flops = sum(I.prefill_flops(chunk, start, s) for start in range(0, Lp, chunk))
            tf = flops / (med * 1e-3) / 1e12
            res[f"chunk_{chunk}"] = {"ms": round(med, 3), "ms_min": round(min(ts), 3), "ms_max": round(max(ts), 3),
                                     "ms_runs": [round(t, 2) for t in ts],
                                     "tflops": round(tf, 1), "launches": len(calls),
                                     "tflops_best": round(flops / (min(ts) * 1e-3) / 1e12, 1),
                                     "frac_of_measured_bf16": round(tf / peaks["bf16_tflops"], 4),
                                     "frac_of_measured_bf16_sustained": round(tf / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]), 4),
                                     "frac_of_nominal_2250": round(tf / 2250.0, 4)}
            if len(calls) == 1 and sustained:
                # the same launch back to back for about a second, clocks sampled meanwhile: the figure to hold
                # against the sustained matmul peak, which was measured the same way
                n_loop = max(8, int(1000.0 / med))
                with ClockSampler(device.index or 0) as cs:
                    cs.wait_for_samples(1)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    torch.cuda.synchronize(device)
                    t0 = time.perf_counter()
                    e0.record()
                    for _ in range(n_loop):
                        run()
                    e1.record()
                    torch.cuda.synchronize(device)
                    t1 = time.perf_counter()
                    clk = cs.summary(t0, t1)
                ms_loop = e0.elapsed_time(e1) / n_loop
                tf_loop = flops / (ms_loop * 1e-3) / 1e12
                res[f"chunk_{chunk}"]["sustained"] = {
                    "launches": n_loop, "ms": round(ms_loop, 3), "tflops": round(tf_loop, 1),
                    "frac_of_measured_bf16_sustained": round(tf_loop / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]), 4),
                    "sm_mhz": clk["sm_mhz"], "reasons": clk["reasons"]}
                time.sleep(0.5)     # let the part leave its power cap before the next measurement
        res["workload"] = (f"c3 prompt {Lp} tokens, {s.num_q_heads}/{s.num_kv_heads} heads d{s.head_dim}, causal-exact FLOPs of both "
                           f"contractions, median of {reps} runs with {int(PREFILL_IDLE_S * 1e3)} ms of idle before each")
        return res
    finally:
        pool.close()


def measure_prefill_short(device, peaks, reps=5):
    """The same 32768 query tokens as many short prompts without a cached prefix, one call per batch:
    64 prompts of 512 tokens and 256 prompts of 128 tokens (what a batch of fresh short requests looks like)."""
    import paper_2608_23658_b200 as ekv
    cfg, s = I.C3, I.C3.shape
    T = 32768
    res = {}
    for R, c in ((64, 512), (256, 128)):
        lengths = torch.full((R,), c, dtype=torch.int64)
        pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim,
                        base_blocks=T // s.block_size + 64, device=device.index or 0)
        try:
            tables, _ = I.assign_blocks(cfg.seed, 15, lengths, s.block_size, pool.info.live_blocks)
            I.fill_pool_layer_(pool.layer_tensor(0), cfg.seed)
            q = I.normal_bf16(cfg.seed, 6, 0, T * s.num_q_heads * s.head_dim, device=device).view(T, s.num_q_heads, s.head_dim)
            out = torch.empty_like(q)
            cu = torch.arange(0, T + 1, c, dtype=torch.int32)
            d_cu, d_tables, d_lens = cu.to(device), tables.to(device), lengths.to(torch.int32).to(device)
            scale = 1.0 / math.sqrt(s.head_dim)
            ts = _time_reps(lambda: pool.attn_prefill_chunk(0, q, d_tables, d_cu, cu, d_lens, scale, out=out), device, reps)
            med = statistics.median(ts)
            tf = R * I.prefill_flops(c, 0, s) / (med * 1e-3) / 1e12
            res[f"{R}x{c}"] = {"ms": round(med, 4), "ms_min": round(min(ts), 4), "tflops": round(tf, 1),
                               "frac_of_measured_bf16": round(tf / peaks["bf16_tflops"], 4)}
        finally:
            pool.close()
    res["workload"] = "32768 query tokens as R prompts of c tokens, no cached prefix, one call, 32/8 heads d128"
    return res


def measure_mixed_step(device, peaks, reps=5):
    """configs[2] as one engine step: the last 8192-token chunk of the 32768-token prompt (cached prefix 24576)
    co-scheduled with the 256-sequence decode batch.  Timed three ways: each call alone, both back to back on
    one stream, and both at once on two streams (what a scheduler that batches them gets)."""
    import paper_2608_23658_b200 as ekv
    cfg, s = I.C3, I.C3.shape
    Lp, chunk = cfg.prompt_len, 8192
    lengths = torch.cat([torch.tensor([Lp]), I.decode_lengths(cfg)])
    need = int(I.blocks_for(lengths, s.block_size).sum())
    pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim,
                    base_blocks=int(need * 1.05) + 64, device=device.index or 0)
    try:
        tables, _ = I.assign_blocks(cfg.seed, 14, lengths, s.block_size, pool.info.live_blocks)
        I.fill_pool_layer_(pool.layer_tensor(0), cfg.seed)
        B = len(lengths) - 1
        d_tables = tables.to(device)
        p_table, d_table = d_tables[:1].contiguous(), d_tables[1:].contiguous()
        d_lens = lengths[1:].to(torch.int32).to(device)
        qp = I.normal_bf16(cfg.seed, 6, 0, chunk * s.num_q_heads * s.head_dim, device=device).view(chunk, s.num_q_heads, s.head_dim)
        qd = I.normal_bf16(cfg.seed, 7, 0, B * s.num_q_heads * s.head_dim, device=device).view(B, s.num_q_heads, s.head_dim)
        op, od = torch.empty_like(qp), torch.empty_like(qd)
        cu_h = torch.tensor([0, chunk], dtype=torch.int32)
        cu_d = cu_h.to(device)
        p_len = torch.tensor([Lp], dtype=torch.int32, device=device)
        ws = pool.workspace(B, int(d_table.shape[1]) * s.block_size)
        scale = 1.0 / math.sqrt(s.head_dim)
        side = torch.cuda.Stream(device)
        main = torch.cuda.current_stream(device)

        def prefill():
            pool.attn_prefill_chunk(0, qp, p_table, cu_d, cu_h, p_len, scale, out=op)

        def decode():
            pool.attn_decode(0, qd, d_table, d_lens, scale, out=od, workspace=ws)

        def serial():
            prefill()
            decode()

        def concurrent():
            fork, join = torch.cuda.Event(), torch.cuda.Event()
            fork.record(main)
            side.wait_event(fork)
            with torch.cuda.stream(side):
                decode()
                join.record(side)
            prefill()
            main.wait_event(join)

        def best_of(fn):
            fn()
            torch.cuda.synchronize(device)
            best = float("inf")
            for _ in range(reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                torch.cuda.synchronize(device)
                best = min(best, e0.elapsed_time(e1))
            return best

        t_p, t_d, t_s, t_c = best_of(prefill), best_of(decode), best_of(serial), best_of(concurrent)
        flops = I.prefill_flops(chunk, Lp - chunk, s)
        dbytes = I.decode_algorithmic_bytes(lengths[1:], s)
        return {"prefill_alone_ms": round(t_p, 3), "prefill_alone_tflops": round(flops / (t_p * 1e-3) / 1e12, 1),
                "decode_alone_ms": round(t_d, 3), "decode_alone_gbs": round(dbytes / (t_d * 1e-3) / 1e9, 1),
                "serial_ms": round(t_s, 3), "two_streams_ms": round(t_c, 3),
                "workload": "c3 step: 8192-token chunk over a 24576-token cached prefix + 256 decode sequences U[2048,8192]"}
    finally:
        pool.close()


def _toggle_modes(device, num_layers, per_layer_bytes, cycles, fused=False):
    """grow / shrink ms for one geometry, three ways: keep the range and re-create the handle (default), keep
    range and handle (EKV_KEEP_PHYSICAL), and the naive way -- a fresh range + handle + mapping per toggle."""
    import paper_2608_23658_b200 as ekv
    s = I.C5.shape
    el_blocks = per_layer_bytes // s.block_bytes
    geom = dict(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, num_layers=num_layers,
                device=device.index or 0, fused_range=fused)
    pool = ekv.Pool(base_blocks=el_blocks + 512, elastic_blocks=el_blocks, **geom)
    try:
        rows = {"grow_release": [], "shrink_release": [], "grow_keep": [], "shrink_keep": []}
        for _ in range(cycles):
            rows["grow_release"].append(pool.grow())
            rows["shrink_release"].append(pool.shrink())
        pool.grow()
        for _ in range(cycles):
            rows["shrink_keep"].append(pool.shrink(keep_physical=True))
            rows["grow_keep"].append(pool.grow())
        out = {k: {"driver_ms_median": round(statistics.median(r[0] for r in v), 3),
                   "call_ms_median": round(statistics.median(r[1] for r in v), 3),
                   "call_ms_max": round(max(r[1] for r in v), 3)} for k, v in rows.items()}
        # drain: move every elastic block of every layer to a base block (what a decommit does before the unmap)
        src = torch.arange(pool.info.base_blocks, pool.info.base_blocks + el_blocks, dtype=torch.int32, device=device)
        dst = torch.arange(0, el_blocks, dtype=torch.int32, device=device)
        ekv.ekv_move_blocks(pool.handle, src, dst)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ekv.ekv_move_blocks(pool.handle, src, dst)
        e1.record()
        torch.cuda.synchronize(device)
        moved = 2 * num_layers * el_blocks * s.block_bytes
        out["drain_move_blocks"] = {"ms": round(e0.elapsed_time(e1), 3), "gbs_read_plus_write": round(moved / e0.elapsed_time(e1) / 1e6, 1),
                                    "blocks": el_blocks * num_layers}
    finally:
        pool.close()
    # naive: nothing is kept between toggles -- reserve, create, map and grant a new range per layer at every commit
    naive_c, naive_d = [], []
    for _ in range(cycles):
        torch.cuda.synchronize(device)
        t0 = time.perf_counter()
        fresh = ekv.Pool(base_blocks=el_blocks, **geom)
        t1 = time.perf_counter()
        fresh.close()
        t2 = time.perf_counter()
        naive_c.append((t1 - t0) * 1e3)
        naive_d.append((t2 - t1) * 1e3)
    out["naive_commit_fresh_range"] = {"call_ms_median": round(statistics.median(naive_c), 3), "call_ms_max": round(max(naive_c), 3)}
    out["naive_decommit_fresh_range"] = {"call_ms_median": round(statistics.median(naive_d), 3), "call_ms_max": round(max(naive_d), 3)}
    out["workload"] = f"{num_layers} layers x {per_layer_bytes >> 20} MiB elastic ({num_layers * per_layer_bytes / 2**30:.2f} GiB), {cycles} cycles per mode"
    return out


def measure_toggle(device, cycles=5):
    """grow / shrink ms on the configs[4] geometry (32 layers x 96 MiB = 3 GiB) and on the paper's own toggle
    microbenchmark geometry (28 layers, 3.09 GiB in all; its numbers are from another machine: context only)."""
    cfg = I.C5
    out = _toggle_modes(device, cfg.num_layers, cfg.elastic_total_bytes // cfg.num_layers, cycles)
    # the same reserve as ONE range and two handles for all layers (EKV_FUSED_RANGE): one map / unmap per toggle
    out["fused_range"] = _toggle_modes(device, cfg.num_layers, cfg.elastic_total_bytes // cfg.num_layers, cycles, fused=True)
    out["paper_geometry_28_layers"] = _toggle_modes(device, 28, (int(3.09 * 2**30) // 28 // (2 << 20) + 1) * (2 << 20), cycles)
    out["paper_a100_context_ms"] = {"decommit": 3.0, "commit": 30.0, "naive_commit": 180.0, "live_decommit": 3.8, "live_commit": 23.8}
    return out


def measure_write_kv(device, peaks):
    """ekv_write_kv bandwidth at the chunk sizes of configs[2] (8192 and 32768 tokens), L2 flushed between reps."""
    import paper_2608_23658_b200 as ekv
    s = I.C3.shape
    res = {}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    for T in (8192, 32768):
        pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim, base_blocks=T // 16 + 64,
                        device=device.index or 0)
        try:
            live = pool.info.live_blocks
            slots = (I.permutation(I.C3.seed, 14, live)[:T // 16].repeat_interleave(16) * 16 + torch.arange(T) % 16).to(device)
            n = T * s.num_kv_heads * s.head_dim
            k = I.normal_bf16(I.C3.seed, 7, 0, n, device=device).view(T, s.num_kv_heads, s.head_dim)
            v = I.normal_bf16(I.C3.seed, 8, 0, n, device=device).view(T, s.num_kv_heads, s.head_dim)
            for _ in range(3):
                pool.write_kv(0, k, v, slots)
            ts = []
            for _ in range(7):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                pool.write_kv(0, k, v, slots)
                e1.record()
                torch.cuda.synchronize(device)
                ts.append(e0.elapsed_time(e1))
            ms = statistics.median(ts)
            gbs = I.write_algorithmic_bytes(T, s) / ms / 1e6
            # the same number of bytes moved by one plain device copy, timed the same way: what a launch of this
            # size can reach at all (the measured peak is for a 2 GiB copy)
            src = torch.cat([k.view(-1), v.view(-1)])
            dst = torch.empty_like(src)
            tc = []
            for _ in range(7):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                dst.copy_(src)
                e1.record()
                torch.cuda.synchronize(device)
                tc.append(e0.elapsed_time(e1))
            res[f"tokens_{T}"] = {"ms": round(ms, 4), "gbs_read_plus_write": round(gbs, 1),
                                  "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 4),
                                  "plain_copy_same_bytes_ms": round(statistics.median(tc), 4)}
        finally:
            pool.close()
    res["workload"] = "slot-mapped write of K and V rows, 8 kv heads x 128 channels, blocks scattered over the pool"
    return res


def measure_decode_long_context(device, peaks, reps=5, hbm_filling=False):
    """Decode attention on the configs[3] batch (64 sequences, 64q/8kv heads, contexts U[32768,131072], 21.3 GB of KV
    per launch).  hbm_filling=False: a pool just large enough for the batch.  hbm_filling=True: the pool configs[3]
    describes -- min(140 GiB, free memory - 10 GiB), 16 % of its block ids elastic, the batch's blocks drawn by a
    uniform permutation over ALL of it (only the blocks the batch touches are filled) -- so that the table walk
    jumps over the whole of HBM and the translation reach of the memory system is part of what is timed."""
    import paper_2608_23658_b200 as ekv
    cfg, s = I.C4, I.C4.shape
    lengths = I.decode_lengths(cfg)
    need = int(I.blocks_for(lengths, s.block_size).sum())
    if hbm_filling:
        free, _ = torch.cuda.mem_get_info(device)
        total = min(140 << 30, free - (10 << 30)) // s.block_bytes
        if total < need * 1.02:
            return {"skipped": f"only {free / 2**30:.1f} GiB free: the pool cannot hold the draw"}
    else:
        total = int(need * 1.02)
    elastic = int(total * cfg.elastic_fraction)
    pool = ekv.Pool(num_q_heads=s.num_q_heads, num_kv_heads=s.num_kv_heads, head_dim=s.head_dim,
                    base_blocks=total - elastic, elastic_blocks=elastic, start_grown=True, device=device.index or 0)
    try:
        live = pool.info.live_blocks
        tables, _ = I.assign_blocks(cfg.seed, 12, lengths, s.block_size, live)
        view = pool.layer_tensor(0)
        if hbm_filling:
            ids_sorted = torch.sort(tables[tables >= 0].long()).values.to(device)
            ar = torch.arange(s.block_elems, device=device)[None]
            for o in range(0, len(ids_sorted), 4096):
                idx = ids_sorted[o:o + 4096]
                vals = I.normal_bf16_at(cfg.seed, I.KV_STREAM, (idx[:, None] * s.block_elems + ar).reshape(-1))
                view[idx] = vals.view(len(idx), 2, s.num_kv_heads, s.block_size, s.head_dim)
        else:
            I.fill_pool_layer_(view, cfg.seed, chunk=1 << 26)
        B = len(lengths)
        q = I.normal_bf16(cfg.seed, 3, 0, B * s.num_q_heads * s.head_dim, device=device).view(B, s.num_q_heads, s.head_dim)
        d_tables, d_lens = tables.to(device), lengths.to(torch.int32).to(device)
        ws = pool.workspace(B, int(tables.shape[1]) * s.block_size)
        out = torch.empty_like(q)
        scale = 1.0 / math.sqrt(s.head_dim)
        for _ in range(3):
            pool.attn_decode(0, q, d_tables, d_lens, scale, out=out, workspace=ws)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            pool.attn_decode(0, q, d_tables, d_lens, scale, out=out, workspace=ws)
        e1.record()
        torch.cuda.synchronize(device)
        ms = e0.elapsed_time(e1) / reps
        nbytes = I.decode_algorithmic_bytes(lengths, s)
        gbs = nbytes / ms / 1e6
        return {"ms": round(ms, 3), "gbs": round(gbs, 1), "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 4),
                "frac_of_nominal_8000": round(gbs / 8000.0, 4), "algorithmic_bytes": nbytes,
                "pool_gib": round(live * s.block_bytes / 2**30, 1), "elastic_fraction_of_blocks": round(elastic / live, 3),
                "workload": "c4 decode: 64 seqs, 64q/8kv heads d128, contexts U[32768,131072], " +
                            ("HBM-filling pool, blocks scattered over all of it" if hbm_filling else "pool just large enough")}
    finally:
        pool.close()


# ----------------------------------------------------------------------------- CPU oracle legs


def _generator_device():
    """Where the seeded value generator runs when a host mirror is built: the bits are the same on every torch
    device (integer arithmetic and one IEEE multiply), a GPU just produces gigabytes of them in seconds."""
    return "cuda" if torch.cuda.is_available() else "cpu"


def oracle_decode_sample(cfg, max_seqs=None):
    """Times the CPU oracle, as it stands, on the decode workload: all of its sequences when the host mirror can be
    generated quickly (a GPU is present), otherwise the first 24."""
    import oracle
    s = cfg.shape
    lengths = I.decode_lengths(cfg)
    if max_seqs is None:
        max_seqs = len(lengths) if _generator_device() == "cuda" else 24
    need = int(I.blocks_for(lengths, s.block_size).sum())
    tables, _ = I.assign_blocks(cfg.seed, 12, lengths, s.block_size, int(need * 1.1) + 64)
    ids = list(range(min(max_seqs, len(lengths))))
    cache, ctab, clen = I.compact_host_cache(cfg.seed, 0, tables, lengths, ids, s, device=_generator_device())
    q = I.normal_bf16(cfg.seed, 3, 0, len(lengths) * s.num_q_heads * s.head_dim).view(len(lengths), s.num_q_heads, s.head_dim)
    qs = q[ids].contiguous()
    scale = 1.0 / math.sqrt(s.head_dim)
    oracle.attn_decode(cache, s.num_q_heads, s.num_kv_heads, s.block_size, s.head_dim, qs[:1], ctab[:1], clen[:1], scale)
    nbytes = I.decode_algorithmic_bytes(clen, s)

    def one():
        t0 = time.perf_counter()
        oracle.attn_decode(cache, s.num_q_heads, s.num_kv_heads, s.block_size, s.head_dim, qs, ctab, clen, scale)
        return time.perf_counter() - t0
    which = "all" if len(ids) == len(lengths) else f"{len(ids)} of"
    return one, nbytes, f"{which} {len(lengths)} sequences of the workload ({int(clen.sum())} cached tokens, all heads)", \
        oracle.threads()


def oracle_prefill_sample(rows_per_chunk=16):
    """The CPU oracle on a row sample of the configs[2] prompt (32768 tokens, one request, no prefix): first and
    last row of every 8192-token chunk plus rows spread evenly, all 32 heads.  Returns a dict with its GFLOP/s
    (causal-exact FLOPs of the sampled rows only)."""
    import oracle
    cfg, s = I.C3, I.C3.shape
    Lp = cfg.prompt_len
    table, _ = I.assign_blocks(cfg.seed, 13, torch.tensor([Lp]), s.block_size, Lp // s.block_size + 64)
    cache, ctab, clen = I.compact_host_cache(cfg.seed, 0, table, torch.tensor([Lp]), [0], s, device=_generator_device())
    q = I.normal_bf16(cfg.seed, 6, 0, Lp * s.num_q_heads * s.head_dim).view(Lp, s.num_q_heads, s.head_dim)
    rows = set()
    for start in range(0, Lp, 8192):
        rows |= {start, start + 8191} | {start + (8192 * k) // rows_per_chunk for k in range(rows_per_chunk)}
    rows = sorted(rows)
    cu = torch.tensor([0, Lp], dtype=torch.int32)
    scale = 1.0 / math.sqrt(s.head_dim)
    t0 = time.perf_counter()
    oracle.attn_prefill_chunk(cache, s.num_q_heads, s.num_kv_heads, s.block_size, s.head_dim, q, ctab, cu, clen, scale,
                              rows=torch.tensor(rows, dtype=torch.int32))
    dt = time.perf_counter() - t0
    flops = 4 * s.head_dim * s.num_q_heads * sum(r + 1 for r in rows)
    return {"gflops": round(flops / dt / 1e9, 2), "seconds": round(dt, 3), "cores": oracle.threads(),
            "sample": f"{len(rows)} of {Lp} query rows of the c3 prompt (chunk borders + evenly spread), all heads"}


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = I.C2
    one, nbytes, sample, cores = oracle_decode_sample(cfg)
    for _ in range(args.warmup):
        one()
    times = [one() for _ in range(args.steps)]
    total = sum(times)
    value = nbytes * args.steps / total / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(1e3 * total / args.steps, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "batch": cfg.decode.batch, "heads": "32q/8kv", "head_dim": 128, "block_size": 16,
                       "step": "oracle attn_decode (the write of the step's 256 rows is not timed)", "sample": sample},
            "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- main


def _free_port():
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def spawn_ranks(n: int, argv) -> int:
    """`bench.py --gpus N` started plainly (no torchrun): start the N ranks here, one process per GPU, each with
    the environment torchrun would give it (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR, MASTER_PORT).  Rank 0's
    stdout is this process's stdout, so its JSON line is the job's.  Returns the worst exit code."""
    port = _free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *argv], env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    return max(abs(p.wait()) for p in procs)


def run_stub(args, rank, world):
    """Test hook (--stub-ms): the launch, rendezvous, timing and reporting logic of a replica run with the GPU step
    replaced by a host sleep of (rank + 1) x stub_ms and the process group on gloo, so that the multi-rank path can
    be exercised on a machine without GPUs."""
    import torch.distributed as dist
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cpu = torch.device("cpu")
    dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(args.stub_ms * (rank + 1) * 1e-3)
    local_ms = (time.perf_counter() - t0) * 1e3
    ms = max_over_ranks(local_ms, dist, cpu)
    dist.barrier()
    if rank == 0:
        step_bytes = 1_000_000_000
        print(json.dumps({"metric": METRIC, "value": round(whole_job_gbs(step_bytes, args.steps, ms, world), 3), "unit": UNIT,
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4),
                          "scaling": "weak", "data": "stub", "local_ms_rank0": round(local_ms, 3),
                          "config": {"workload": "stub step (host sleep), replicas only"}}), flush=True)
    dist.destroy_process_group()


def main(argv=None):
    argv = list(sys.argv[1:] if argv is None else argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ekv", choices=["ekv", "reference"])
    ap.add_argument("--batch", type=int, default=None, help="debug: fewer sequences than the named workload")
    ap.add_argument("--no-extras", action="store_true", help="skip prefill / toggle / cpu_baseline side measurements")
    ap.add_argument("--prefill-only", type=int, default=0, metavar="PROMPT_LEN",
                    help="profiling aid: run only the prefill-chunk measurement on a prompt of this length "
                         "(one-shot and in 4 chunks) and print its JSON")
    ap.add_argument("--prefill-short-only", action="store_true",
                    help="profiling aid: run only the many-short-prompts prefill measurement and print its JSON")
    ap.add_argument("--write-kv-only", action="store_true",
                    help="profiling aid: run only the ekv_write_kv measurement (8192 and 32768 tokens) and print its JSON")
    ap.add_argument("--stub-ms", type=float, default=0.0,
                    help="test hook: replace the GPU step by a host sleep of (rank+1) x this many ms, ranks on gloo")
    args = ap.parse_args(argv)
    args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        run_reference(args)
        return 0

    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        return spawn_ranks(args.gpus, argv)
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if args.stub_ms > 0:
        run_stub(args, rank, world)
        return 0
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the ekv path has no CPU fallback (use --impl reference for the oracle)")
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=device)
        dist = dist_mod

    peaks, peaks_kind = measured_peaks()
    if args.prefill_only:
        n = args.prefill_only
        print(json.dumps({"prefill": measure_prefill(device, peaks, reps=3, prompt_len=n, chunks=(n // 4, n))}), flush=True)
        return 0
    if args.prefill_short_only:
        print(json.dumps({"prefill_short": measure_prefill_short(device, peaks, reps=3)}), flush=True)
        return 0
    if args.write_kv_only:
        print(json.dumps({"write_kv": measure_write_kv(device, peaks)}), flush=True)
        return 0
    cfg = I.C2
    wl = DecodeWorkload(cfg, device, args.batch)
    assert wl.decode_bytes > 200e6 or args.batch, "working set must exceed L2"

    for _ in range(args.warmup):
        wl.step_resident()
    # per-step kernel-group durations, measured live inside the timed region
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    it = iter(evs)
    with ClockSampler(device.index or 0) as clk:
        clk.wait_for_samples(1)
        t_load0 = time.perf_counter()
        ms = timed_loop(lambda: wl.step_resident(next(it)), args.steps, device, dist)
        t_load1 = time.perf_counter()
        clocks = clk.summary(t_load0, t_load1)
        clocks["window"] = "timed region"
        if clocks["samples"] < 3:
            # The timed region is shorter than the sampling period: keep the SAME load running, untimed,
            # until the sampler has seen it, and report those samples (the window says so).
            t_load0 = time.perf_counter()
            while time.perf_counter() - t_load0 < 0.6:
                for _ in range(20):
                    wl.step_resident()
                torch.cuda.synchronize(device)
            clocks = clk.summary(t_load0, time.perf_counter())
            clocks["window"] = "same steps repeated for 0.6 s right after the timed region (region < sampling period)"
    write_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in evs)
    decode_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in evs)
    st = wl.pool.poll_status()
    if st != 0:
        raise SystemExit(f"bench.py: device status {st!r} after the timed region")

    wl.setup_e2e()
    for _ in range(args.warmup):
        wl.step_e2e()
    wl.finish_e2e()
    e2e_count = [0]

    def e2e_step():
        wl.step_e2e()
        e2e_count[0] += 1
        if e2e_count[0] == args.steps:
            wl.finish_e2e()                              # the last D2H copies end inside the timed region
    ms_e2e = timed_loop(e2e_step, args.steps, device, dist)
    assert torch.equal(wl.h_outs[0], wl.h_out_check()) and torch.equal(wl.h_outs[1], wl.h_outs[0])

    step_bytes = wl.decode_bytes + wl.write_bytes
    value = whole_job_gbs(step_bytes, args.steps, ms, world)
    e2e_value = whole_job_gbs(step_bytes, args.steps, ms_e2e, world)
    achieved = wl.decode_bytes / (decode_ms * 1e-3) / 1e9
    h2d, d2h = wl.e2e_bytes()
    nsplit = wl.ekv.ekv_attn_decode_plan(wl.pool.handle, wl.B, int(wl.tables.shape[1]))[1]
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms / args.steps, 4), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "batch": wl.B, "heads": "32q/8kv", "head_dim": 128, "block_size": 16,
                   "context_tokens": int(wl.lengths.sum()), "step": "ekv_write_kv + ekv_attn_decode (split + combine)",
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                   "l2": "inputs larger than L2 (%.2f GB of KV per step)" % (wl.decode_bytes / 1e9)},
        "gpu_launches": (2 + (1 if nsplit > 1 else 0)) * args.steps,
        "clocks": clocks,
    }
    roofline = {"bound": "hbm", "kernel": "decode_split_kernel<128, false> + decode_combine_kernel<128>",
                "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": round(achieved / peaks["hbm_gbs"], 4), "peak_kind": f"{peaks_kind} copy bandwidth",
                "frac_of_nominal_8000": round(achieved / 8000.0, 4), "traffic": int(DECODE_SPLIT_DRAM_TRAFFIC_RATIO * wl.decode_bytes),
                "algorithmic_bytes_per_launch": wl.decode_bytes, "launch_ms": round(decode_ms, 4),
                "write_kv_ms": round(write_ms, 4)}
    e2e = {"value": round(e2e_value, 1), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "ms_per_step": round(ms_e2e / args.steps, 4)}
    wl.close()
    if rank == 0 and world == 1 and not args.no_extras:
        # Side measurements of the other hot-path rows.  They are MEASURED in the order prefill, short prompts, mixed
        # step, write, long-context decode, toggles (the tensor-bound kernel first, before minutes of pool filling have
        # heated the part), and PRINTED with the bulky one (toggle) first and the compact ones last, so that the end
        # of the line holds prefill, mixed step, long-context decode, write and the CPU baseline.
        torch.cuda.empty_cache()
        pf = measure_prefill(device, peaks)
        # the same prompt on the head layout of the paper's model (28 query / 4 kv heads: groups of 7, an odd number)
        pf_g7 = measure_prefill(device, peaks, reps=5, chunks=(I.C3.prompt_len,), shape=I.Shape(28, 4, 128), sustained=False)
        torch.cuda.empty_cache()
        pf_short = measure_prefill_short(device, peaks)
        torch.cuda.empty_cache()
        mixed = measure_mixed_step(device, peaks)
        torch.cuda.empty_cache()
        wkv = measure_write_kv(device, peaks)
        torch.cuda.empty_cache()
        c4 = measure_decode_long_context(device, peaks)
        torch.cuda.empty_cache()
        c4_full = measure_decode_long_context(device, peaks, hbm_filling=True)
        torch.cuda.empty_cache()
        line["toggle"] = measure_toggle(device)
        line["decode_long_context_hbm_filling_pool"] = c4_full
        line["decode_long_context"] = c4
        line["write_kv"] = wkv
        line["mixed_step"] = mixed
        line["prefill_short"] = pf_short
        g7 = pf_g7[f"chunk_{I.C3.prompt_len}"]
        line["prefill_group_of_7"] = {"ms": g7["ms"], "ms_min": g7["ms_min"], "tflops": g7["tflops"],
                                      "frac_of_measured_bf16": g7["frac_of_measured_bf16"], "workload": pf_g7["workload"]}
        line["prefill"] = pf
        one_shot = pf["chunk_32768"]
        line["roofline_prefill"] = {
            "bound": "tensor", "kernel": "prefill_tc_kernel", "achieved": one_shot["tflops"], "peak": peaks["bf16_tflops"],
            "unit": "TFLOP/s", "frac": one_shot["frac_of_measured_bf16"], "peak_kind": f"{peaks_kind} cuBLAS bf16 burst",
            "frac_of_sustained_peak": one_shot["frac_of_measured_bf16_sustained"], "best_of_runs": one_shot["tflops_best"],
            "launch_ms": one_shot["ms"],
            "workload": f"c3 prompt, one 32768-token chunk, median of 7 launches timed alone ({int(PREFILL_IDLE_S * 1e3)} ms of idle before each); "
                        "sustained_loop = the same launch back to back for a second",
            "chunked_4x8192_tflops": pf["chunk_8192"]["tflops"], "sustained_loop": one_shot.get("sustained"),
            "traffic": None}
        one, nbytes, sample, cores = oracle_decode_sample(cfg)
        one()
        reps, t = 0, 0.0
        while t < 10.0 and reps < 60:
            t += one()
            reps += 1
        line["cpu_baseline"] = {"value": round(nbytes * reps / t / 1e9, 3), "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{sample}, {reps} passes", "ms_per_pass": round(1e3 * t / reps, 1),
                                "prefill_rows": oracle_prefill_sample()}
    line["e2e"] = e2e
    line["roofline"] = roofline
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
