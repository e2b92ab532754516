#!/usr/bin/env python
"""Benchmark of the GEAR hot path on B200: decode steps over a compressed KV cache.

Workload (configuration C2): one LLaMA-2-7B-shaped attention layer, batch 8, 32 heads, d_H = 128,
context 4096, 2-bit codes with group 64, s = 2 % outliers, rank 4, streaming buffer n_b = 64.
`--layers` independent layer caches are rotated so that the bytes touched between two uses of a cache
exceed the 126 MB L2.

A step is one buffer cycle of every layer: n_b decode iterations, each = gear_append_buffer (the push that
fills the buffer compresses it: Filter, Quant, residual, power iteration, store) + gear_decode_attn over the
whole compressed cache and the fp16 buffer.  `value` = batch / mean latency of one layer's decode iteration
(append + its share of the flush + attention), summed over ranks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2]
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2403_05527_b200 import synth  # noqa: E402

METRIC = "compressed-KV decode attn tokens/s"
DECODE_DRAM_BYTES_PER_ALGORITHMIC_BYTE = 1.015
UNIT = "tokens/s"


def workload_name(w, layers):
    return (f"{w.name}; state: prefill segment + growing flush segments + fp16 buffer; "
            f"{layers} rotating layer caches (inputs larger than L2)")


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.rows:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                clk, mxc = float(parts[0]), float(parts[1])
            except ValueError:
                continue
            mx = mxc
            if t0 - 0.05 <= ts <= t1 + 0.15:
                sm.append(clk)
                for n, v in zip(names, parts[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------- the oracle arm
def oracle_unit_cycle(w, unit_seed, n_decode):
    """One (batch, head) unit through the oracle: prefill compress (untimed), then one buffer cycle of n_b pushes
    with `n_decode` evenly spaced decode-attention calls timed; returns seconds per decode iteration of the unit
    (push + flush share + attention)."""
    from oracle import gear_oracle as O
    k16, v16 = synth.make_kv(w.config_id, 1, 1, w.n, 128, extra=unit_seed)
    b0 = synth.make_b0(w.config_id, 1, 1, 128, w.rank, extra=unit_seed)
    cache = O.OracleCache(1, 1, 1, 128, w.bits, w.group, w.s_pct, w.buffer_cap, w.rank, w.power_iters)
    cache.compress(k16, v16, w.rank, b0)
    ks, vs = synth.make_appended(w.config_id, 1, 1, 128, w.buffer_cap)
    q = synth.make_query(w.config_id, 1, 1, 128, extra=unit_seed)
    every = max(1, w.buffer_cap // n_decode)
    t_push = t_attn = 0.0
    n_attn = 0
    for i in range(w.buffer_cap):
        t0 = time.perf_counter()
        cache.append(ks[i], vs[i], synth.make_b0(w.config_id, 1, 1, 128, w.rank, extra=7000 + i))
        t1 = time.perf_counter()
        t_push += t1 - t0
        if i % every == 0:
            cache.decode_attn(q)
            t_attn += time.perf_counter() - t1
            n_attn += 1
    return t_push / w.buffer_cap + t_attn / n_attn


def run_reference(args, w):
    from threadpoolctl import threadpool_limits
    units = w.batch * w.n_kv_heads
    per_iter = []
    with threadpool_limits(limits=1):
        for s in range(args.warmup + args.steps):
            t = oracle_unit_cycle(w, 100 + s, n_decode=4)
            if s >= args.warmup:
                per_iter.append(t)
    t_layer_iter = statistics.mean(per_iter) * units            # one core walks all (batch, head) units
    value = w.batch / t_layer_iter
    sample = (f"per step: 1 of {units} (batch, head) units, one buffer cycle of {w.buffer_cap} pushes incl. the flush, "
              f"4 of {w.buffer_cap} decode-attention calls timed; scaled by the unit count")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_layer_iter * w.buffer_cap * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(w, 1)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------- multi-rank reduction
def max_over_ranks(value, dist, device):
    """Largest `value` over all ranks (the job is as slow as its slowest rank); `dist` None means one rank."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world, batch_per_rank, calls_per_rank, seconds):
    """Every rank attends `batch_per_rank` sequences per call on its own shard of the batch (no exchange between
    ranks: (batch, head) units are independent), so the job's throughput is the sum over ranks."""
    return world * batch_per_rank * calls_per_rank / seconds


# --------------------------------------------------------------------------- our arm
def device_kv(torch, w, dev, seed):
    """K, V fp16 [B, H, n, 128] drawn on the device with the distribution of synth.make_kv."""
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    shape = (w.batch, w.n_kv_heads, w.n, 128)
    c = torch.exp(torch.randn(w.n_kv_heads, 128, generator=g, device=dev))[None, :, None, :]
    k = torch.randn(shape, generator=g, device=dev) * c
    k = torch.where(torch.rand(shape, generator=g, device=dev) < 0.01, k * 20.0, k).half()
    v = torch.randn(shape, generator=g, device=dev)
    v = torch.where(torch.rand(shape, generator=g, device=dev) < 0.01, v * 20.0, v).half()
    return k.contiguous(), v.contiguous()


def run_ours(args, w):
    import torch
    from paper_2403_05527_b200 import binding as G

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the GEAR path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    G.lib()

    L, nb, B = args.layers, w.buffer_cap, w.batch
    total_steps = args.warmup + args.steps + args.e2e_steps + 2
    max_tokens = w.n + total_steps * nb + nb
    cfg = G.make_config(B, w.n_q_heads, w.n_kv_heads, w.bits, w.group, w.s_pct, nb, w.rank, max_tokens,
                        rank_max=w.rank, power_iters=w.power_iters, seed=1234 + rank)
    caches, compress_ms = [], []
    # one untimed compress first: it grows the library's workspace pool to its working size (a driver allocation
    # that later calls do not repeat)
    k, v = device_kv(torch, w, dev, 999 + 1000 * rank)
    G.gear_free(G.gear_compress(G.gear_create(cfg), None, k, v, w.n, w.rank, None))
    del k, v
    for layer in range(L):
        k, v = device_kv(torch, w, dev, 1000 * rank + layer)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        cache = G.gear_create(cfg)                     # allocation is not part of the compress figure
        torch.cuda.synchronize()
        e0.record()
        caches.append(G.gear_compress(cache, None, k, v, w.n, w.rank, None))
        e1.record()
        torch.cuda.synchronize()
        compress_ms.append(e0.elapsed_time(e1))
        del k, v
    tok_shape = (B, w.n_kv_heads, 128)
    n_tok = 8
    g = torch.Generator(device=dev)
    g.manual_seed(77 + rank)
    new_k = (torch.randn((n_tok, *tok_shape), generator=g, device=dev)).half()
    new_v = (torch.randn((n_tok, *tok_shape), generator=g, device=dev)).half()
    q = torch.randn((B, w.n_q_heads, 128), generator=g, device=dev).half()
    outs = [torch.empty((B, w.n_q_heads, 128), dtype=torch.float32, device=dev) for _ in range(L)]
    # start the cycle with a half-full buffer
    for c in caches:
        for i in range(nb // 2):
            G.gear_append_buffer(c, new_k[i % n_tok], new_v[i % n_tok])
    torch.cuda.synchronize()

    def read_bytes(c):
        b = G.gear_cache_bytes(c)
        return b.codes + b.scale_zero + b.outliers + b.lowrank_a + b.lowrank_b + b.buffer

    buf_lens = [nb // 2] * L

    def step(events=None, bytes_log=None, flush_events=None):
        # One token per iteration: every layer pushes its new K/V row, then every layer attends.  The L decode launches
        # of an iteration sit between one pair of events with nothing else in between, so the decode figure holds the
        # kernels and the gaps between back-to-back launches, not the cost of recording events.
        for i in range(nb):
            for li, c in enumerate(caches):
                buf_lens[li] = (buf_lens[li] + 1) % nb
                will_flush = flush_events is not None and buf_lens[li] == 0
                if will_flush:
                    f0 = torch.cuda.Event(enable_timing=True); f0.record()
                G.gear_append_buffer(c, new_k[i % n_tok], new_v[i % n_tok])
                if will_flush:
                    f1 = torch.cuda.Event(enable_timing=True); f1.record()
                    flush_events.append((f0, f1))
            if events is not None:
                a0 = torch.cuda.Event(enable_timing=True); a0.record()
            for li, c in enumerate(caches):
                G.gear_decode_attn(c, q, outs[li])
            if events is not None:
                a1 = torch.cuda.Event(enable_timing=True); a1.record()
                events.append((a0, a1))
                bytes_log.append(sum(read_bytes(c) for c in caches))

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = G.gear_kernel_launches()
    events, bytes_log, flush_events = [], [], []
    t_wall0 = time.time()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record()
    for _ in range(args.steps):
        step(events, bytes_log, flush_events)
    s1.record()
    barrier()
    t_wall1 = time.time()
    launches = G.gear_kernel_launches() - launches0
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    ms_total = max_over_ranks(s0.elapsed_time(s1), dist, dev)
    status = [G.gear_last_device_status(c) for c in caches]
    if any(status):
        raise SystemExit(f"device status word set: {status}")
    if not all(torch.isfinite(o).all().item() for o in outs):
        raise SystemExit("non-finite attention output")

    n_calls = args.steps * nb * L
    value = whole_job_tokens_per_s(world, B, n_calls, ms_total * 1e-3)
    dec_ms = [a.elapsed_time(b) for a, b in events]       # one entry per group of L back-to-back decode launches
    dec_launches = len(dec_ms) * L
    dec_bytes = float(sum(bytes_log))
    achieved = dec_bytes / (sum(dec_ms) * 1e-3) / 1e9
    flush_ms = [a.elapsed_time(b) for a, b in flush_events]

    # ---- end to end through the host-buffer entry points (pinned host memory, copies inside the timed region)
    hk = torch.empty((n_tok, *tok_shape), dtype=torch.float16).pin_memory().copy_(new_k.cpu())
    hv = torch.empty((n_tok, *tok_shape), dtype=torch.float16).pin_memory().copy_(new_v.cpu())
    hq = torch.empty((B, w.n_q_heads, 128), dtype=torch.float16).pin_memory().copy_(q.cpu())
    hout = torch.empty((B, w.n_q_heads, 128), dtype=torch.float32).pin_memory()
    hk_np, hv_np, hq_np, hout_np = hk.numpy(), hv.numpy(), hq.numpy(), hout.numpy()

    def step_e2e():
        for i in range(nb):
            for c in caches:
                G.gear_append_buffer_host(c, hk_np[i % n_tok], hv_np[i % n_tok])
                G.gear_decode_attn_host(c, hq_np, hout_np)
    if args.e2e_steps > 0:
        step_e2e()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        step_e2e()
    barrier()
    e2e_s = max_over_ranks(max(time.perf_counter() - t0, 1e-9), dist, dev)
    e2e_value = whole_job_tokens_per_s(world, B, args.e2e_steps * nb * L, e2e_s)
    h2d = nb * L * (2 * hk_np[0].nbytes + hq_np.nbytes)
    d2h = nb * L * hout_np.nbytes

    line = None
    if rank == 0:
        peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(peaks_path):
            peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
        else:
            peak, peak_src = 6650.0, "fallback"
        # dram__bytes_read + dram__bytes_write of gear_decode_kernel<2,1,2> per algorithmic byte, from the ncu capture
        # summarised in profiles/gear_decode_kernel_C2.md (one layer cache; traffic grows in proportion to the cache)
        traffic = DECODE_DRAM_BYTES_PER_ALGORITHMIC_BYTE * dec_bytes / dec_launches if w.config_id == 2 else None
        in_bytes = 2 * B * w.n_kv_heads * w.n * 128 * 2
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic",
                "config": {"workload": workload_name(w, L), "batch_per_gpu": B, "layers_rotated": L,
                           "l2": "rotating caches: %.0f MB touched between reuses" % (dec_bytes / dec_launches * L / 1e6)},
                "roofline": {"bound": "hbm", "kernel": "gear_decode_kernel", "achieved": achieved, "peak": peak,
                             "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                             "frac_of_8000_nominal": achieved / 8000.0, "traffic": traffic,
                             "algorithmic_bytes_per_launch": dec_bytes / dec_launches,
                             "us_per_launch": 1e3 * sum(dec_ms) / dec_launches},
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
                "gpu_launches": int(launches),
                "clocks": clocks,
                "compress": {"prefill_gbs": in_bytes / (statistics.median(compress_ms) * 1e-3) / 1e9,
                             "prefill_ms": statistics.median(compress_ms),
                             "flush_us": 1e3 * statistics.median(flush_ms) if flush_ms else None,
                             "flush_gbs": (2 * B * w.n_kv_heads * nb * 128 * 2) / (statistics.median(flush_ms) * 1e-3) / 1e9
                             if flush_ms else None},
                "decode_attn_tokens_per_s_kernel_only": B / (1e-3 * sum(dec_ms) / dec_launches)}
        if not args.no_cpu and world == 1:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                t0 = time.perf_counter()
                per = [oracle_unit_cycle(w, 100 + s, n_decode=8) for s in range(args.cpu_units)]
                spent = time.perf_counter() - t0
            units = B * w.n_kv_heads
            line["cpu_baseline"] = {"value": B / (statistics.mean(per) * units), "unit": UNIT, "cores": 1,
                                    "kind": "oracle",
                                    "sample": f"{args.cpu_units} of {units} (batch, head) units, one buffer cycle each "
                                              f"(64 pushes incl. the flush, 8 decode-attention calls timed), scaled by "
                                              f"the unit count; {spent:.1f} s of CPU work incl. the untimed prefill compress"}
    for c in caches:
        G.gear_free(c)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--cpu-units", type=int, default=128)
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.config]
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) == 0:
            run_reference(args, w)
        return
    run_ours(args, w)


if __name__ == "__main__":
    main()
