#!/usr/bin/env python
"""Benchmark of the GEAR hot path on B200: decode steps over a compressed KV cache.

Headline workload (configuration C2): one LLaMA-2-7B-shaped attention layer, batch 8, 32 heads, d_H = 128,
context 4096, 2-bit codes with group 64, s = 2 % outliers, rank 4, streaming buffer n_b = 64.
`--layers` independent layer caches are rotated so that the bytes touched between two uses of a cache
exceed the 126 MB L2.

A step is one buffer cycle of every layer: n_b decode iterations, each = gear_append_buffer (the push that
fills the buffer compresses it: Filter, Quant, residual, power iteration, store) + gear_decode_attn over the
whole compressed cache and the fp16 buffer.  `value` = batch / mean latency of one layer's decode iteration
(append + its share of the flush + attention), summed over ranks.

The line also carries, under `extra`, the decode and compress figures of the other configurations (LLaMA-2-13B
shaped layer with 4- and 2-bit codes, Mistral-shaped grouped-query layer), each with its own roofline entry.

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
UNIT = "tokens/s"
# dram__bytes_read + dram__bytes_write of one gear_decode_kernel launch per algorithmic byte, by configuration, from ncu
# captures (one pass, the two counters) of the kernel as it stands on one layer cache: C2 137.40 MB of DRAM traffic for
# 134.26 MB; C4 121.77 MB for 118.48 MB; C3 4-bit 1072.05 MB for 1077.91 MB; C3 2-bit 736.20 MB for 738.39 MB; C6
# 193.67 MB for 191.34 MB (a ratio below one: the segment flushed just before the captured launch was still in L2);
# traffic grows in proportion to the cache
DECODE_DRAM_BYTES_PER_ALGORITHMIC_BYTE = {2: 1.0234, 4: 1.0277, 3: 0.9946, 32: 0.9970, 6: 1.0122}
EXTRA_CONFIGS = (3, 32, 4, 6)


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
    group = w.group if w.group else 1 << 30      # group 0 = per-vector grouping: no vector reaches this length
    cache = O.OracleCache(1, 1, 1, 128, w.bits, group, w.s_pct, w.buffer_cap, w.rank, w.power_iters)
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


def _pool_unit(job):
    """One oracle unit in a worker process, numeric libraries held to one thread."""
    config_id, seed, n_decode = job
    from threadpoolctl import threadpool_limits
    with threadpool_limits(limits=1):
        return oracle_unit_cycle(synth.WORKLOADS[config_id], seed, n_decode)


def oracle_all_cores(w, units_per_core=8, max_workers=32):
    """The oracle over independent (batch, head) units on every core the process may use: a pool of one-thread workers.
    Returns (tokens/s of the whole layer, cores used, units timed, wall seconds)."""
    import multiprocessing as mp
    cores = min(len(os.sched_getaffinity(0)), max_workers)
    jobs = [(w.config_id, 300 + i, 4) for i in range(cores * units_per_core)]
    ctx = mp.get_context("spawn")
    with ctx.Pool(cores) as pool:
        pool.map(_pool_unit, jobs[:cores])            # start the workers (imports, page-in) outside the timed region
        t0 = time.perf_counter()
        per = pool.map(_pool_unit, jobs)
        wall = time.perf_counter() - t0
    units = w.batch * w.n_kv_heads
    # `cores` units advance side by side: the layer's iteration takes units / cores rounds of the mean unit time
    t_layer_iter = statistics.mean(per) * units / cores
    return w.batch / t_layer_iter, cores, len(jobs), wall


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
            "extrapolated": "value and ms_per_step are the sampled unit's times scaled by the unit count",
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(w, args.layers)},
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


def rank_environment(rank, world, port):
    """Environment of one spawned rank (the launcher below sets it before the rank's main runs)."""
    return {"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world), "MASTER_ADDR": "127.0.0.1",
            "MASTER_PORT": str(port)}


def _spawned_rank(rank, world, port, argv, main_name):
    os.environ.update(rank_environment(rank, world, port))
    sys.argv = list(argv)
    globals()[main_name]()


def spawn_ranks(world, argv, main_name="main", port=None):
    """`python bench.py --gpus N` without a launcher: start N ranks of this file, one GPU each."""
    import socket
    import torch.multiprocessing as mp
    if port is None:
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
    mp.spawn(_spawned_rank, args=(world, port, argv, main_name), nprocs=world, join=True)


def rank_probe():
    """What a spawned rank sees, without a GPU: joins a gloo group from the environment the launcher set, reduces a
    time with max_over_ranks and writes its view to the file named last on the command line (one line per rank)."""
    import torch
    import torch.distributed as dist
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = max_over_ranks(10.0 + rank, dist, torch.device("cpu"))
        with open(sys.argv[-1] + f".{rank}", "w") as f:
            json.dump({"rank": rank, "world": world, "local_rank": int(os.environ["LOCAL_RANK"]), "ms": ms,
                       "value": whole_job_tokens_per_s(world, 8, 10, ms * 1e-3)}, f)
        dist.barrier()
    finally:
        dist.destroy_process_group()


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


def hbm_peak():
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        return float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def measure_config(torch, G, dev, w, layers, steps, warmup, rank, e2e_steps=0, dist=None, world=1, sampler_index=None):
    """Build `layers` caches of workload w, run `warmup` + `steps` buffer cycles and time them.  Returns a dict of raw
    measurements (CUDA events on the launching stream)."""
    L, nb, B = layers, w.buffer_cap, w.batch
    total_steps = warmup + steps + e2e_steps + 2
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
    prefill_out_bytes = G.gear_cache_bytes(caches[0]).stored_total
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

    for _ in range(warmup):
        step()
    barrier()
    sampler = ClockSampler(sampler_index) if sampler_index is not None else None
    launches0 = G.gear_kernel_launches()
    events, bytes_log, flush_events = [], [], []
    t_wall0 = time.time()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record()
    for _ in range(steps):
        step(events, bytes_log, flush_events)
    s1.record()
    barrier()
    t_wall1 = time.time()
    launches = G.gear_kernel_launches() - launches0
    clocks = sampler.stop(t_wall0, t_wall1) if sampler else None
    ms_total = max_over_ranks(s0.elapsed_time(s1), dist, dev)
    status = [G.gear_last_device_status(c) for c in caches]
    if any(status):
        raise SystemExit(f"device status word set: {status} ({w.name})")
    if not all(torch.isfinite(o).all().item() for o in outs):
        raise SystemExit(f"non-finite attention output ({w.name})")

    dec_ms = [a.elapsed_time(b) for a, b in events]       # one entry per group of L back-to-back decode launches
    flush_ms = [a.elapsed_time(b) for a, b in flush_events]
    res = {"ms_total": ms_total, "n_calls": steps * nb * L, "dec_ms": sum(dec_ms), "dec_launches": len(dec_ms) * L,
           "dec_bytes": float(sum(bytes_log)), "flush_ms": flush_ms, "compress_ms": compress_ms,
           "prefill_out_bytes": prefill_out_bytes, "launches": int(launches), "clocks": clocks}

    # ---- end to end through the host-buffer entry points (pinned host memory, copies inside the timed region)
    if e2e_steps > 0:
        hk = torch.empty((n_tok, *tok_shape), dtype=torch.float16).pin_memory().copy_(new_k.cpu())
        hv = torch.empty((n_tok, *tok_shape), dtype=torch.float16).pin_memory().copy_(new_v.cpu())
        hq = torch.empty((B, w.n_q_heads, 128), dtype=torch.float16).pin_memory().copy_(q.cpu())
        hout = torch.empty((L, B, w.n_q_heads, 128), dtype=torch.float32).pin_memory()
        hk_np, hv_np, hq_np, hout_np = hk.numpy(), hv.numpy(), hq.numpy(), hout.numpy()

        def step_e2e():
            # one model step per token: every layer's rows and query go up, every layer's attention output comes
            # back, and the host waits once, for the last of them
            for i in range(nb):
                for li, c in enumerate(caches):
                    G.gear_step_host(c, hk_np[i % n_tok], hv_np[i % n_tok], hq_np, hout_np[li])
                for c in caches:
                    G.gear_cache_wait(c)
        step_e2e()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            step_e2e()
        barrier()
        e2e_s = max_over_ranks(max(time.perf_counter() - t0, 1e-9), dist, dev)
        res["e2e_value"] = whole_job_tokens_per_s(world, B, e2e_steps * nb * L, e2e_s)
        res["h2d"] = nb * L * (2 * hk_np[0].nbytes + hq_np.nbytes)
        res["d2h"] = nb * hout_np.nbytes
    for c in caches:
        G.gear_free(c)
    G.gear_release_workspace()
    torch.cuda.empty_cache()
    return res


def decode_roofline(w, res, peak, peak_src):
    achieved = res["dec_bytes"] / (res["dec_ms"] * 1e-3) / 1e9
    per_launch = res["dec_bytes"] / res["dec_launches"]
    ratio = DECODE_DRAM_BYTES_PER_ALGORITHMIC_BYTE.get(w.config_id)
    return {"bound": "hbm", "kernel": "gear_decode_kernel", "achieved": achieved, "peak": peak,
            "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak, "frac_of_8000_nominal": achieved / 8000.0,
            "traffic": ratio * per_launch if ratio else None,
            "traffic_source": "ncu capture of one launch on one layer cache, scaled by the algorithmic bytes" if ratio else None,
            "algorithmic_bytes_per_launch": per_launch, "us_per_launch": 1e3 * res["dec_ms"] / res["dec_launches"]}


def compress_roofline(w, res, peak):
    """Prefill: fp16 K and V in, the packed segment out.  Flush: one full buffer of every (batch, head) in, its segment
    out.  Both against the HBM peak: what they must move is small next to what the kernels do per byte."""
    B, H, nb = w.batch, w.n_kv_heads, w.buffer_cap
    in_bytes = 2 * B * H * w.n * 128 * 2
    pre_ms = statistics.median(res["compress_ms"])
    pre_alg = in_bytes + res["prefill_out_bytes"]
    out = {"prefill": {"bound": "hbm", "kernel": "Filter/Quant kernel of the group shape (quant_fast*_kernel, quant_pack_kernel, kcvt_*) + pi_pass_kernel (dominant)", "ms": pre_ms,
                       "input_gbs": in_bytes / (pre_ms * 1e-3) / 1e9, "algorithmic_bytes": pre_alg,
                       "achieved": pre_alg / (pre_ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                       "frac": pre_alg / (pre_ms * 1e-3) / 1e9 / peak}}
    if res["flush_ms"]:
        f_ms = statistics.median(res["flush_ms"])
        f_in = 2 * B * H * nb * 128 * 2
        f_alg = f_in + res["prefill_out_bytes"] * nb // w.n
        out["flush"] = {"bound": "latency (one launch, less than one wave of tiles)", "kernel": "compress_tile_kernel",
                        "us": 1e3 * f_ms, "input_gbs": f_in / (f_ms * 1e-3) / 1e9, "algorithmic_bytes": f_alg,
                        "achieved": f_alg / (f_ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                        "frac": f_alg / (f_ms * 1e-3) / 1e9 / peak}
    return out


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

    res = measure_config(torch, G, dev, w, args.layers, args.steps, args.warmup, rank, args.e2e_steps, dist, world,
                         sampler_index=local if rank == 0 else None)
    value = whole_job_tokens_per_s(world, w.batch, res["n_calls"], res["ms_total"] * 1e-3)

    line = None
    if rank == 0:
        peak, peak_src = hbm_peak()
        roof = decode_roofline(w, res, peak, peak_src)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": res["ms_total"] / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "s32 (codes x fixed-point query on the integer tensor cores), f32 elsewhere",
                "data": "synthetic",
                "config": {"workload": workload_name(w, args.layers), "batch_per_gpu": w.batch, "layers_rotated": args.layers,
                           "l2": "rotating caches: %.0f MB touched between reuses" % (roof["algorithmic_bytes_per_launch"] * args.layers / 1e6)},
                "roofline": roof,
                "e2e": {"value": res.get("e2e_value"), "unit": UNIT, "h2d_bytes_per_step": res.get("h2d"),
                        "d2h_bytes_per_step": res.get("d2h")},
                "gpu_launches": res["launches"],
                "clocks": res["clocks"],
                "compress": compress_roofline(w, res, peak),
                "decode_attn_tokens_per_s_kernel_only": w.batch / (1e-3 * res["dec_ms"] / res["dec_launches"])}
    # ---- the other configurations, a few steps each (rank 0's GPU at N = 1 only: they are context, not the headline)
    if rank == 0 and world == 1 and not args.no_extra and w.config_id == 2:
        extra = {}
        for cid in EXTRA_CONFIGS:
            we = synth.WORKLOADS[cid]
            r = measure_config(torch, G, dev, we, 2, 1, 3, rank)
            extra[f"C{cid}"] = {"workload": workload_name(we, 2), "steps": 1, "warmup": 3,
                                "decode_attn_tokens_per_s_kernel_only": we.batch / (1e-3 * r["dec_ms"] / r["dec_launches"]),
                                "roofline": decode_roofline(we, r, peak, peak_src),
                                "compress": compress_roofline(we, r, peak)}
        line["extra"] = extra
    if rank == 0 and not args.no_cpu and world == 1:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            t0 = time.perf_counter()
            per = [oracle_unit_cycle(w, 100 + s, n_decode=8) for s in range(args.cpu_units)]
            spent = time.perf_counter() - t0
        units = w.batch * w.n_kv_heads
        line["cpu_baseline"] = {"value": w.batch / (statistics.mean(per) * units), "unit": UNIT, "cores": 1,
                                "kind": "oracle",
                                "sample": f"{args.cpu_units} of {units} (batch, head) units, one buffer cycle each "
                                          f"({w.buffer_cap} pushes incl. the flush, 8 decode-attention calls timed), scaled by "
                                          f"the unit count; {spent:.1f} s of CPU work incl. the untimed prefill compress"}
        v_all, cores, n_units, wall = oracle_all_cores(w)
        line["cpu_baseline_all_cores"] = {"value": v_all, "unit": UNIT, "cores": cores, "kind": "oracle",
                                          "sample": f"{n_units} of {units} units over a pool of {cores} one-thread workers "
                                                    f"(4 decode-attention calls timed per unit), scaled by the unit count; "
                                                    f"{wall:.1f} s wall"}
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
    ap.add_argument("--no-extra", action="store_true")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.config]
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) == 0:
            run_reference(args, w)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args.gpus, sys.argv)                  # no launcher: start the ranks here, one GPU each
        return
    run_ours(args, w)


if __name__ == "__main__":
    main()
