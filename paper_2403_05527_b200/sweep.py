"""Batch sweep of one decode step over a multi-layer compressed cache, next to an FP16 cache.

For a LLaMA-2-7B-shaped model (32 layers, 32 heads, d_H = 128, context 4096, 2-bit codes, group 64, s = 2 %,
rank 4, n_b = 64) one decode step runs gear_decode_attn once per layer.  All layers of a real model hold
different data; here `--resident` distinct layer caches are built (enough to exceed the L2) and the 32 calls of
a step rotate over them, so every call streams its cache from HBM.  The FP16 reference point is
gear_fp16_decode_attn on an fp16 cache of the same shape.

    python -m paper_2403_05527_b200.sweep [--batches 1,2,4,...] [--layers 32] [--context 4096]

Prints one JSON line per batch size: latency of a step (all layers), tokens/s, achieved GB/s on the bytes read,
for the compressed cache and for the FP16 cache, and the bytes both caches would occupy over all layers.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as G


def _kv(shape, n_heads, dev, seed):
    """K, V fp16 of `shape` = (B, H, n, 128), drawn in slices of 16 sequences so that the fp32 temporaries stay small."""
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    c = torch.exp(torch.randn(n_heads, 128, generator=g, device=dev))[None, :, None, :]
    k = torch.empty(shape, dtype=torch.float16, device=dev)
    v = torch.empty(shape, dtype=torch.float16, device=dev)
    for b0 in range(0, shape[0], 16):
        part = (min(16, shape[0] - b0), *shape[1:])
        x = torch.randn(part, generator=g, device=dev) * c
        k[b0:b0 + part[0]] = torch.where(torch.rand(part, generator=g, device=dev) < 0.01, x * 20.0, x).half()
        x = torch.randn(part, generator=g, device=dev)
        v[b0:b0 + part[0]] = torch.where(torch.rand(part, generator=g, device=dev) < 0.01, x * 20.0, x).half()
        del x
    return k, v


def _time(fn, reps):
    fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e-3 / reps


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batches", default="1,2,4,8,16,32,64,128,256")
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--heads", type=int, default=32)
    ap.add_argument("--context", type=int, default=4096)
    ap.add_argument("--bits", type=int, default=2)
    ap.add_argument("--group", type=int, default=64)
    ap.add_argument("--s-pct", type=float, default=2.0)
    ap.add_argument("--rank", type=int, default=4)
    ap.add_argument("--buffer", type=int, default=64)
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--fp16-max-batch", type=int, default=64)
    ap.add_argument("--state", default="s1", choices=["s1", "s2"],
                    help="s1: one prefill segment of `context` tokens + half a buffer; "
                         "s2: prefill of context/2 tokens, then context/2 tokens pushed one by one "
                         "(context/2/buffer flushed segments) + half a buffer")
    args = ap.parse_args()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    H, n, L = args.heads, args.context, args.layers
    for B in [int(x) for x in args.batches.split(",")]:
        cfg = G.make_config(B, H, H, args.bits, args.group, args.s_pct, args.buffer, args.rank, n + 2 * args.buffer,
                            rank_max=args.rank, seed=B)
        n_pre = n if args.state == "s1" else n // 2
        n_push = args.buffer // 2 + (0 if args.state == "s1" else n - n_pre)
        shape = (B, H, n_pre, 128)
        toks = torch.randn(16, B, H, 128, device=dev).half()

        def build(seed):
            k, v = _kv(shape, H, dev, seed)
            c = G.gear_compress(None, cfg, k, v, n_pre, args.rank, None)
            del k, v
            for i in range(n_push):
                G.gear_append_buffer(c, toks[i % 16], toks[(i + 5) % 16])
            return c
        probe = build(100 + B)
        by = G.gear_cache_bytes(probe)
        read = by.codes + by.scale_zero + by.outliers + by.lowrank_a + by.lowrank_b + by.buffer
        # distinct resident caches: enough that a step's working set is well beyond the 126 MB L2
        resident = max(1, min(L, int(1.2e9 // max(read, 1)) + 1))
        caches = [probe]
        for i in range(1, resident):
            caches.append(build(100 + B + 1000 * i))
        q = torch.randn(B, H, 128, device=dev).half()
        out = torch.empty(B, H, 128, dtype=torch.float32, device=dev)

        def step():
            for layer in range(L):
                G.gear_decode_attn(caches[layer % resident], q, out)
        t_gear = _time(step, args.reps)
        line = {"batch": B, "layers": L, "context": n, "state": args.state, "resident_caches": resident,
                "gear": {"step_ms": t_gear * 1e3, "tokens_per_s": B / t_gear, "gbs": L * read / t_gear / 1e9,
                         "cache_gb_all_layers": L * by.stored_total / 1e9}}
        fp16_bytes = 2 * B * H * (n + args.buffer // 2) * 128 * 2
        line["fp16"] = {"cache_gb_all_layers": L * fp16_bytes / 1e9}
        if B <= args.fp16_max_batch:
            nres = max(1, min(L, int(1.2e9 // fp16_bytes) + 1))
            n_tok = n + args.buffer // 2
            fk = [torch.empty((B, H, n_tok, 128), dtype=torch.float16, device=dev).normal_() for _ in range(nres)]
            fv = [torch.empty((B, H, n_tok, 128), dtype=torch.float16, device=dev).normal_() for _ in range(nres)]
            scratch = torch.empty(G.gear_fp16_attn_scratch_bytes(B, H), dtype=torch.uint8, device=dev)

            def step16():
                for layer in range(L):
                    G.gear_fp16_decode_attn(fk[layer % nres], fv[layer % nres], q, out, B, H, H, n_tok, n_tok, scratch)
            t16 = _time(step16, args.reps)
            line["fp16"].update({"step_ms": t16 * 1e3, "tokens_per_s": B / t16, "gbs": L * fp16_bytes / t16 / 1e9,
                                 "resident_caches": nres})
            line["speedup_vs_fp16"] = t16 / t_gear
            del fk, fv, scratch
        print(json.dumps(line), flush=True)
        for c in caches:
            G.gear_free(c)
        G.gear_release_workspace()
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
