"""Shared helpers of the GPU parity tests: run the same seeded inputs through the CPU oracle and through the
CUDA library (C ABI), and compare piece by piece."""
from __future__ import annotations

import numpy as np

from oracle import gear_oracle as O
from paper_2403_05527_b200 import binding as G
from paper_2403_05527_b200 import synth

TOL = 1e-3   # max-norm relative tolerance on low-rank reconstructions and attention outputs


def rel_max(a, b):
    den = np.abs(b).max()
    return np.abs(a - b).max() / (den if den > 0 else 1.0)


class Pair:
    """An oracle cache and a GPU cache fed with identical inputs."""

    def __init__(self, config_id, batch, hq, hkv, bits, group, s, nb, r_flush, max_tokens, r_max=None, iters=3,
                 keep_fp32=True):
        import torch
        self.torch = torch
        self.dev = torch.device("cuda:0")
        self.cid, self.B, self.Hq, self.Hkv = config_id, batch, hq, hkv
        self.r_flush = r_flush
        # group 0: per-vector grouping -- for the oracle, a group length no vector reaches
        self.oracle = O.OracleCache(batch, hq, hkv, 128, bits, group if group else 1 << 30, s, nb, r_flush, iters)
        flags = G.GEAR_FLAG_KEEP_FP32_FACTORS if keep_fp32 else 0
        self.cfg = G.make_config(batch, hq, hkv, bits, group, s, nb, r_flush, max_tokens,
                                 rank_max=r_max if r_max is not None else max(r_flush, 0), power_iters=iters, flags=flags)
        self.cache = G.gear_create(self.cfg)
        self.n_app = 0

    def close(self):
        G.gear_free(self.cache)
        self.cache = None

    def compress(self, n, rank, extra=0):
        t = self.torch
        k16, v16 = synth.make_kv(self.cid, self.B, self.Hkv, n, 128, extra=extra)
        b0 = synth.make_b0(self.cid, self.B, self.Hkv, 128, rank, extra=extra)
        self.oracle.compress(k16, v16, rank, b0)
        kd, vd = t.from_numpy(k16).to(self.dev), t.from_numpy(v16).to(self.dev)
        b0d = t.from_numpy(np.ascontiguousarray(b0)).to(self.dev) if rank > 0 else None
        G.gear_compress(self.cache, None, kd, vd, n, rank, b0d)
        t.cuda.synchronize()

    def append(self, steps):
        t = self.torch
        ks, vs = synth.make_appended(self.cid, self.B, self.Hkv, 128, self.n_app + steps)
        flushed = 0
        for i in range(self.n_app, self.n_app + steps):
            b0 = synth.make_b0(self.cid, self.B, self.Hkv, 128, self.r_flush, extra=5000 + i)
            fo = self.oracle.append(ks[i], vs[i], b0)
            b0d = t.from_numpy(np.ascontiguousarray(b0)).to(self.dev) if self.r_flush > 0 else None
            fg = G.gear_append_buffer(self.cache, t.from_numpy(ks[i]).to(self.dev), t.from_numpy(vs[i]).to(self.dev), b0d)
            assert (fg == G.GEAR_FLUSHED) == fo
            flushed += int(fo)
        t.cuda.synchronize()
        self.n_app += steps
        return flushed

    # ---------------------------------------------------------------- comparisons
    def check_segment(self, si, tol=TOL):
        B, H = self.B, self.Hkv
        seg = self.oracle.segments[si]
        ex = lambda what: G.gear_export(self.cache, si, what, B, H)
        for side in ("K", "V"):
            tiles = seg[side]
            stack = lambda key: np.stack([np.stack([tiles[b][h][key] for h in range(H)]) for b in range(B)])
            assert np.array_equal(ex(f"{side}_CODES"), stack("codes")), f"{side} codes differ in segment {si}"
            assert np.array_equal(ex(f"{side}_SCALE").view(np.uint16), stack("scale").view(np.uint16)), f"{side} scale"
            assert np.array_equal(ex(f"{side}_ZERO").view(np.uint16), stack("zero").view(np.uint16)), f"{side} zero"
            k2 = tiles[0][0]["out_idx"].shape[1]
            if k2:
                gi, gv = ex(f"{side}_OUT_IDX"), ex(f"{side}_OUT_VAL")
                oi, ov = stack("out_idx"), stack("out_val")
                assert np.array_equal(gi.reshape(oi.shape), oi), f"{side} outlier index sets"
                assert np.array_equal(gv.reshape(ov.shape).view(np.uint16), ov.view(np.uint16)), f"{side} outlier values"
            if seg["rank"]:
                for suffix in ("", "_FP32"):
                    a, bm = ex(f"{side}_A{suffix}").astype(np.float64), ex(f"{side}_B{suffix}").astype(np.float64)
                    for b in range(B):
                        for h in range(H):
                            ref = tiles[b][h]["A"] @ tiles[b][h]["B"].T
                            got = a[b, h] @ bm[b, h].T
                            err = rel_max(got, ref)
                            assert err <= tol, f"{side} low-rank reconstruction seg {si} b{b} h{h}{suffix}: {err:.2e}"

    def check_attention(self, extra=0, tol=TOL, scale=0.0):
        t = self.torch
        q = synth.make_query(self.cid, self.B, self.Hq, 128, extra=extra)
        ref = self.oracle.decode_attn(q, scale if scale > 0 else None)
        out = t.full((self.B, self.Hq, 128), float("nan"), dtype=t.float32, device=self.dev)
        G.gear_decode_attn(self.cache, t.from_numpy(q).to(self.dev), out, scale)
        t.cuda.synchronize()
        assert G.gear_last_device_status(self.cache) == 0
        got = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        worst = 0.0
        for b in range(self.B):
            for h in range(self.Hq):
                worst = max(worst, rel_max(got[b, h], ref[b, h]))
        assert worst <= tol, f"attention max relative error {worst:.2e}"
        return worst, got
