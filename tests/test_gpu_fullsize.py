"""Parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times.

The whole layer is compressed and attended on the GPU; the float64 oracle then recomputes a few sampled
(batch, kv head) units one by one from the very same inputs (pulled back from the device), and every piece of
those units is compared: codes, scales, zero-points, outlier sets and values bit-exact; low-rank reconstruction
and attention output within 1e-3 max-norm relative.  Units are independent, so a sampled unit checks the same
code path as all the others of the launch."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = 1e-3


def _rel_max(a, b):
    den = np.abs(b).max()
    return np.abs(a - b).max() / (den if den > 0 else 1.0)


def _device_inputs(torch, w, dev, seed, n_app):
    """Same distribution as synth.make_kv, drawn on the device (per-channel lognormal key scales, 1 % spikes x 20)."""
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    shape = (w.batch, w.n_kv_heads, w.n, 128)
    c = torch.exp(torch.randn(w.n_kv_heads, 128, generator=g, device=dev))[None, :, None, :]
    k = torch.randn(shape, generator=g, device=dev) * c
    k = torch.where(torch.rand(shape, generator=g, device=dev) < 0.01, k * 20.0, k).half().contiguous()
    v = torch.randn(shape, generator=g, device=dev)
    v = torch.where(torch.rand(shape, generator=g, device=dev) < 0.01, v * 20.0, v).half().contiguous()
    b0 = torch.randn((w.batch, w.n_kv_heads, 2, 128, w.rank), generator=g, device=dev)
    b0f = torch.randn((w.batch, w.n_kv_heads, 2, 128, w.rank), generator=g, device=dev)
    ks = (torch.randn((n_app, w.batch, w.n_kv_heads, 128), generator=g, device=dev) * c[:, :, 0, :]).half().contiguous()
    vs = torch.randn((n_app, w.batch, w.n_kv_heads, 128), generator=g, device=dev).half().contiguous()
    q = torch.randn((w.batch, w.n_q_heads, 128), generator=g, device=dev).half().contiguous()
    return k, v, b0, b0f, ks, vs, q


@pytest.mark.parametrize("config_id,units", [(2, [(0, 0), (3, 17), (7, 31)]), (4, [(0, 0), (3, 7)]), (3, [(5, 11), (15, 39)]), (32, [(2, 3)]),
                                             (21, [(1, 30)]), (22, [(0, 5), (3, 31)]), (6, [(0, 0), (6, 29)])])
def test_full_size_layer_sampled_units_match_the_oracle(config_id, units):
    import torch
    from oracle import gear_oracle as O
    from paper_2403_05527_b200 import binding as G, synth

    w = synth.WORKLOADS[config_id]
    dev = torch.device("cuda:0")
    n_app = w.buffer_cap + w.buffer_cap // 2 + 5          # one flush and a ragged buffer
    k, v, b0, b0f, ks, vs, q = _device_inputs(torch, w, dev, 4242 + config_id, n_app)
    cfg = G.make_config(w.batch, w.n_q_heads, w.n_kv_heads, w.bits, w.group, w.s_pct, w.buffer_cap, w.rank,
                        w.n + 4 * w.buffer_cap, rank_max=w.rank, power_iters=w.power_iters)
    cache = G.gear_compress(None, cfg, k, v, w.n, w.rank, b0)
    try:
        flushed = 0
        for i in range(n_app):
            flushed += G.gear_append_buffer(cache, ks[i], vs[i], b0f) == G.GEAR_FLUSHED
        assert flushed == 1
        out = torch.full((w.batch, w.n_q_heads, 128), float("nan"), dtype=torch.float32, device=dev)
        G.gear_decode_attn(cache, q, out)
        torch.cuda.synchronize()
        assert G.gear_last_device_status(cache) == 0
        out = out.cpu().numpy().astype(np.float64)
        assert np.isfinite(out).all()

        rep = w.n_q_heads // w.n_kv_heads
        exported = {}

        def ex(seg, what):
            if (seg, what) not in exported:
                exported[(seg, what)] = G.gear_export(cache, seg, what, w.batch, w.n_kv_heads)
            return exported[(seg, what)]

        for b, h in units:
            group = w.group if w.group else 1 << 30          # group 0: per-vector grouping
            ref = O.OracleCache(1, rep, 1, 128, w.bits, group, w.s_pct, w.buffer_cap, w.rank, w.power_iters)
            ref.compress(k[b:b + 1, h:h + 1].cpu().numpy(), v[b:b + 1, h:h + 1].cpu().numpy(), w.rank,
                         b0[b:b + 1, h:h + 1].cpu().numpy())
            for i in range(n_app):
                ref.append(ks[i, b, h].cpu().numpy(), vs[i, b, h].cpu().numpy(), b0f[b:b + 1, h:h + 1].cpu().numpy())
            for si, seg in enumerate(ref.segments):
                for side in ("K", "V"):
                    tile = seg[side][0][0]
                    assert np.array_equal(ex(si, f"{side}_CODES")[b, h], tile["codes"]), (side, si, "codes")
                    assert np.array_equal(ex(si, f"{side}_SCALE")[b, h].view(np.uint16), tile["scale"].view(np.uint16))
                    assert np.array_equal(ex(si, f"{side}_ZERO")[b, h].view(np.uint16), tile["zero"].view(np.uint16))
                    oi, ov = tile["out_idx"], tile["out_val"]
                    assert np.array_equal(ex(si, f"{side}_OUT_IDX")[b, h].reshape(oi.shape), oi), (side, si, "outlier sets")
                    assert np.array_equal(ex(si, f"{side}_OUT_VAL")[b, h].reshape(ov.shape).view(np.uint16), ov.view(np.uint16))
                    got = ex(si, f"{side}_A")[b, h].astype(np.float64) @ ex(si, f"{side}_B")[b, h].astype(np.float64).T
                    err = _rel_max(got, tile["A"] @ tile["B"].T)
                    assert err <= TOL, f"low-rank reconstruction {side} segment {si} unit {(b, h)}: {err:.2e}"
            want = ref.decode_attn(q[b:b + 1, h * rep:(h + 1) * rep].cpu().numpy())[0]
            for j in range(rep):
                err = _rel_max(out[b, h * rep + j], want[j])
                assert err <= TOL, f"attention unit {(b, h)} query head {j}: {err:.2e}"
    finally:
        G.gear_free(cache)
