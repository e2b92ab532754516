"""The method's variants that are parameter choices of the same path, and several query rows per head.

* GEAR-L (quantization + low rank, s = 0) and outlier-aware quantization only (r = 0): Section 3 and the ablations of
  Section 4.3.
* Error reduction on the prefill tokens only ("GEAR-L Prefill", Section 4.3): rank r_p for the prefill segment, rank 0
  for every flushed buffer; and the ranks of Section 4 "Implementation details": r_p = 4 for the prefill segment,
  r_g = 2 for the flushed buffers.
* gear_decode_attn_multi: n query rows per head against the same cache (Eq. 1 row by row, no mask among the rows).
  With dozens of rows per kv head on a cache of a few hundred tokens, the fp16 rounding of the stored factors A and B
  (kept in fp16 as the paper keeps them) alone moves single rows by up to 1.1e-3 from the oracle's float64 factors --
  measured: 5e-4 from either factor -- while the kernel's own arithmetic stays below 4e-5.  The rows are therefore
  held to 1e-3 against the oracle evaluated on the factors as stored (exported from the cache; every other piece is
  bit-identical on both sides), and to 2e-3 against the oracle's own factors.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,s_pct,r_prefill,r_flush", [("gear_l", 0.0, 4, 4), ("prefill_only_low_rank", 2.0, 4, 0),
                                                          ("paper_ranks_4_and_2", 2.0, 4, 2), ("gear_l_prefill", 0.0, 4, 0)])
def test_variants_of_the_recipe_match_the_oracle(name, s_pct, r_prefill, r_flush):
    from tests.gear_harness import Pair
    p = Pair(14, 2, 4, 2, 2, 64, s_pct, 64, r_flush, 1024, r_max=max(r_prefill, r_flush))
    try:
        p.compress(256, r_prefill)
        p.check_segment(0)
        assert p.append(64 + 64 + 9) == 2
        p.check_segment(1)
        p.check_segment(2)
        p.check_attention()
        from paper_2403_05527_b200 import binding as G
        assert [G.gear_segment_info_get(p.cache, i).rank for i in range(3)] == [r_prefill, r_flush, r_flush]
    finally:
        p.close()


@pytest.mark.parametrize("hq,hkv,nq,bits,group", [(2, 2, 4, 2, 64), (2, 2, 16, 4, 64), (8, 2, 3, 2, 128), (4, 4, 1, 2, 64)])
def test_several_query_rows_per_head(hq, hkv, nq, bits, group):
    import torch
    from oracle import gear_oracle as O
    from paper_2403_05527_b200 import binding as G, synth

    B, n, nb, rank = 2, 256, 64, 4
    k16, v16 = synth.make_kv(15, B, hkv, n, 128)
    b0 = synth.make_b0(15, B, hkv, 128, rank)
    ks, vs = synth.make_appended(15, B, hkv, 128, nb + 11)
    dev = torch.device("cuda:0")
    cfg = G.make_config(B, hq, hkv, bits, group, 2.0, nb, rank, 1024, rank_max=rank, max_queries=16)
    cache = G.gear_compress(None, cfg, torch.from_numpy(k16).to(dev), torch.from_numpy(v16).to(dev), n, rank,
                            torch.from_numpy(b0).to(dev))
    try:
        # the oracle sees the rows as hq * nq query heads: rows of one kv head are consecutive either way
        ref = O.OracleCache(B, hq * nq, hkv, 128, bits, group, 2.0, nb, rank, 3)
        ref.compress(k16, v16, rank, b0)
        for i in range(nb + 11):
            fb0 = synth.make_b0(15, B, hkv, 128, rank, extra=100 + i)
            ref.append(ks[i], vs[i], fb0)
            G.gear_append_buffer(cache, torch.from_numpy(ks[i]).to(dev), torch.from_numpy(vs[i]).to(dev),
                                 torch.from_numpy(fb0).to(dev))
        q = synth.make_query(15, B, hq * nq, 128).reshape(B, hq, nq, 128)
        out = torch.full((B, hq, nq, 128), float("nan"), dtype=torch.float32, device=dev)
        G.gear_decode_attn_multi(cache, torch.from_numpy(q).to(dev), out, nq)
        torch.cuda.synchronize()
        assert G.gear_last_device_status(cache) == 0
        got = out.cpu().numpy().astype(np.float64).reshape(B, hq * nq, 128)
        want = ref.decode_attn(q.reshape(B, hq * nq, 128))
        import copy
        stored = copy.deepcopy(ref)                      # the oracle's cache with the library's fp16 factors in place
        for si, seg in enumerate(stored.segments):
            for side in ("K", "V"):
                a = G.gear_export(cache, si, f"{side}_A", B, hkv).astype(np.float64)
                bm = G.gear_export(cache, si, f"{side}_B", B, hkv).astype(np.float64)
                for b in range(B):
                    for h in range(hkv):
                        ref_ab = seg[side][b][h]["A"] @ seg[side][b][h]["B"].T
                        assert np.abs(a[b, h] @ bm[b, h].T - ref_ab).max() <= 1e-3 * np.abs(ref_ab).max()
                        seg[side][b][h]["A"], seg[side][b][h]["B"] = a[b, h], bm[b, h]
        want_stored = stored.decode_attn(q.reshape(B, hq * nq, 128))
        for b in range(B):
            for h in range(hq * nq):
                err = np.abs(got[b, h] - want_stored[b, h]).max() / np.abs(want_stored[b, h]).max()
                assert err <= 1e-3, f"batch {b} row {h} against the oracle on the stored factors: {err:.2e}"
                err = np.abs(got[b, h] - want[b, h]).max() / np.abs(want[b, h]).max()
                assert err <= 2e-3, f"batch {b} row {h}: {err:.2e}"
        # the one-row call still works on the same cache, and more rows than the cache was sized for are refused
        q1 = synth.make_query(15, B, hq, 128, extra=5)
        out1 = torch.empty((B, hq, 128), dtype=torch.float32, device=dev)
        G.gear_decode_attn(cache, torch.from_numpy(q1).to(dev), out1)
        torch.cuda.synchronize()
        ref1 = O.OracleCache(B, hq, hkv, 128, bits, group, 2.0, nb, rank, 3)
        ref1.segments, ref1.buf_k, ref1.buf_v = ref.segments, ref.buf_k, ref.buf_v
        want1 = ref1.decode_attn(q1)
        assert np.abs(out1.cpu().numpy() - want1).max() / np.abs(want1).max() <= 1e-3
        with pytest.raises(G.GearError) as e:
            big = torch.zeros((B, hq, 17, 128), dtype=torch.float16, device=dev)
            G.gear_decode_attn_multi(cache, big, torch.zeros((B, hq, 17, 128), dtype=torch.float32, device=dev), 17)
        assert e.value.status == G.GEAR_ERR_ARG
    finally:
        G.gear_free(cache)


def test_groups_of_128_with_ties_and_constant_groups():
    """g = 128, s = 2 %: two entries per side leave every group.  Entries drawn from five values put the thresholds of
    Filter_s inside runs of equal entries (ties go to the lower index); constant groups make the smallest entries the
    ones right after the largest.  Codes, scales and outlier sets must still match the oracle bit for bit."""
    import torch
    from tests.gear_harness import Pair
    from paper_2403_05527_b200 import binding as G
    B, H, n = 1, 2, 256
    rng = np.random.default_rng(19)
    vals = np.array([-1.5, -0.25, 0.0, 0.25, 2.0], np.float16)
    k16 = rng.choice(vals, size=(B, H, n, 128))
    v16 = rng.choice(vals, size=(B, H, n, 128))
    k16[:, :, :, 7] = np.float16(0.5)              # a constant key channel
    k16[:, :, 5, 8] = np.float16(3.0)              # one entry above a sea of ties
    v16[:, :, 3, :] = np.float16(-0.75)            # a constant value row
    v16[:, :, 9, :] = np.float16(1.0); v16[:, :, 9, 100] = np.float16(-4.0)
    k16[:, :, 130:140, :] = (rng.standard_normal((B, H, 10, 128)) * 3).astype(np.float16)    # and ordinary entries
    p = Pair(4, B, H, H, 2, 128, 2.0, 64, 0, n + 64, r_max=0)
    try:
        p.oracle.compress(k16, v16, 0, None)
        G.gear_compress(p.cache, None, torch.from_numpy(k16).to(p.dev), torch.from_numpy(v16).to(p.dev), n, 0, None)
        torch.cuda.synchronize()
        si = G.gear_segment_info_get(p.cache, 0)
        assert (si.g_k, si.k_k, si.g_v, si.k_v) == (128, 2, 128, 2)
        p.check_segment(0)
        p.check_attention()
    finally:
        p.close()


@pytest.mark.parametrize("rank", [3, 6, 12, 16])
def test_ranks_of_a_long_segment(rank):
    """Long segments run the power iteration as streaming passes: four rank columns per CTA (ranks up to 4), eight
    (5..8, with the first Gram matrix summed inside the last pass), two such CTAs per chunk above that."""
    from tests.gear_harness import Pair
    p = Pair(6, 1, 2, 2, 4, 64, 2.0, 64, 2, 512 + 128, r_max=16)
    try:
        p.compress(512, rank)
        p.check_segment(0)
        p.check_attention()
    finally:
        p.close()
