"""The allocation-free fp16 attention entry point, through the C ABI.

gear_fp16_decode_attn_static exists for callers that may not allocate device memory (a plug-in inside a
framework that owns the device heap, a loop that cannot afford an allocation): it keeps its bookkeeping in an
array built into the library instead of a caller-supplied scratch buffer.  It must give the same attention output
as gear_fp16_decode_attn, also when it is called again on the array the previous call left behind, and it must
refuse problems that do not fit the array instead of launching.  Both entry points are also held against the
textbook softmax(q K^T / sqrt(d_H)) V in float64 (Eq. 1), so that a fault they share cannot hide.

This file sorts last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = 1e-3      # max-norm relative tolerance, the one the other attention tests use


def _rel_max(a, b):
    return np.abs(a - b).max() / np.abs(b).max()


def _textbook(k16, v16, q, n, rep):
    """Eq. 1 in float64 on the fp16 inputs: [B, Hq, d_H]."""
    B, Hq = q.shape[:2]
    out = np.zeros((B, Hq, 128))
    for b in range(B):
        for h in range(Hq):
            kk, vv = k16[b, h // rep, :n].astype(np.float64), v16[b, h // rep, :n].astype(np.float64)
            z = kk @ q[b, h].astype(np.float64) / np.sqrt(128.0)
            w = np.exp(z - z.max())
            out[b, h] = (w / w.sum()) @ vv
    return out


def test_static_scratch_attention_matches_the_caller_scratch_one_twice_in_a_row():
    import torch
    from paper_2403_05527_b200 import binding as G, synth

    dev = torch.device("cuda:0")
    # different problems back to back: every call after the first starts from the previous call's leftovers
    # (grouped queries; one query head per kv head; the largest problem the array takes: 256 query heads; nine query
    # heads per kv head, i.e. two passes of the kernel)
    cases = [(2, 8, 2, 333, 400, 0), (1, 4, 4, 1500, 1500, 1), (8, 32, 32, 150, 160, 2), (2, 9, 1, 77, 80, 3)]
    for B, Hq, Hkv, n, n_alloc, extra in cases:
        k16, v16 = synth.make_kv(2, B, Hkv, n_alloc, 128, extra=extra)
        q = synth.make_query(2, B, Hq, 128, extra=extra)
        kd, vd, qd = (torch.from_numpy(x).to(dev) for x in (k16, v16, q))
        scratch = torch.empty(G.gear_fp16_attn_scratch_bytes(B, Hq), dtype=torch.uint8, device=dev)
        want = torch.empty(B, Hq, 128, dtype=torch.float32, device=dev)
        G.gear_fp16_decode_attn(kd, vd, qd, want, B, Hq, Hkv, n, n_alloc, scratch)
        torch.cuda.synchronize()
        want = want.cpu().numpy().astype(np.float64)
        exact = _textbook(k16, v16, q, n, Hq // Hkv)
        for b in range(B):
            for h in range(Hq):
                assert _rel_max(want[b, h], exact[b, h]) <= TOL, f"caller-scratch call vs float64, batch {b}, head {h}"
        for call in range(2):
            got = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device=dev)
            G.gear_fp16_decode_attn_static(kd, vd, qd, got, B, Hq, Hkv, n, n_alloc)
            torch.cuda.synchronize()
            got = got.cpu().numpy().astype(np.float64)
            assert np.isfinite(got).all()
            for b in range(B):
                for h in range(Hq):
                    err = _rel_max(got[b, h], want[b, h])
                    assert err <= TOL, f"call {call}, batch {b}, head {h}: {err:.2e}"
                    err = _rel_max(got[b, h], exact[b, h])
                    assert err <= TOL, f"call {call} vs float64, batch {b}, head {h}: {err:.2e}"


def test_static_scratch_attention_rejects_what_does_not_fit():
    import torch
    from paper_2403_05527_b200 import binding as G

    dev = torch.device("cuda:0")
    B, Hq = 9, 32                                   # 288 query heads: beyond GEAR_STATIC_MAX_QUERY_HEADS = 256
    kv = torch.zeros(B, Hq, 16, 128, dtype=torch.float16, device=dev)
    q = torch.zeros(B, Hq, 128, dtype=torch.float16, device=dev)
    out = torch.zeros(B, Hq, 128, dtype=torch.float32, device=dev)
    with pytest.raises(G.GearError) as e:
        G.gear_fp16_decode_attn_static(kv, kv, q, out, B, Hq, Hq, 16, 16)
    assert e.value.status == G.GEAR_ERR_CAPACITY
    torch.cuda.synchronize()
