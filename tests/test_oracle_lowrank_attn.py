"""Pins for the oracle's SVDSolver (Algorithm 2), cache (Algorithm 1) and decode attention (Eq. 1)."""
import numpy as np
import pytest

from oracle import gear_oracle as O
from paper_2403_05527_b200 import synth


def orth(m):
    """Orthonormal basis of range(m) by an SVD (independent of the oracle's QR route)."""
    u, s, _ = np.linalg.svd(m, full_matrices=False)
    return u[:, s > s[0] * 1e-13]


def make_residual(n_c=64, d=128, seed=0, decay=0.7):
    gen = np.random.default_rng(seed)
    u, _ = np.linalg.qr(gen.standard_normal((n_c, min(n_c, d))))
    v, _ = np.linalg.qr(gen.standard_normal((d, min(n_c, d))))
    s = decay ** np.arange(min(n_c, d))
    return (u * s) @ v.T


@pytest.mark.parametrize("rank,iters", [(1, 1), (2, 3), (4, 3), (8, 2), (4, 1)])
def test_projection_structure(rank, iters):
    r = make_residual(96, 128, seed=rank)
    b0 = np.random.default_rng(1).standard_normal((128, rank))
    a, b = O.svd_solver(r, b0, rank, iters)
    assert a.shape == (96, rank) and b.shape == (128, rank)
    assert np.allclose(a.T @ a, np.eye(rank), atol=1e-12)           # A orthonormal
    assert np.allclose(b, r.T @ a, atol=1e-12)                      # B = R^T A
    lr = a @ b.T
    assert np.allclose(lr, a @ a.T @ r, atol=1e-12)                 # A B^T is an orthogonal projection of R
    lhs = np.linalg.norm(r - lr) ** 2
    assert np.isclose(lhs, np.linalg.norm(r) ** 2 - np.linalg.norm(b) ** 2, rtol=1e-10)


@pytest.mark.parametrize("rank,iters", [(2, 1), (3, 2), (4, 3), (2, 4)])
def test_closed_form_subspace(rank, iters):
    """A B^T = P R with P the projector on range(R (R^T R)^(L-1) B0)."""
    r = make_residual(48, 32, seed=3 + rank, decay=0.8)
    b0 = np.random.default_rng(7).standard_normal((32, rank))
    a, b = O.svd_solver(r, b0, rank, iters)
    m = r @ np.linalg.matrix_power(r.T @ r, iters - 1) @ b0
    q = orth(m)
    assert q.shape[1] == rank
    assert np.allclose(a @ b.T, q @ q.T @ r, atol=1e-9)


def test_full_rank_and_exact_low_rank_recovery():
    gen = np.random.default_rng(2)
    r = gen.standard_normal((40, 16))
    a, b = O.svd_solver(r, gen.standard_normal((16, 16)), 16, 3)     # r = d_H <= n_c
    assert np.allclose(a @ b.T, r, atol=1e-10)
    low = gen.standard_normal((50, 3)) @ gen.standard_normal((3, 24))
    a, b = O.svd_solver(low, gen.standard_normal((24, 3)), 3, 1)     # exactly rank r, one loop
    assert np.allclose(a @ b.T, low, atol=1e-10)
    a, b = O.svd_solver(low, gen.standard_normal((24, 3)), 0, 3)
    assert a.shape == (50, 0) and b.shape == (24, 0)
    with pytest.raises(ValueError):
        O.svd_solver(low, gen.standard_normal((24, 30)), 30, 3)


def test_eckart_young_bound_and_convergence():
    r = make_residual(40, 24, seed=5, decay=0.75)
    sv = np.linalg.svd(r, compute_uv=False)
    rank = 3
    bound = np.sqrt(np.sum(sv[rank:] ** 2))
    b0 = np.random.default_rng(9).standard_normal((24, rank))
    gaps = []
    for iters in range(1, 7):
        a, b = O.svd_solver(r, b0, rank, iters)
        err = np.linalg.norm(r - a @ b.T)
        assert err >= bound * (1 - 1e-12)
        gaps.append(err - bound)
    assert gaps[-1] < 0.05 * gaps[0]
    assert gaps[2] < gaps[0]


def test_b0_columns_beyond_rank_are_ignored_and_start_is_used():
    r = make_residual(32, 16, seed=6)
    gen = np.random.default_rng(4)
    b0 = gen.standard_normal((16, 6))
    a1, b1 = O.svd_solver(r, b0, 2, 2)
    a2, b2 = O.svd_solver(r, b0[:, :2], 2, 2)
    assert np.allclose(a1 @ b1.T, a2 @ b2.T)
    a3, b3 = O.svd_solver(r, gen.standard_normal((16, 2)), 2, 1)
    assert not np.allclose(a1 @ b1.T, a3 @ b3.T)


# ----------------------------------------------------------------- attention
def textbook_attention(q, k, v):
    z = k @ q / np.sqrt(k.shape[1])
    w = np.exp(z - z.max())
    return (w / w.sum()) @ v


def new_cache(batch=1, hq=2, hkv=1, bits=4, g=32, s=2.0, nb=16, rflush=2, iters=3, d=32):
    return O.OracleCache(batch, hq, hkv, d, bits, g, s, nb, rflush, iters)


def test_buffer_only_cache_is_textbook_attention():
    gen = np.random.default_rng(0)
    c = new_cache()
    ks = gen.standard_normal((5, 1, 1, 32)).astype(np.float16)
    vs = gen.standard_normal((5, 1, 1, 32)).astype(np.float16)
    for t in range(5):
        assert c.append(ks[t], vs[t]) is False
    q = gen.standard_normal((1, 2, 32)).astype(np.float16)
    out = c.decode_attn(q)
    for h in range(2):
        want = textbook_attention(q[0, h].astype(np.float64), ks[:, 0, 0].astype(np.float64), vs[:, 0, 0].astype(np.float64))
        assert np.allclose(out[0, h], want, atol=1e-13)
    # zero query -> uniform weights -> column mean of V^
    out0 = c.decode_attn(np.zeros((1, 2, 32), np.float16))
    assert np.allclose(out0[0, 0], vs[:, 0, 0].astype(np.float64).mean(axis=0), atol=1e-13)


def test_grid_inputs_make_gear_attention_exact():
    """Inputs on the b-bit grid of every group: D^ = X, R = 0, so GEAR attention equals exact attention on X."""
    gen = np.random.default_rng(1)
    n, d, g = 64, 32, 32
    # K: per channel (column) grid; V: per token grid
    ck = gen.integers(0, 16, (n, d)); ck[0::32] = 0; ck[1::32] = 15
    k16 = (-2.0 + 0.25 * ck).astype(np.float16)
    cv = gen.integers(0, 16, (n, d)); cv[:, 0] = 0; cv[:, 1] = 15
    v16 = (1.0 + 0.125 * cv).astype(np.float16)
    c = new_cache(s=0.0, g=g)
    b0 = gen.standard_normal((1, 1, 2, d, 2)).astype(np.float32)
    c.compress(k16[None, None], v16[None, None], 2, b0)
    tk = c.segments[0]["K"][0][0]
    assert np.array_equal(tk["D"], k16.astype(np.float64)) and not tk["R"].any()
    q = gen.standard_normal((1, 2, d)).astype(np.float16)
    out = c.decode_attn(q)
    for h in range(2):
        want = textbook_attention(q[0, h].astype(np.float64), k16.astype(np.float64), v16.astype(np.float64))
        assert np.allclose(out[0, h], want, atol=1e-12)


def test_factored_low_rank_and_sparse_evaluation_matches_materialised():
    """(q B) A^T and (p A) B^T -- the down- then up-projection of Section 4 -- equal the dense products;
    segment order does not change the output; GQA heads read the shared kv head."""
    gen = np.random.default_rng(2)
    d = 32
    c = new_cache(hq=4, hkv=2, batch=2, bits=2, g=32, s=4.0, nb=16, rflush=2, d=d)
    k16 = (gen.standard_normal((2, 2, 64, d)) * gen.lognormal(0, 1, (1, 2, 1, d))).astype(np.float16)
    v16 = gen.standard_normal((2, 2, 64, d)).astype(np.float16)
    c.compress(k16, v16, 3, gen.standard_normal((2, 2, 2, d, 3)).astype(np.float32))
    flushed = []
    for t in range(20):
        flushed.append(c.append(gen.standard_normal((2, 2, d)).astype(np.float16),
                                gen.standard_normal((2, 2, d)).astype(np.float16),
                                gen.standard_normal((2, 2, 2, d, 2)).astype(np.float32)))
    assert flushed.index(True) == 15 and sum(flushed) == 1          # flush on the push that fills the buffer
    assert len(c.segments) == 2 and c.buf_k.shape[2] == 4
    assert c.segments[1]["n_c"] == 16 and c.segments[1]["rank"] == 2
    q = gen.standard_normal((2, 4, d)).astype(np.float16)
    out = c.decode_attn(q)
    scale = 1 / np.sqrt(d)
    for b in range(2):
        for h in range(4):
            hk = h // 2
            qq = q[b, h].astype(np.float64)
            z_parts, segs = [], []
            for s in c.segments:
                tk, tv = s["K"][b][hk], s["V"][b][hk]
                z_parts.append(tk["D"] @ qq + tk["A"] @ (tk["B"].T @ qq) + tk["S"] @ qq)
                segs.append(tv)
            z_parts.append(c.buf_k[b, hk].astype(np.float64) @ qq)
            z = np.concatenate(z_parts) * scale
            p = np.exp(z - z.max()); p /= p.sum()
            o = np.zeros(d); off = 0
            for tv in segs:
                pp = p[off:off + tv["n_c"]]; off += tv["n_c"]
                o += pp @ tv["D"] + (pp @ tv["A"]) @ tv["B"].T + pp @ tv["S"]
            o += p[off:] @ c.buf_v[b, hk].astype(np.float64)
            assert np.allclose(out[b, h], o, atol=1e-12)
    # swapping the two segments leaves the output unchanged
    c.segments.reverse()
    assert np.allclose(c.decode_attn(q), out, atol=1e-12)
    # explicit softmax scale
    assert not np.allclose(c.decode_attn(q, 0.5), out)


def test_compressed_attention_close_to_fp16_attention():
    """Sanity on the synthetic workload: 4-bit GEAR attention stays near exact attention, and adding
    the low-rank and sparse parts does not hurt."""
    w = synth.WORKLOADS[1]
    k16, v16 = synth.make_kv(1, 1, 1, w.n, 128)
    q = synth.make_query(1, 1, 1, 128)
    b0 = synth.make_b0(1, 1, 1, 128, 4)
    exact = textbook_attention(q[0, 0].astype(np.float64), k16[0, 0].astype(np.float64), v16[0, 0].astype(np.float64))
    errs = {}
    for name, s, r in (("quant", 0.0, 0), ("gear", 2.0, 4)):
        c = O.OracleCache(1, 1, 1, 128, 4, 64, s, 16, r, 3)
        c.compress(k16, v16, r, b0)
        errs[name] = np.abs(c.decode_attn(q)[0, 0] - exact).max() / np.abs(exact).max()
    assert errs["gear"] < 0.5 * errs["quant"]
    assert errs["gear"] < 0.2


def test_algorithmic_bytes_table():
    # per (token, kv head): 2-bit g64 k1 r4 -> 120 B; 4-bit r8 -> 200; 2-bit r8 -> 136; g128 k2 r4 -> 112
    assert O.algorithmic_bytes_per_token_head(128, 2, 64, 64, 1, 1, 4) == 120
    assert O.algorithmic_bytes_per_token_head(128, 4, 64, 64, 1, 1, 8) == 200
    assert O.algorithmic_bytes_per_token_head(128, 2, 64, 64, 1, 1, 8) == 136
    assert O.algorithmic_bytes_per_token_head(128, 2, 128, 128, 2, 2, 4) == 112
