"""Pins for the oracle's Filter_s (Eq. 4) and outlier-aware Quant_b (Eq. 2, Eq. 5).

None of these retypes the oracle's formula: they use brute force on tiny groups,
exact rational arithmetic, closed forms and invariants the equations imply."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import gear_oracle as O
from paper_2403_05527_b200 import synth


def brute_filter(x, k):
    """Independent statement of the selection: repeatedly take the best remaining entry."""
    x = [float(v) for v in x]
    free = list(range(len(x)))
    top, bottom = [], []
    for _ in range(k):
        best = free[0]
        for i in free:
            if x[i] > x[best]:
                best = i
        top.append(best)
        free.remove(best)
    for _ in range(k):
        best = free[0]
        for i in free:
            if x[i] < x[best]:
                best = i
        bottom.append(best)
        free.remove(best)
    return sorted(top), sorted(bottom)


@pytest.mark.parametrize("length,k", [(8, 1), (16, 2), (64, 1), (64, 3), (128, 2), (5, 2)])
def test_filter_matches_brute_force_with_ties(length, k):
    gen = np.random.default_rng(length * 31 + k)
    for trial in range(40):
        # few distinct values -> many ties, including +0 / -0
        x = gen.integers(-3, 4, size=length).astype(np.float16)
        if trial % 3 == 0:
            x[gen.integers(0, length)] = np.float16(-0.0)
        mask = O.filter_groups(x[None, :].astype(np.float64), k)[0]
        top, bottom = brute_filter(x, k)
        assert sorted(np.nonzero(mask)[0].tolist()) == sorted(top + bottom)
        assert mask.sum() == 2 * k
        # separation: nothing left is larger than a top entry or smaller than a bottom entry
        rest = x[~mask].astype(np.float64)
        assert rest.max() <= min(float(x[i]) for i in top)
        assert rest.min() >= max(float(x[i]) for i in bottom)


def test_filter_tie_prefers_low_index_and_top_first():
    x = np.array([5, 5, 5, 1, 1, 1, 3, 3], dtype=np.float64)
    m = O.filter_groups(x[None], 2)[0]
    assert np.nonzero(m)[0].tolist() == [0, 1, 3, 4]
    # all equal: top takes 0..k-1, bottom the next k
    m = O.filter_groups(np.ones((1, 8)), 2)[0]
    assert np.nonzero(m)[0].tolist() == [0, 1, 2, 3]


def test_outlier_count_rule():
    # k = ceil(s * len / 200), zero only for s = 0
    assert O.outlier_count(2.0, 64) == 1
    assert O.outlier_count(1.0, 64) == 1
    assert O.outlier_count(2.0, 128) == 2
    assert O.outlier_count(2.0, 100) == 1
    assert O.outlier_count(2.0, 101) == 2
    assert O.outlier_count(0.0, 64) == 0
    assert O.outlier_count(2.0, 16) == 1
    assert O.outlier_count(10.0, 64) == 4
    for s in (0.5, 1.0, 2.0, 3.3, 10.0):
        for n in (16, 32, 64, 128, 4096):
            assert O.outlier_count(s, n) == int(np.ceil(Fraction(str(s)) * n / 200))
    with pytest.raises(ValueError):
        O.outlier_count(60.0, 4)


def test_s_zero_gives_empty_sparse_part():
    k16, _ = synth.make_kv(1, 1, 1, 64, 128)
    t = O.compress_tile(k16[0, 0], "K", 4, 64, 0.0, 0, 3, None)
    assert not t["mask"].any() and not t["S"].any() and t["out_idx"].shape[1] == 0


@pytest.mark.parametrize("kind", ["K", "V"])
@pytest.mark.parametrize("bits", [2, 4])
def test_outliers_reproduced_exactly_and_counts(kind, bits):
    k16, v16 = synth.make_kv(1, 1, 1, 128, 128)
    x16 = (k16 if kind == "K" else v16)[0, 0]
    t = O.compress_tile(x16, kind, bits, 64, 2.0, 0, 3, None)
    x = x16.astype(np.float64)
    # S carries the exact input bits on its support, D^ is zero there, so D^ + S == X there
    assert np.array_equal(t["S"][t["mask"]], x[t["mask"]])
    assert np.array_equal((t["D"] + t["S"])[t["mask"]], x[t["mask"]])
    assert np.all(t["R"][t["mask"]] == 0.0)
    assert np.all(t["codes"][t["mask"]] == 0)
    # exactly 2k per group, along tokens for K and along channels for V
    if kind == "K":
        per = t["mask"].reshape(2, 64, 128).sum(axis=1)
    else:
        per = t["mask"].reshape(128, 2, 64).sum(axis=2)
    assert np.all(per == 2)
    # exported lists agree with the mask and the input
    gr = O.tile_to_groups(x, kind, 64)
    for gi in range(0, gr.shape[0], 17):
        idx = t["out_idx"][gi].astype(int)
        assert np.all(np.diff(idx) > 0)
        assert np.array_equal(t["out_val"][gi].astype(np.float64), gr[gi, idx])


@pytest.mark.parametrize("kind", ["K", "V"])
@pytest.mark.parametrize("bits", [2, 4])
@pytest.mark.parametrize("s", [0.0, 2.0])
def test_quant_error_bound_and_code_range(kind, bits, s):
    k16, v16 = synth.make_kv(1, 1, 1, 128, 128, extra=3)
    x16 = (k16 if kind == "K" else v16)[0, 0]
    t = O.compress_tile(x16, kind, bits, 64, s, 0, 3, None)
    lv = 2 ** bits - 1
    assert t["codes"].max() <= lv
    x = x16.astype(np.float64)
    gr_x = O.tile_to_groups(x, kind, 64)
    gr_m = O.tile_to_groups(t["mask"], kind, 64)
    gr_c = O.tile_to_groups(t["codes"], kind, 64)
    scale = t["scale"].astype(np.float64).reshape(-1) if kind == "V" else t["scale"].astype(np.float64).reshape(-1)
    zero = t["zero"].astype(np.float64).reshape(-1)
    for gi in range(gr_x.shape[0]):
        keep = ~gr_m[gi]
        xs, cs = gr_x[gi][keep], gr_c[gi][keep].astype(np.float64)
        d, m = scale[gi], zero[gi]
        # stored zero-point is the minimum of the kept entries, which maps to code 0; the max maps to 2^b-1
        assert m == xs.min()
        assert cs[np.argmin(xs)] == 0
        if d > 0:
            assert cs[np.argmax(xs)] == lv
            if d >= 2.0 ** -14:       # normal fp16 scale: |x - dequant| <= scale * (1/2 + 2^-17)
                assert np.all(np.abs(xs - (cs * d + m)) <= d * (0.5 + 2.0 ** -17) + 1e-300)


def test_quant_agrees_with_exact_rational_rounding():
    """Eq. 2 evaluated in exact rational arithmetic on the stored scale: the
    binary32 recipe may differ only where the exact quotient is within 2^-16
    of a half-integer."""
    gen = np.random.default_rng(5)
    x16 = (gen.standard_normal((200, 64)) * gen.lognormal(0, 1, (200, 1))).astype(np.float16)
    for bits in (2, 4):
        codes, sc, ze = O.quantize_groups(x16, np.zeros(x16.shape, bool), bits)
        lv = 2 ** bits - 1
        n_close = 0
        for gi in range(x16.shape[0]):
            d = Fraction(float(sc[gi]))
            m = Fraction(float(ze[gi]))
            assert float(ze[gi]) == float(x16[gi].astype(np.float64).min())
            # scale = fp16( fp32( fp32(max-min) / levels ) ): check against the exact quotient
            exact = (Fraction(float(x16[gi].astype(np.float64).max())) - m) / lv
            assert abs(Fraction(float(sc[gi])) - exact) <= exact * Fraction(1, 2 ** 11) + Fraction(1, 2 ** 25)
            if d == 0:
                assert not codes[gi].any()
                continue
            for j in range(64):
                tq = (Fraction(float(x16[gi, j])) - m) / d
                fl = tq.numerator // tq.denominator
                frac = tq - fl
                if abs(frac - Fraction(1, 2)) < Fraction(1, 2 ** 16):
                    n_close += 1
                    assert int(codes[gi, j]) in (min(fl, lv), min(fl + 1, lv))
                else:
                    want = fl + (1 if frac > Fraction(1, 2) else 0)
                    assert int(codes[gi, j]) == min(max(want, 0), lv)
        assert n_close < 200


def test_quant_grid_inputs_round_trip_exactly():
    """A group lying on m + c * d with fp16-representable d is reproduced with zero error."""
    gen = np.random.default_rng(11)
    for bits in (2, 4):
        lv = 2 ** bits - 1
        for d, m in ((0.25, -1.5), (0.5, 3.0), (2.0 ** -6, 0.125), (3.0, -24.0)):
            c = gen.integers(0, lv + 1, size=(7, 64))
            c[:, 0], c[:, 1] = 0, lv                    # make min and max present
            x16 = (m + c * d).astype(np.float16)
            assert np.array_equal(x16.astype(np.float64), m + c * d)
            codes, sc, ze = O.quantize_groups(x16, np.zeros(x16.shape, bool), bits)
            assert np.array_equal(codes, c)
            assert np.all(sc.astype(np.float64) == d) and np.all(ze.astype(np.float64) == m)
            deq = O.dequantize_groups(codes, sc, ze, np.zeros(x16.shape, bool))
            assert np.array_equal(deq, x16.astype(np.float64))


def test_constant_group_gives_zero_codes():
    x16 = np.full((3, 32), 1.75, np.float16)
    codes, sc, ze = O.quantize_groups(x16, np.zeros(x16.shape, bool), 4)
    assert not codes.any() and np.all(sc == 0) and np.all(ze == np.float16(1.75))
    assert np.array_equal(O.dequantize_groups(codes, sc, ze, np.zeros(x16.shape, bool)), x16.astype(np.float64))


def test_s0_r0_is_plain_group_quantization():
    """With s = 0 and r = 0 the tile is Eq. 2 per group: per-token groups for V,
    per-channel groups for K -- check against a direct per-group evaluation in
    a different layout (explicit loops over tokens / channels)."""
    k16, v16 = synth.make_kv(1, 1, 1, 64, 128, extra=9)
    tv = O.compress_tile(v16[0, 0], "V", 4, 64, 0.0, 0, 3, None)
    tk = O.compress_tile(k16[0, 0], "K", 4, 32, 0.0, 0, 3, None)
    assert tv["A"].shape[1] == 0 and not tv["S"].any()
    xv = v16[0, 0].astype(np.float64)
    for i in (0, 5, 63):
        for c in range(2):
            grp = xv[i, c * 64:(c + 1) * 64]
            d = float(tv["scale"][i, c])
            want = np.clip(np.rint((grp - grp.min()) / d), 0, 15)
            got = tv["codes"][i, c * 64:(c + 1) * 64]
            assert np.abs(got - want).max() <= 1 and (got != want).mean() < 0.05
            assert float(tv["zero"][i, c]) == grp.min()
            assert abs(d - (grp.max() - grp.min()) / 15) <= d * 2.0 ** -10
    xk = k16[0, 0].astype(np.float64)
    for j in (0, 17, 127):
        for blk in range(2):
            grp = xk[blk * 32:(blk + 1) * 32, j]
            assert float(tk["zero"][blk, j]) == grp.min()
            d = float(tk["scale"][blk, j])
            assert abs(d - (grp.max() - grp.min()) / 15) <= d * 2.0 ** -10
    # X^ = D^ exactly and the error obeys the half-step bound
    assert np.array_equal(O.reconstruct_tile(tv), tv["D"])
    err = np.abs(xv - tv["D"]).reshape(64, 2, 64).max(axis=2)
    assert np.all(err <= tv["scale"].astype(np.float64) * (0.5 + 2.0 ** -17))


def test_short_segment_uses_whole_column_groups():
    """A 16-token segment with g = 64: keys are quantized per whole column (g_K = 16)."""
    k16, _ = synth.make_kv(1, 1, 1, 16, 128, extra=2)
    t = O.compress_tile(k16[0, 0], "K", 4, 64, 2.0, 0, 3, None)
    assert t["scale"].shape == (1, 128) and t["g_len"] == 16 and t["k"] == 1
    assert np.all(t["mask"].sum(axis=0) == 2)
    with pytest.raises(ValueError):
        O.group_lengths(100, 128, 64)


def test_error_ordering_of_the_three_components():
    """||X - D^|| >= ||X - D^ - S|| >= ||X - D^ - S - L||  (objective of Eq. 3)."""
    k16, v16 = synth.make_kv(1, 1, 1, 128, 128, extra=4)
    b0 = synth.make_b0(1, 1, 1, 128, 4)
    for kind, x16, j in (("K", k16, 0), ("V", v16, 1)):
        t = O.compress_tile(x16[0, 0], kind, 2, 64, 2.0, 4, 3, b0[0, 0, j])
        x = x16[0, 0].astype(np.float64)
        e_d = np.linalg.norm(x - t["D"])
        e_ds = np.linalg.norm(x - t["D"] - t["S"])
        e_all = np.linalg.norm(x - O.reconstruct_tile(t))
        assert e_d >= e_ds >= e_all
        # and filtering outliers before quantizing beats quantizing everything
        t0 = O.compress_tile(x16[0, 0], kind, 2, 64, 0.0, 0, 3, None)
        assert np.linalg.norm(x - t0["D"]) > e_ds


def test_exact_half_steps_round_to_even():
    """Entries exactly halfway between two levels go to the even code (the tie rule this build fixes for Eq. 2)."""
    x16 = np.array([[0.0, 3.0, 0.5, 1.5, 2.5, 1.0, 2.0, 0.75]], np.float16)
    codes, sc, ze = O.quantize_groups(x16, np.zeros(x16.shape, bool), 2)
    assert float(sc[0]) == 1.0 and float(ze[0]) == 0.0
    assert codes[0].tolist() == [0, 3, 0, 2, 2, 1, 2, 1]


# --------------------------------------------------------------------------- the other readings of Section 3
def _vec_brute_force(vec, k):
    """k largest then k smallest of what is left, value first, lower index on ties: plain loops."""
    chosen = []
    for sign in (-1.0, 1.0):
        order = sorted((i for i in range(len(vec)) if i not in chosen), key=lambda i: (sign * float(vec[i]), i))
        chosen += order[:k]
    return sorted(chosen)


def test_per_vector_filter_is_eq4_on_whole_channels_and_tokens():
    """filter_len = the vector length: s/2 % of the largest and smallest entries of every key channel over all tokens
    and of every value token over all channels (Eq. 4 as printed), while the quantization groups keep length g."""
    rng = np.random.default_rng(21)
    n_c, d, g = 64, 128, 16
    x = rng.standard_normal((n_c, d)).astype(np.float16)
    x[rng.random((n_c, d)) < 0.02] *= 12
    tk = O.compress_tile(x, "K", 4, g, 8.0, 0, 3, None, filter_len=n_c)
    tv = O.compress_tile(x, "V", 4, g, 8.0, 0, 3, None, filter_len=d)
    kk, kv = O.outlier_count(8.0, n_c), O.outlier_count(8.0, d)
    for j in range(0, d, 17):
        assert sorted(np.nonzero(tk["mask"][:, j])[0]) == _vec_brute_force(x[:, j], kk)
    for i in range(0, n_c, 9):
        assert sorted(np.nonzero(tv["mask"][i])[0]) == _vec_brute_force(x[i], kv)
    for t in (tk, tv):
        assert np.array_equal(t["S"][t["mask"]], x.astype(np.float64)[t["mask"]])     # outliers kept exactly
        assert np.all(t["D"][t["mask"]] == 0) and np.all(t["R"][t["mask"]] == 0)
        keep = ~t["mask"]
        scale = np.repeat(t["scale"].astype(np.float64), g, axis=0 if t["kind"] == "K" else 1)
        assert np.all(np.abs(t["R"][keep]) <= scale[keep] * (0.5 + 2.0 ** -10))


def test_filter_length_equal_to_the_group_is_the_default_and_whole_vector_groups_are_kcvt():
    rng = np.random.default_rng(22)
    x = (rng.standard_normal((128, 128)) * np.exp(rng.standard_normal(128))).astype(np.float16)
    for kind, g in (("K", 32), ("V", 64)):
        a = O.compress_tile(x, kind, 2, g, 4.0, 2, 3, rng.standard_normal((128, 2)))
        b = O.compress_tile(x, kind, 2, g, 4.0, 2, 3, rng.standard_normal((128, 2)), filter_len=g)
        for key in ("codes", "mask", "D"):
            assert np.array_equal(a[key], b[key])
    # groups as long as the vectors: one (scale, zero) per key channel over all tokens, one per value token
    tk = O.compress_tile(x, "K", 4, 10 ** 6, 2.0, 0, 3, None)
    tv = O.compress_tile(x, "V", 4, 10 ** 6, 2.0, 0, 3, None)
    assert tk["scale"].shape == (1, 128) and tv["scale"].shape == (128, 1)
    j = 5
    keep = ~tk["mask"][:, j]
    col = x[:, j].astype(np.float64)
    assert tk["zero"][0, j] == np.float16(col[keep].min())
    d32 = np.float32(np.float32(col[keep].max() - col[keep].min()) / np.float32(15))
    assert tk["scale"][0, j] == np.float16(d32)
    assert tk["mask"][:, j].sum() == 2 * O.outlier_count(2.0, 128)


def test_literal_eq5_codes_the_zeros_left_by_the_outliers():
    """Quant_b(X - S) with the zeros in the range: an all-positive group's minimum becomes 0, its range widens, and the
    outlier positions carry D^ = dequant(code of 0), R = -D^ there; X^ = D^ + S + R still equals X everywhere."""
    rng = np.random.default_rng(23)
    x = (np.abs(rng.standard_normal((64, 128))) + 3.0).astype(np.float16)        # every group is strictly positive
    lit = O.compress_tile(x, "V", 4, 64, 4.0, 0, 3, None, literal_eq5=True)
    msk = O.compress_tile(x, "V", 4, 64, 4.0, 0, 3, None)
    assert np.array_equal(lit["mask"], msk["mask"])
    assert np.all(lit["zero"] == 0) and np.all(msk["zero"].astype(np.float64) >= 3.0)
    assert np.all(lit["scale"].astype(np.float64) > msk["scale"].astype(np.float64))
    m = lit["mask"]
    assert np.all(lit["D"][m] == 0.0) and np.all(lit["codes"][m] == 0)           # quant(0) with zero-point 0 is code 0
    x64 = x.astype(np.float64)
    assert np.allclose(lit["D"] + lit["S"] + lit["R"], x64, atol=0, rtol=0)
    # a group that straddles zero: the zero entries land on a grid point near 0, not on 0
    y = rng.standard_normal((64, 128)).astype(np.float16)
    lit2 = O.compress_tile(y, "K", 2, 64, 4.0, 0, 3, None, literal_eq5=True)
    m2 = lit2["mask"]
    scale = np.repeat(lit2["scale"].astype(np.float64), 64, axis=0)
    assert np.all(np.abs(lit2["D"][m2]) <= scale[m2] * (0.5 + 2.0 ** -10))
    assert np.any(lit2["D"][m2] != 0.0)
    assert np.array_equal(lit2["R"][m2], -lit2["D"][m2])


def test_per_vector_grouping_on_a_long_segment_by_brute_force():
    """With g beyond every vector (Section 2, per-vector grouping) a key group is a whole channel: Eq. 4 takes the
    k = ceil(s n / 200) largest and smallest of its n tokens (ties to the lower token, the smallest among what the
    largest left), and Eq. 2 sees the rest.  Checked entry by entry against a sort written out here; the index of an
    outlier no longer fits a byte."""
    rng = np.random.default_rng(11)
    n = 320
    x = np.round(rng.standard_normal((n, 128)) * 4).astype(np.float16) / np.float16(4)      # many equal entries
    t = O.compress_tile(x, "K", 4, 1 << 30, 2.0, 0, 3, None)
    k = O.outlier_count(2.0, n)
    assert (t["g_len"], k, t["out_idx"].dtype, t["scale"].shape) == (n, 4, np.int32, (1, 128))
    for ch in (0, 17, 127):
        col = x[:, ch].astype(np.float64)
        order = sorted(range(n), key=lambda i: (-col[i], i))
        top = order[:k]
        rest = [i for i in range(n) if i not in top]
        bot = sorted(rest, key=lambda i: (col[i], i))[:k]
        out = sorted(top + bot)
        assert list(t["out_idx"][ch]) == out
        kept = [i for i in range(n) if i not in out]
        lo, hi = col[kept].min(), col[kept].max()
        assert float(t["zero"][0, ch]) == lo
        assert float(t["scale"][0, ch]) == float(np.float16(np.float32(hi - lo) / np.float32(15)))
        assert not t["mask"][kept, ch].any() and t["mask"][out, ch].all()
