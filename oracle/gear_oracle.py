"""CPU oracle for the GEAR hot path (arXiv 2403.05527) -- TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 numpy restatement of what the paper's method computes:
Filter_s (Eq. 4), outlier-aware group quantization (Eq. 2, Eq. 5), the residual
R = X - D^ - S (Section 3, "Low-rank approximation"), the power-iteration
SVDSolver (Algorithm 2), the prefill/decode cache of Algorithm 1 with its
streaming buffer, and decode attention (Eq. 1) over K^ = D^ + A B^T + S.

This module is the parity reference for the CUDA library.  It shares no code
with it, imports nothing from it, and must only be imported by the tests, by
the smoke check and by the benchmark's CPU-baseline leg.  No blocking, fusion
or reordering beyond what the paper's definitions state.

Every function is pinned by the CPU tests (invariants, closed forms, brute
force on tiny inputs, textbook special cases); none is "parity unpinned".

Readings taken where the paper is silent (each is restated where used):
  * Filter acts on each quantization group ("to align with grouping",
    Section 3): k = ceil(s * len / 200) largest and k smallest entries.
  * Ties: larger value first, then lower in-group index; the top set is chosen
    before the bottom set; +0 and -0 compare equal.
  * min / max / codes are taken over the non-outlier entries of a group; the
    code stored at an outlier position is 0 and D^ is 0 there, so D^ + S
    reproduces an outlier exactly.
  * The quantizer arithmetic is a fixed sequence of binary32 operations
    (round-to-nearest-even, no fused multiply-add); scale and zero-point are
    stored in binary16.  Each op is done here in float64 and cast to float32,
    which yields the same bits as a correctly rounded binary32 op.
  * Group length along tokens for keys is min(g, n_c); along channels for
    values min(g, d_H).
"""
from __future__ import annotations

import numpy as np

F64 = np.float64
F32 = np.float32
F16 = np.float16


# --------------------------------------------------------------------------
# geometry and counts
# --------------------------------------------------------------------------
def group_lengths(n_c: int, d_h: int, g: int) -> tuple[int, int]:
    """Group length of keys (tokens of one channel) and values (channels of one
    token): per-channel keys, per-token values (Section 2, "Group-wise
    Quantization"); a vector shorter than g forms one group (the per-vector
    KCVT limit of the same section)."""
    g_k = min(g, n_c)
    g_v = min(g, d_h)
    if n_c % g_k or d_h % g_v:
        raise ValueError("segment length / head dim must be a multiple of the group length")
    return g_k, g_v


def outlier_count(s_pct: float, length: int) -> int:
    """k = ceil(s/2 % of `length`) entries per side (Eq. 4: s/2 % of the maxima
    and s/2 % of the minima).  Integer arithmetic on s in units of 1e-4 %."""
    s_units = int(round(float(s_pct) * 10000.0))
    if s_units < 0:
        raise ValueError("s must be >= 0")
    k = -((-s_units * length) // 2_000_000)
    if 2 * k >= length and k > 0:
        raise ValueError("too many outliers for the group length")
    return k


# --------------------------------------------------------------------------
# Filter_s  (Eq. 4) on an array of groups [n_groups, length]
# --------------------------------------------------------------------------
def filter_groups(groups: np.ndarray, k: int) -> np.ndarray:
    """Boolean mask [n_groups, length] of the entries Filter_s extracts: the k
    largest, then the k smallest of what is left.  Order: value, then lower
    index (a stable sort on the negated / plain values gives exactly that)."""
    x = np.asarray(groups, dtype=F64)
    mask = np.zeros(x.shape, dtype=bool)
    if k == 0:
        return mask
    rows = np.arange(x.shape[0])[:, None]
    top = np.argsort(-x, axis=1, kind="stable")[:, :k]
    mask[rows, top] = True
    rest = np.where(mask, np.inf, x)            # remove the top set from the candidates
    bottom = np.argsort(rest, axis=1, kind="stable")[:, :k]
    mask[rows, bottom] = True
    return mask


# --------------------------------------------------------------------------
# Quant_b  (Eq. 2 applied to X - S, Eq. 5) on an array of groups
# --------------------------------------------------------------------------
def quantize_groups(groups16: np.ndarray, outlier_mask: np.ndarray, bits: int):
    """Asymmetric uniform quantization of each row (one group).

    Returns (codes uint8 [n_groups, length], scale float16 [n_groups],
    zero float16 [n_groups]).  Recipe, all in binary32 RNE without FMA:
        m, M   = min / max of the non-outlier entries          (exact, fp16 values)
        range  = f32(M - m)
        d32    = f32(range / (2^b - 1))
        scale  = f16(d32)            (stored);  zero = m (stored)
        scale == 0  ->  all codes 0
        inv    = f32(1 / f32(scale))
        t      = f32(f32(x - m) * inv)
        code   = clamp(round_half_even(t), 0, 2^b - 1);   outlier positions -> 0
    """
    x = np.asarray(groups16, dtype=F16).astype(F64)
    keep = ~np.asarray(outlier_mask, dtype=bool)
    levels = (1 << bits) - 1
    m = np.min(np.where(keep, x, np.inf), axis=1)
    big = np.max(np.where(keep, x, -np.inf), axis=1)
    rng = (big - m).astype(F32)
    d32 = (rng.astype(F64) / levels).astype(F32)
    scale16 = d32.astype(F16)
    zero16 = m.astype(F16)                      # exact: m is an fp16 input value
    sc = scale16.astype(F64)
    nz = sc != 0.0
    inv = np.zeros_like(sc, dtype=F32)
    inv[nz] = (1.0 / sc[nz]).astype(F32)
    diff = (x - m[:, None]).astype(F32)
    t = (diff.astype(F64) * inv.astype(F64)[:, None]).astype(F32)
    codes = np.clip(np.rint(t.astype(F64)), 0, levels)
    codes = np.where(keep & nz[:, None], codes, 0).astype(np.uint8)
    return codes, scale16, zero16


def dequantize_groups(codes, scale16, zero16, outlier_mask):
    """D^ = code * scale + zero at non-outlier positions, 0 at outlier positions."""
    d = codes.astype(F64) * scale16.astype(F64)[:, None] + zero16.astype(F64)[:, None]
    return np.where(outlier_mask, 0.0, d)


# --------------------------------------------------------------------------
# tile <-> groups  (per-channel keys, per-token values)
# --------------------------------------------------------------------------
def tile_to_groups(x: np.ndarray, kind: str, g_len: int) -> np.ndarray:
    """[n_c, d_H] -> [n_groups, g_len].
    'K': group (blk, j) = tokens blk*g_len .. of channel j; row = blk*d_H + j.
    'V': group (i, c)   = channels c*g_len .. of token i;   row = i*(d_H/g_len) + c."""
    n_c, d_h = x.shape
    if kind == "K":
        return x.reshape(n_c // g_len, g_len, d_h).transpose(0, 2, 1).reshape(-1, g_len)
    if kind == "V":
        return x.reshape(n_c * (d_h // g_len), g_len)
    raise ValueError(kind)


def groups_to_tile(gr: np.ndarray, kind: str, n_c: int, d_h: int) -> np.ndarray:
    g_len = gr.shape[1]
    if kind == "K":
        return gr.reshape(n_c // g_len, d_h, g_len).transpose(0, 2, 1).reshape(n_c, d_h)
    return gr.reshape(n_c, d_h)


# --------------------------------------------------------------------------
# SVDSolver  (Algorithm 2)
# --------------------------------------------------------------------------
def svd_solver(r_h: np.ndarray, b0: np.ndarray, rank: int, iters: int):
    """Power iteration of Algorithm 2 on R_h [n_c, d_H] from the start B0
    [d_H, >=rank].  The random start of A in the listing is dead (A is
    overwritten before use); B0 is an explicit input.  Loop l = 0..L-1:
    A = R B ; B = R^T A, with B orthonormalised before and A after the product
    A = R B in the last loop only.  Returns A [n_c, r] (orthonormal columns)
    and B [d_H, r] = R^T A."""
    r_h = np.asarray(r_h, dtype=F64)
    n_c, d_h = r_h.shape
    if rank == 0:
        return np.zeros((n_c, 0)), np.zeros((d_h, 0))
    if rank > min(n_c, d_h):
        raise ValueError("rank exceeds the tile")
    if iters < 1:
        raise ValueError("need at least one loop")
    b = np.asarray(b0, dtype=F64)[:, :rank].copy()
    a = None
    for l in range(iters):
        last = l == iters - 1
        if last:
            b, _ = np.linalg.qr(b)
        a = r_h @ b
        if last:
            a, _ = np.linalg.qr(a)
        b = r_h.T @ a
    return a, b


# --------------------------------------------------------------------------
# one tile: Filter -> Quant -> residual -> SVDSolver   (Algorithm 1, prefill body)
# --------------------------------------------------------------------------
def compress_tile(x16: np.ndarray, kind: str, bits: int, g: int, s_pct: float,
                  rank: int, iters: int, b0: np.ndarray | None,
                  filter_len: int | None = None, literal_eq5: bool = False):
    """Compress one (batch, head) tile X [n_c, d_H] (fp16) of keys ('K') or
    values ('V').

    Two switches select the other readings of Section 3 (defaults: the readings
    listed in the module header):
      filter_len   length of the vectors Filter_s acts on, along the grouping
                   axis (tokens of a channel for keys, channels of a token for
                   values).  None: the quantization group.  n_c for keys / d_H
                   for values is Eq. 4 read literally: s/2 % of the largest and
                   of the smallest entries of each whole channel / token vector.
                   Must be a multiple of the group length.
      literal_eq5  Eq. 5 read literally: the zeros that X - S holds at the
                   outlier positions take part in min / max and receive a code
                   like every other entry, so D^ is not 0 there and the residual
                   at an outlier position is -D^.
    With g at least the vector length the groups are the whole vectors (the
    per-vector grouping, KCVT, of Section 2).

    Returns a dict with the canonical (unpacked) pieces:
      codes u8 [n_c, d_H]; scale, zero fp16 ('K': [n_c/g_K, d_H]; 'V': [n_c, d_H/g_V]);
      mask bool [n_c, d_H] (support of S); S float64 (exact fp16 values on the mask);
      out_idx u8 (int32 for groups longer than 256) / out_val fp16 [n_groups, 2k] (in-group index ascending);
      D float64 (dequantised backbone, 0 on the mask); R; A [n_c, r]; B [d_H, r]."""
    x16 = np.asarray(x16, dtype=F16)
    n_c, d_h = x16.shape
    g_k, g_v = group_lengths(n_c, d_h, g)
    g_len = g_k if kind == "K" else g_v
    k = outlier_count(s_pct, g_len)
    x = x16.astype(F64)

    gr = tile_to_groups(x, kind, g_len)
    if filter_len is None or filter_len == g_len:
        gmask = filter_groups(gr, k)                               # Eq. 4, per quantization group
        kf = k
    else:
        vec_len = n_c if kind == "K" else d_h
        if filter_len % g_len or vec_len % filter_len:
            raise ValueError("filter length must be a multiple of the group length and divide the vector")
        kf = outlier_count(s_pct, filter_len)
        fmask = filter_groups(tile_to_groups(x, kind, filter_len), kf)          # Eq. 4 on longer vectors
        gmask = tile_to_groups(groups_to_tile(fmask, kind, n_c, d_h), kind, g_len)
    if literal_eq5:
        none = np.zeros_like(gmask)
        codes_g, scale16, zero16 = quantize_groups(np.where(gmask, 0.0, gr).astype(F16), none, bits)   # Quant_b(X - S)
        d_g = dequantize_groups(codes_g, scale16, zero16, none)
    else:
        codes_g, scale16, zero16 = quantize_groups(gr.astype(F16), gmask, bits)   # Eq. 5, outliers masked out
        d_g = dequantize_groups(codes_g, scale16, zero16, gmask)

    mask = groups_to_tile(gmask, kind, n_c, d_h)
    codes = groups_to_tile(codes_g, kind, n_c, d_h)
    d_hat = groups_to_tile(d_g, kind, n_c, d_h)
    s_mat = np.where(mask, x, 0.0)
    resid = x - d_hat - s_mat                                      # R = X - (D^ + S)

    if k and (filter_len is None or filter_len == g_len):
        idx_t = np.uint8 if g_len <= 256 else np.int32                       # an index inside a long vector needs more than a byte
        out_idx = np.nonzero(gmask)[1].reshape(-1, 2 * k).astype(idx_t)      # ascending per group
        out_val = gr[gmask].reshape(-1, 2 * k).astype(F16)
    else:                                        # none, or a varying number per group: the mask and S carry them
        out_idx = np.zeros((gr.shape[0], 0), np.uint8)
        out_val = np.zeros((gr.shape[0], 0), F16)

    if kind == "K":
        scale = scale16.reshape(n_c // g_len, d_h)
        zero = zero16.reshape(n_c // g_len, d_h)
    else:
        scale = scale16.reshape(n_c, d_h // g_len)
        zero = zero16.reshape(n_c, d_h // g_len)

    if rank:
        a, b = svd_solver(resid, b0, rank, iters)                  # Algorithm 2, per head
    else:
        a, b = np.zeros((n_c, 0)), np.zeros((d_h, 0))
    return dict(kind=kind, n_c=n_c, codes=codes, scale=scale, zero=zero, mask=mask,
                S=s_mat, out_idx=out_idx, out_val=out_val, D=d_hat, R=resid, A=a, B=b,
                g_len=g_len, k=k, rank=rank)


def reconstruct_tile(t: dict) -> np.ndarray:
    """X^ = D^ + A B^T + S  (the three components of Section 3)."""
    return t["D"] + t["A"] @ t["B"].T + t["S"]


# --------------------------------------------------------------------------
# the cache of Algorithm 1: compressed segments followed by the fp16 buffer
# --------------------------------------------------------------------------
class OracleCache:
    """Compressed KV cache of one layer: a list of compressed segments (the
    prefill block, then one per flushed buffer) followed by the streaming
    buffer of up to n_b fp16 tokens (Algorithm 1; Section 3 "Streaming
    Buffer").  Decoding reads the listing's loop as: every step pushes
    (k_t, v_t); the push that fills the buffer compresses it (rank r_g, on
    the buffered tokens only), appends the segment and clears the buffer."""

    def __init__(self, batch, n_q_heads, n_kv_heads, head_dim, bits, group, s_pct,
                 buffer_cap, rank_flush, iters):
        assert n_q_heads % n_kv_heads == 0
        self.B, self.Hq, self.Hkv, self.d = batch, n_q_heads, n_kv_heads, head_dim
        self.bits, self.g, self.s, self.nb = bits, group, s_pct, buffer_cap
        self.r_flush, self.iters = rank_flush, iters
        self.segments: list[dict] = []          # each: {'K': [[tile]*Hkv]*B, 'V': ..., 'n_c', 'rank'}
        self.buf_k = np.zeros((batch, n_kv_heads, 0, head_dim), F16)
        self.buf_v = np.zeros((batch, n_kv_heads, 0, head_dim), F16)

    def compress(self, k16, v16, rank, b0):
        """k16, v16: fp16 [B, Hkv, n, d_H]; b0: fp32 [B, Hkv, 2, d_H, rank] (0 = K, 1 = V)."""
        k16 = np.asarray(k16, F16)
        v16 = np.asarray(v16, F16)
        seg = {"K": [], "V": [], "n_c": k16.shape[2], "rank": rank}
        for b in range(self.B):
            rk, rv = [], []
            for h in range(self.Hkv):
                b0k = None if rank == 0 else b0[b, h, 0]
                b0v = None if rank == 0 else b0[b, h, 1]
                rk.append(compress_tile(k16[b, h], "K", self.bits, self.g, self.s, rank, self.iters, b0k))
                rv.append(compress_tile(v16[b, h], "V", self.bits, self.g, self.s, rank, self.iters, b0v))
            seg["K"].append(rk)
            seg["V"].append(rv)
        self.segments.append(seg)

    def append(self, k_new, v_new, b0_flush=None) -> bool:
        """Push one token per (batch, head); returns True when the push flushed."""
        k_new = np.asarray(k_new, F16).reshape(self.B, self.Hkv, 1, self.d)
        v_new = np.asarray(v_new, F16).reshape(self.B, self.Hkv, 1, self.d)
        self.buf_k = np.concatenate([self.buf_k, k_new], axis=2)
        self.buf_v = np.concatenate([self.buf_v, v_new], axis=2)
        if self.buf_k.shape[2] == self.nb:
            self.compress(self.buf_k, self.buf_v, self.r_flush, b0_flush)
            self.buf_k = self.buf_k[:, :, :0]
            self.buf_v = self.buf_v[:, :, :0]
            return True
        return False

    def materialise(self, b, h_kv):
        """K^, V^ [n_total, d_H] in float64 for one (batch, kv head): the
        concatenation of every segment's D^ + A B^T + S and the fp16 buffer."""
        ks = [reconstruct_tile(s["K"][b][h_kv]) for s in self.segments]
        vs = [reconstruct_tile(s["V"][b][h_kv]) for s in self.segments]
        ks.append(self.buf_k[b, h_kv].astype(F64))
        vs.append(self.buf_v[b, h_kv].astype(F64))
        return np.concatenate(ks, axis=0), np.concatenate(vs, axis=0)

    def decode_attn(self, q16, scale=None):
        """Eq. 1 for one query per sequence: out[b, h] = softmax(q K^^T * scale) V^,
        scale = 1/sqrt(d_H) unless given; query head h reads kv head
        h // (H_q / H_kv).  No mask: the query attends to every cached token."""
        q = np.asarray(q16, F16).astype(F64)
        scale = 1.0 / np.sqrt(self.d) if scale is None or scale <= 0 else float(scale)
        rep = self.Hq // self.Hkv
        out = np.zeros((self.B, self.Hq, self.d), F64)
        for b in range(self.B):
            for hk in range(self.Hkv):
                k_hat, v_hat = self.materialise(b, hk)
                for h in range(hk * rep, (hk + 1) * rep):
                    out[b, h] = attention_one(q[b, h], k_hat, v_hat, scale)
        return out


def attention_one(q, k_hat, v_hat, scale):
    """softmax(K^ q * scale)^T V^ with the usual max subtraction."""
    z = (k_hat @ q) * scale
    z = z - np.max(z)
    p = np.exp(z)
    p = p / np.sum(p)
    return p @ v_hat


# --------------------------------------------------------------------------
# byte accounting of a compressed cache (what the method must keep / move)
# --------------------------------------------------------------------------
def algorithmic_bytes_per_token_head(d_h, bits, g_k, g_v, k_k, k_v, rank):
    """Bytes per (token, kv head), keys and values together: b-bit codes,
    fp16 scale + zero per group, outliers as (fp16 value, 8-bit index), and
    one fp16 row of A per side."""
    codes = 2 * d_h * bits / 8.0
    sz = d_h * 4.0 / g_k + (d_h / g_v) * 4.0
    outl = (d_h / g_k) * 2 * k_k * 3.0 + (d_h / g_v) * 2 * k_v * 3.0
    low = 2 * rank * 2.0
    return codes + sz + outl + low
