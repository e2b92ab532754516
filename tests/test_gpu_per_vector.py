"""Per-vector grouping (Section 2, "Group-wise Quantization"; the KCVT backbone of Section 4): one key group per
channel over the whole segment, one value group per token, Filter_s (Eq. 4) on those whole vectors.  The CUDA path
(C ABI, group = GEAR_GROUP_PER_VECTOR) against the float64 oracle run with a group length no vector reaches:
bit-exact on codes, scales, zero-points and outlier sets / values, <= 1e-3 on the low-rank product and on attention."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture
def pair_factory():
    from tests.gear_harness import Pair
    made = []

    def make(*a, **k):
        p = Pair(*a, **k)
        made.append(p)
        return p
    yield make
    for p in made:
        if p.cache is not None:
            p.close()


def test_four_bit_prefill_of_4096_tokens_then_flushed_buffers(pair_factory):
    """The paper's 4-bit setting (s = 2 %, r = 4) at n = 4096: 41 entries per side leave every key channel."""
    from paper_2403_05527_b200 import binding as G
    p = pair_factory(2, 1, 4, 2, 4, 0, 2.0, 32, 2, 4096 + 128, r_max=4)
    p.compress(4096, 4)
    si = G.gear_segment_info_get(p.cache, 0)
    assert (si.g_k, si.k_k, si.g_v, si.k_v) == (4096, 41, 128, 2)
    p.check_segment(0)
    p.check_attention()
    assert p.append(40) == 1                      # one flushed 32-token segment (a key group = its 32 tokens), 8 buffered
    si = G.gear_segment_info_get(p.cache, 1)
    assert (si.g_k, si.k_k) == (32, 1)
    p.check_segment(1)
    p.check_attention(extra=1)


@pytest.mark.parametrize("bits,group,n,hq,r_flush", [(4, 0, 1024, 4, 2), (2, 64, 256, 4, 2), (4, 128, 128, 4, 2),
                                                     (4, 0, 1024, 2, 4), (2, 128, 256, 2, 4), (2, 64, 256, 2, 3)])
def test_buffer_of_twenty_tokens(pair_factory, bits, group, n, hq, r_flush):
    """n_b = 20 (Section 4, "Implementation details"): a flushed buffer is one block of 20 tokens, a key group its
    20 tokens of a channel; the record keeps two 16-token slabs, the second one partly empty."""
    from paper_2403_05527_b200 import binding as G
    p = pair_factory(2, 2, hq, 2, bits, group, 2.0, 20, r_flush, n + 100, r_max=4)     # hq = 2: the one-head kernel
    p.compress(n, 4)
    assert p.append(67) == 3                      # three flushed 20-token segments, seven tokens buffered
    for si in (1, 2, 3):
        info = G.gear_segment_info_get(p.cache, si)
        assert (info.n_c, info.g_k, info.k_k) == (20, 20, 1)
        p.check_segment(si)
    p.check_attention(extra=3)
    assert p.append(13) == 1                      # the buffer is empty right after a flush
    p.check_segment(4)
    p.check_attention(extra=4)


@pytest.mark.parametrize("bits,n,s,rank", [(2, 512, 2.0, 2), (4, 1024, 5.0, 0), (2, 192, 0.0, 4), (4, 8192, 1.0, 2)])
def test_other_shapes(pair_factory, bits, n, s, rank):
    p = pair_factory(3, 2, 2, 2, bits, 0, s, 64, 2, n + 128, r_max=max(rank, 2))
    p.compress(n, rank)
    p.check_segment(0)
    p.check_attention()
    p.append(70)
    p.check_segment(1)
    p.check_attention(extra=2)


def test_ties_go_to_the_lower_token(pair_factory):
    """Keys drawn from a handful of values: the thresholds of Filter_s sit inside long runs of equal entries, and a
    channel that is constant has its k largest and k smallest in the first 2k tokens."""
    import torch
    from oracle import gear_oracle as O
    from paper_2403_05527_b200 import binding as G, synth
    B, H, n = 1, 2, 512
    rng = np.random.default_rng(7)
    k16 = rng.choice(np.array([-1.5, -0.25, 0.0, 0.25, 2.0], np.float16), size=(B, H, n, 128))
    k16[:, :, :, 5] = np.float16(0.75)            # a constant channel
    k16[:, :, ::7, 9] = np.float16(-0.0)          # both zeros in one channel
    _, v16 = synth.make_kv(3, B, H, n, 128)
    p = pair_factory(3, B, H, H, 4, 0, 3.0, 64, 0, n + 64, r_max=0)
    p.oracle.compress(k16, v16, 0, None)
    dev = p.dev
    G.gear_compress(p.cache, None, torch.from_numpy(k16).to(dev), torch.from_numpy(v16).to(dev), n, 0, None)
    torch.cuda.synchronize()
    p.check_segment(0)
    p.check_attention()
    assert O.outlier_count(3.0, n) == 8


def test_limits_are_errors(pair_factory):
    import torch
    from paper_2403_05527_b200 import binding as G
    with pytest.raises(G.GearError):              # a buffer longer than one block of per-vector keys
        G.gear_create(G.make_config(1, 1, 1, 4, 0, 2.0, 256, 0, 1024))
    cfg = G.make_config(1, 1, 1, 4, 0, 2.0, 64, 0, 16384)
    cache = G.gear_create(cfg)
    try:
        x = torch.zeros(1, 1, 16384, 128, dtype=torch.float16, device="cuda:0")
        with pytest.raises(G.GearError):          # longer than the select kernel's shared memory holds
            G.gear_compress(cache, None, x, x, 16384, 0, None)
        with pytest.raises(G.GearError):          # not a multiple of the 64-token record block
            G.gear_compress(cache, None, x, x, 208, 0, None)
    finally:
        G.gear_free(cache)


def test_two_long_segments_a_short_one_and_a_buffer(pair_factory):
    """Two prefill calls of per-vector keys (each its own groups and outlier list), a 128-token segment that is a
    single ordinary block, then a flushed buffer and buffered tokens."""
    import torch
    from paper_2403_05527_b200 import binding as G, synth
    p = pair_factory(5, 2, 2, 2, 2, 0, 2.0, 32, 2, 2048, r_max=4)
    p.compress(512, 4)
    p.compress(256, 2, extra=1)
    p.compress(128, 3, extra=2)
    infos = [G.gear_segment_info_get(p.cache, i) for i in range(3)]
    assert [(i.n_c, i.g_k, i.k_k) for i in infos] == [(512, 512, 6), (256, 256, 3), (128, 128, 2)]
    for si in range(3):
        p.check_segment(si)
    p.append(37)
    p.check_segment(3)
    p.check_attention(extra=5)
    b = G.gear_cache_bytes(p.cache)
    assert b.stored_total >= b.codes + b.scale_zero + b.outliers + b.lowrank_a + b.lowrank_b + b.buffer


def test_capacity_of_the_arena_is_an_error_not_a_fault():
    import torch
    from paper_2403_05527_b200 import binding as G
    cfg = G.make_config(1, 1, 1, 4, 0, 2.0, 32, 0, 512)
    cache = G.gear_create(cfg)
    try:
        x = torch.randn(1, 1, 512, 128, device="cuda:0").half()
        G.gear_compress(cache, None, x, x, 512, 0, None)
        with pytest.raises(G.GearError):          # the cache was sized for 512 tokens
            G.gear_compress(cache, None, x, x, 192, 0, None)
        assert G.gear_last_device_status(cache) == 0
    finally:
        G.gear_free(cache)
