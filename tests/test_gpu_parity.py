"""GPU parity: the CUDA path (through the C ABI) against the float64 oracle on the same seeded inputs.
Bit-exact on codes, scales, zero-points and outlier sets / values; <= 1e-3 max-norm relative on the low-rank
reconstruction A B^T and on the decode-attention output."""
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


def test_config1_single_head_4bit(pair_factory):
    """Configuration C1: n=256, d_H=128, 4-bit, g=64, s=2 %, r=4, 3 loops, n_b=16, one query."""
    p = pair_factory(1, 1, 1, 1, 4, 64, 2.0, 16, 4, 512)
    p.compress(256, 4)
    p.check_segment(0)
    p.check_attention()
    assert p.append(20) == 1                       # one flush of 16 tokens, 4 left in the buffer
    p.check_segment(1)
    p.check_attention(extra=1)


@pytest.mark.parametrize("bits", [2, 4])
def test_llama_like_slice_with_flushes(pair_factory, bits):
    """A (batch, head) slice of the LLaMA-shaped configs: g=64, n_b=64, several blocks, a flush and a ragged buffer."""
    p = pair_factory(2, 2, 3, 3, bits, 64, 2.0, 64, 4, 1024)
    p.compress(192, 4)
    p.check_segment(0)
    p.check_attention()
    assert p.append(64 + 37) == 1
    p.check_segment(1)
    p.check_attention(extra=2)


def test_config3_like_rank8_s1(pair_factory):
    p = pair_factory(3, 1, 2, 2, 4, 64, 1.0, 64, 8, 1024)
    p.compress(256, 8)
    p.check_segment(0)
    p.append(64)
    p.check_segment(1)
    p.check_attention()


def test_mistral_like_gqa_group128(pair_factory):
    """GQA 4 query heads per kv head, g=128 (k=2 outliers per side), flushes of 64 tokens quantized per whole column."""
    p = pair_factory(4, 1, 8, 2, 2, 128, 2.0, 64, 4, 1024)
    p.compress(384, 4)
    p.check_segment(0)
    p.append(64 + 5)
    p.check_segment(1)
    p.check_attention()


def test_plain_group_quant_and_outlier_only_variants(pair_factory):
    """s = 0, r = 0 is plain group quantization; r = 0 alone is outlier-aware quantization."""
    for s in (0.0, 2.0):
        p = pair_factory(5, 1, 2, 2, 2, 64, s, 64, 0, 512)
        p.compress(128, 0)
        p.check_segment(0)
        p.append(64 + 3)
        p.check_segment(1)
        p.check_attention()
        p.close()


def test_buffer_only_cache_and_ragged_buffer_lengths(pair_factory):
    p = pair_factory(6, 2, 4, 2, 4, 64, 2.0, 64, 2, 256)
    for steps in (1, 15, 1, 16, 7):            # buffer lengths 1, 16, 17, 33, 40
        p.append(steps)
        p.check_attention(extra=steps)


def test_many_query_heads_per_kv_head(pair_factory):
    for hq, hkv in ((8, 1), (16, 1), (6, 2)):  # 8 (two column tiles), 16 (two passes), 3 (odd)
        p = pair_factory(7, 1, hq, hkv, 2, 64, 2.0, 64, 4, 512)
        p.compress(128, 4)
        p.append(10)
        p.check_attention()
        p.close()


def test_rank_variants_and_small_groups(pair_factory):
    p = pair_factory(8, 1, 1, 1, 4, 32, 4.0, 32, 2, 512, r_max=16)
    p.compress(64, 16)
    p.compress(96, 1, extra=1)
    p.compress(32, 3, extra=2)
    for si in range(3):
        p.check_segment(si)
    p.append(32)
    p.check_segment(3)
    p.check_attention(scale=0.05)


def test_many_small_segments_and_state_errors(pair_factory):
    from paper_2403_05527_b200 import binding as G
    import torch
    p = pair_factory(9, 1, 2, 2, 2, 64, 2.0, 16, 2, 160)
    p.compress(64, 2)
    assert p.append(16 * 5 + 3) == 5
    p.check_attention()
    info = G.gear_cache_info(p.cache)
    assert (info.n_segments, info.buffer_len, info.n_compressed) == (6, 3, 144)
    # compress while the buffer holds tokens is a state error; so is exceeding max_tokens
    z = torch.zeros(1, 2, 64, 128, dtype=torch.float16, device="cuda")
    with pytest.raises(G.GearError) as e:
        G.gear_compress(p.cache, None, z, z, 64, 0)
    assert e.value.status == G.GEAR_ERR_STATE
    p.append(13)                                 # 160 tokens compressed now
    tok = torch.zeros(1, 2, 128, dtype=torch.float16, device="cuda")
    for _ in range(15):
        G.gear_append_buffer(p.cache, tok, tok)
    with pytest.raises(G.GearError) as e:
        G.gear_append_buffer(p.cache, tok, tok)
    assert e.value.status == G.GEAR_ERR_CAPACITY
    with pytest.raises(G.GearError) as e:
        flat = torch.zeros(2 * 128 + 8, dtype=torch.float16, device="cuda")
        G.gear_decode_attn(p.cache, flat[1:], tok.float())           # misaligned query pointer
    assert e.value.status == G.GEAR_ERR_ALIGN


def test_byte_accounting_matches_oracle_formula(pair_factory):
    from oracle import gear_oracle as O
    from paper_2403_05527_b200 import binding as G
    p = pair_factory(2, 2, 2, 2, 2, 64, 2.0, 64, 4, 1024)
    p.compress(256, 4)
    b = G.gear_cache_bytes(p.cache)
    per = O.algorithmic_bytes_per_token_head(128, 2, 64, 64, 1, 1, 4)
    assert b.codes + b.scale_zero + b.outliers + b.lowrank_a == per * 256 * 4
    assert b.lowrank_b == 4 * 2 * 128 * 4 * 2
    assert b.stored_total >= b.codes + b.scale_zero + b.outliers + b.lowrank_a + b.lowrank_b


def test_host_buffer_entry_points(pair_factory):
    from paper_2403_05527_b200 import binding as G, synth
    p = pair_factory(2, 1, 2, 2, 2, 64, 2.0, 64, 4, 512)
    p.compress(128, 4)
    ks, vs = synth.make_appended(2, 1, 2, 128, 3)
    for i in range(3):
        p.oracle.append(ks[i], vs[i], None)
        G.gear_append_buffer_host(p.cache, ks[i], vs[i])
    q = synth.make_query(2, 1, 2, 128)
    out = np.zeros((1, 2, 128), np.float32)
    G.gear_decode_attn_host(p.cache, q, out)
    ref = p.oracle.decode_attn(q)
    assert np.abs(out - ref).max() / np.abs(ref).max() <= 1e-3
    # the queued form: nothing is valid before the wait, the same bits after it
    out2 = np.zeros((1, 2, 128), np.float32)
    G.gear_decode_attn_host_async(p.cache, q, out2)
    G.gear_cache_wait(p.cache)
    assert np.array_equal(out, out2)
    # push and attend in one call
    k1, v1 = synth.make_appended(2, 1, 2, 128, 4)
    p.oracle.append(k1[3], v1[3], None)
    out3 = np.zeros((1, 2, 128), np.float32)
    assert G.gear_step_host(p.cache, k1[3], v1[3], q, out3) == G.GEAR_OK
    G.gear_cache_wait(p.cache)
    ref3 = p.oracle.decode_attn(q)
    assert np.abs(out3 - ref3).max() / np.abs(ref3).max() <= 1e-3
    assert G.gear_cache_info(p.cache).buffer_len == 4


def test_fp16_cache_attention_against_textbook():
    import torch
    from paper_2403_05527_b200 import binding as G, synth
    B, Hq, Hkv, n, n_alloc = 2, 8, 2, 333, 400
    k16, v16 = synth.make_kv(2, B, Hkv, n_alloc, 128)
    q = synth.make_query(2, B, Hq, 128)
    dev = torch.device("cuda:0")
    scratch = torch.empty(G.gear_fp16_attn_scratch_bytes(B, Hq), dtype=torch.uint8, device=dev)
    out = torch.empty(B, Hq, 128, dtype=torch.float32, device=dev)
    G.gear_fp16_decode_attn(torch.from_numpy(k16).to(dev), torch.from_numpy(v16).to(dev), torch.from_numpy(q).to(dev),
                            out, B, Hq, Hkv, n, n_alloc, scratch)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    for b in range(B):
        for h in range(Hq):
            kk, vv = k16[b, h // 4, :n].astype(np.float64), v16[b, h // 4, :n].astype(np.float64)
            z = kk @ q[b, h].astype(np.float64) / np.sqrt(128.0)
            w = np.exp(z - z.max()); w /= w.sum()
            ref = w @ vv
            assert np.abs(got[b, h] - ref).max() / np.abs(ref).max() <= 1e-3


def test_ties_and_constant_groups_follow_the_fixed_tie_break(pair_factory):
    """Inputs drawn from a handful of values (plus constant rows and columns): almost every group has ties among
    its extremes, and some groups are constant.  Outlier sets and codes must still match the oracle bit for bit:
    larger value first, then lower index; the top entry chosen before the bottom one."""
    import torch
    from paper_2403_05527_b200 import binding as G
    for bits, group, s_pct, n in ((2, 64, 2.0, 128), (4, 32, 4.0, 64), (2, 128, 2.0, 256)):
        p = pair_factory(11, 1, 2, 2, bits, group, s_pct, 64 if group != 32 else 32, 2, 512, r_max=2)
        gen = np.random.default_rng(bits * 100 + group)
        k16 = gen.choice(np.array([-2.0, -0.5, 0.0, -0.0, 0.25, 1.0, 3.0], np.float16), size=(1, 2, n, 128))
        v16 = gen.choice(np.array([-1.0, 0.0, 0.5, 0.5, 2.0], np.float16), size=(1, 2, n, 128))
        k16[0, 0, :, 5] = np.float16(1.5)            # a constant key column (one constant group per block)
        v16[0, 1, 7, :] = np.float16(-0.75)          # a constant value row
        b0 = gen.standard_normal((1, 2, 2, 128, 2)).astype(np.float32)
        p.oracle.compress(k16, v16, 2, b0)
        dev = p.dev
        G.gear_compress(p.cache, None, torch.from_numpy(k16).to(dev), torch.from_numpy(v16).to(dev), n, 2,
                        torch.from_numpy(b0).to(dev))
        torch.cuda.synchronize()
        p.check_segment(0)
        p.check_attention()
        p.close()


@pytest.mark.parametrize("bits,group,s_pct,hq,hkv,nb,rank", [(4, 16, 10.0, 8, 1, 16, 2), (2, 16, 0.0, 2, 2, 32, 1),
                                                              (2, 128, 5.0, 16, 2, 128, 8), (4, 32, 6.0, 3, 3, 64, 16)])
def test_unusual_groupings_head_counts_and_ranks(pair_factory, bits, group, s_pct, hq, hkv, nb, rank):
    """The less common corners of the parameter space: 16- and 32-channel value groups (eight and four groups per
    token), eight query heads per kv head, the largest rank, many outliers per group."""
    p = pair_factory(12, 1, hq, hkv, bits, group, s_pct, nb, min(rank, nb), 1024, r_max=rank)
    n = 2 * max(group, 64)
    p.compress(n, rank)
    p.check_segment(0)
    p.append(nb + 3)
    p.check_segment(1)
    p.check_attention()
