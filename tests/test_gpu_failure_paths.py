"""Failure paths, made without faulting, trapping or hanging the GPU.

* A bounded wait that runs out: a test switch makes the decode kernel wait, with a limit of a few dozen polls, on a
  barrier that nothing completes.  The kernel must return on its own, the status word must read GEAR_ERR_TIMEOUT,
  and the very next ordinary call on the same cache must match the oracle again.
* A device allocation that fails: an allocator installed through gear_set_allocator returns NULL on its k-th call;
  gear_create must report GEAR_ERR_ALLOC and hand back every block it had taken.
"""
import ctypes as C

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_sets_the_status_word_and_the_cache_recovers():
    import torch
    from tests.gear_harness import Pair
    from paper_2403_05527_b200 import binding as G, synth

    for hq, hkv in ((2, 2), (8, 2)):
        p = Pair(13, 2, hq, hkv, 2, 64, 2.0, 64, 4, 1024)
        try:
            p.compress(256, 4)
            p.append(70)
            p.check_attention()                                 # clean before
            q = torch.from_numpy(synth.make_query(13, 2, hq, 128)).to(p.dev)
            out = torch.full((2, hq, 128), float("nan"), dtype=torch.float32, device=p.dev)
            G.gear_test_dead_wait(p.cache, True)
            G.gear_decode_attn(p.cache, q, out)                 # returns by itself: every wait is bounded
            torch.cuda.synchronize()
            assert G.gear_last_device_status(p.cache) == G.GEAR_ERR_TIMEOUT
            assert G.gear_last_device_status(p.cache) == 0      # reading clears the word
            G.gear_test_dead_wait(p.cache, False)
            p.check_attention(extra=3)                          # and the same cache is good again
            p.append(5)
            p.check_attention(extra=4)
        finally:
            p.close()


def test_status_word_of_the_fp16_entry_points_is_readable():
    import torch
    from paper_2403_05527_b200 import binding as G, synth

    dev = torch.device("cuda:0")
    B, Hq, Hkv, n = 1, 4, 2, 100
    k16, v16 = synth.make_kv(2, B, Hkv, n, 128)
    q = synth.make_query(2, B, Hq, 128)
    kd, vd, qd = (torch.from_numpy(x).to(dev) for x in (k16, v16, q))
    scratch = torch.empty(G.gear_fp16_attn_scratch_bytes(B, Hq), dtype=torch.uint8, device=dev)
    out = torch.empty(B, Hq, 128, dtype=torch.float32, device=dev)
    G.gear_fp16_decode_attn(kd, vd, qd, out, B, Hq, Hkv, n, n, scratch)
    assert G.gear_fp16_attn_status(scratch) == 0
    G.gear_fp16_decode_attn_static(kd, vd, qd, out, B, Hq, Hkv, n, n)
    assert G.gear_fp16_attn_static_status() == 0


def test_injected_allocation_failure_is_reported_and_nothing_leaks():
    import torch
    from paper_2403_05527_b200 import binding as G

    torch.cuda.init()
    held = {}
    state = {"calls": 0, "fail_at": -1}

    def alloc(nbytes, _ctx):
        state["calls"] += 1
        if state["calls"] == state["fail_at"]:
            return None
        t = torch.empty(max(int(nbytes), 1), dtype=torch.uint8, device="cuda:0")
        held[t.data_ptr()] = t
        return t.data_ptr()

    def free(ptr, _ctx):
        assert ptr in held, "freed a pointer the allocator did not hand out"
        del held[ptr]

    a_cb, f_cb = G.ALLOC_FN(alloc), G.FREE_FN(free)
    cfg = G.make_config(1, 2, 2, 2, 64, 2.0, 64, 4, 512)
    G.gear_set_allocator(a_cb, f_cb)
    try:
        cache = G.gear_create(cfg)                  # count the allocations of a clean create
        total = state["calls"]
        assert total >= 8 and len(held) == total
        G.gear_free(cache)
        assert not held
        for k in (1, 3, total):                     # first, an early one, the last
            state.update(calls=0, fail_at=k)
            with pytest.raises(G.GearError) as e:
                G.gear_create(cfg)
            assert e.value.status == G.GEAR_ERR_ALLOC
            assert not held, f"allocation {k} failed and {len(held)} blocks were not handed back"
    finally:
        G.gear_set_allocator(None, None)
    cache = G.gear_create(cfg)                      # the default allocator is back
    G.gear_free(cache)
