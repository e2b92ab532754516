"""The N > 1 host logic of bench.py on two CPU ranks (gloo): the path shards by (batch, head) with no data-path
collective, so all that crosses ranks is the timing reduction (max over ranks) and the sum of the shards' work."""
import os
import socket
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        ms = bench.max_over_ranks(local_ms, dist, torch.device("cpu"))
        value = bench.whole_job_tokens_per_s(world, 8, 100, ms * 1e-3)
        ret[rank] = (ms, value)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_report_the_slowest_rank_and_the_summed_work():
    import torch.multiprocessing as mp
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        ret = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, ret), nprocs=world, join=True)
        got = dict(ret)
    assert set(got) == {0, 1}
    for rank in (0, 1):
        ms, value = got[rank]
        assert ms == pytest.approx(15.0)                    # every rank sees the maximum
        assert value == pytest.approx(2 * 8 * 100 / 15e-3)  # whole job: both shards over the slowest time


def test_single_rank_passes_through():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5
    assert bench.whole_job_tokens_per_s(1, 8, 10, 2.0) == 40.0


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"])
    bench.main()
    assert capsys.readouterr().out == ""                   # other ranks exit without work or output


def test_launcher_starts_the_ranks_itself_when_no_launcher_did(tmp_path):
    """`bench.py --gpus N` without torchrun: the ranks are spawned by bench.py, each with its own RANK / LOCAL_RANK /
    WORLD_SIZE and a common rendezvous on 127.0.0.1.  Checked with two CPU ranks on gloo."""
    import json
    sys.path.insert(0, ROOT)
    import bench
    env = bench.rank_environment(1, 2, 12345)
    assert env == {"RANK": "1", "LOCAL_RANK": "1", "WORLD_SIZE": "2", "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": "12345"}
    out = str(tmp_path / "probe")
    bench.spawn_ranks(2, ["bench.py", "--gpus", "2", out], main_name="rank_probe", port=_free_port())
    views = [json.load(open(f"{out}.{r}")) for r in (0, 1)]
    for r, v in enumerate(views):
        assert (v["rank"], v["local_rank"], v["world"]) == (r, r, 2)
        assert v["ms"] == pytest.approx(11.0)                       # every rank sees the slowest rank's time
        assert v["value"] == pytest.approx(2 * 8 * 10 / 11e-3)
