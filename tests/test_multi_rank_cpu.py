"""World-size-2 checks of the multi-GPU bench logic on CPU (gloo): every rank draws its own
micro-batch, there is no data-path collective, the time is the max over ranks and the value is the
tokens all ranks processed over that time."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    from paper_2509_06980_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, world, rank)
    spec = synth.scaled(synth.SPECS[1], seed=bench.shard_seed(synth.SPECS[1].seed, rank), len_lo=32, len_hi=32,
                        spans_lo=1, spans_hi=1, obs_lo=2, obs_hi=4)
    tok = synth.make_tokens(spec)
    my_seconds = 0.5 + rank                      # rank 1 is the slow one
    slowest = bench.max_over_ranks(my_seconds, world)
    value = bench.aggregate(len(tok.ids) * 4, world, slowest)
    gathered = [None] * world
    dist.all_gather_object(gathered, (int(tok.ids.sum()), float(tok.rewards.sum()), slowest, value))
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_draw_different_batches_and_report_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    g = out.get()
    assert g[0][0] != g[1][0] and g[0][1] != g[1][1]          # different micro-batches per rank
    assert g[0][2] == g[1][2] == 1.5                          # max over ranks, same on every rank
    assert g[0][3] == g[1][3] == 512 * 4 * 2 / 1.5            # all ranks' tokens over the slowest time


def test_reference_arm_prints_nothing_on_nonzero_ranks(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")

    class A:
        steps, warmup, gpus = 1, 0, 2
    bench.run_reference(A)
    assert capsys.readouterr().out == ""


def test_plain_start_with_several_gpus_becomes_a_launcher_of_that_many_ranks(monkeypatch):
    """`python bench.py --gpus 4` outside torchrun must not time one GPU and call it four: it re-runs
    its own command line as four ranks and hands their exit code on."""
    sys.path.insert(0, ROOT)
    import subprocess
    import pytest
    import bench
    seen = {}

    def fake_call(cmd):
        seen["cmd"] = cmd
        return 7
    monkeypatch.setattr(subprocess, "call", fake_call)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "2", "--warmup", "3"])
    with pytest.raises(SystemExit) as e:
        bench.main()
    assert e.value.code == 7
    cmd = seen["cmd"]
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nnodes=1" in cmd
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4" and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-6:] == ["--gpus", "4", "--steps", "2", "--warmup", "3"] and cmd[-7].endswith("bench.py")


def test_rank_count_that_differs_from_gpus_is_refused(monkeypatch):
    sys.path.insert(0, ROOT)
    import pytest
    import bench
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "8"])
    with pytest.raises(SystemExit) as e:
        bench.main()
    assert "n_gpus" in str(e.value.code)
