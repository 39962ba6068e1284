"""The multi-GPU arm of bench.py is N independent replicas; its only cross-rank logic is the max over
ranks of the timings and the aggregate value.  Checked here with two gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    got = bench.max_over_ranks([1.0 + rank, 10.0 - rank, 5.0], device="cpu")
    dist.barrier()
    out[rank] = got
    dist.destroy_process_group()


def test_max_over_ranks_with_two_gloo_ranks():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == [2.0, 10.0, 5.0] and out[1] == [2.0, 10.0, 5.0]


def test_single_process_and_aggregate_value():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], device="cpu") == [3.0, 4.0]
    assert bench.replica_value(2.0, 1) == 2000.0
    assert bench.replica_value(2.0, 8) == 250.0  # eight replicas finish eight steps in the time of one


def test_gpus_flag_starts_the_replicas_itself(tmp_path):
    """`bench.py --gpus 2` without torchrun's environment starts two processes with the environment torchrun would have
    given them; here the two run a stand-in script that joins a gloo group on the CPU and takes the maximum over ranks
    with the benchmark's own helper."""
    sys.path.insert(0, ROOT)
    import bench
    script = tmp_path / "replica.py"
    script.write_text(
        "import os, sys\n"
        "sys.path.insert(0, %r)\n"
        "import torch.distributed as dist\n"
        "import bench\n"
        "rank, world = int(os.environ['RANK']), int(os.environ['WORLD_SIZE'])\n"
        "assert os.environ['LOCAL_RANK'] == os.environ['RANK'] and os.environ['MASTER_ADDR'] == '127.0.0.1'\n"
        "dist.init_process_group('gloo', rank=rank, world_size=world)\n"
        "got = bench.max_over_ranks([float(rank), 7.0], device='cpu')\n"
        "dist.barrier()\n"
        "open(os.path.join(sys.argv[1], 'rank%%d.txt' %% rank), 'w').write('%%d %%s' %% (world, got))\n"
        "dist.destroy_process_group()\n" % ROOT)
    assert bench.spawn_replicas(2, [str(tmp_path)], script=str(script)) == 0
    assert (tmp_path / "rank0.txt").read_text() == "2 [1.0, 7.0]"
    assert (tmp_path / "rank1.txt").read_text() == "2 [1.0, 7.0]"
    env = bench.replica_env(3, 4, 1234)
    assert (env["RANK"], env["LOCAL_RANK"], env["WORLD_SIZE"], env["MASTER_PORT"]) == ("3", "3", "4", "1234")


def test_reference_arm_runs_on_rank_zero_only(capsys, monkeypatch):
    sys.path.insert(0, ROOT)
    import argparse
    import bench
    monkeypatch.setenv("RANK", "1")
    bench.run_reference(argparse.Namespace())  # returns before touching its arguments
    assert capsys.readouterr().out == ""
