"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own replica of the workload
(the attention path has no exchange step), whole-job time = slowest rank, whole-job work = sum."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import oracle
    from workloads import tables

    # every rank builds its own replica, seeded by its rank, exactly as bench.run_mate does
    cfg = tables.CONFIGS["tiny"]
    rows, cols, info = tables.make_structure(cfg, 1234 + rank)
    hv = tables.head_view(cfg)
    pairs = float(oracle.useful_pairs(rows, cols, cfg.P, hv).sum())
    times = torch.tensor([10.0 + rank, 1.0, 2.0 * (rank + 1), 0.5], dtype=torch.float64)
    work = torch.tensor([pairs, float(sum(info["n_valid"]))], dtype=torch.float64)
    t, w = bench.reduce_over_ranks(times, work, world)
    np.save(os.path.join(out_dir, "rank%d.npy" % rank), np.asarray(t + w + [pairs]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_reduction(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0 = np.load(tmp_path / "rank0.npy")
    r1 = np.load(tmp_path / "rank1.npy")
    # both ranks hold the same reduced figures
    assert np.array_equal(r0[:6], r1[:6])
    # times: max over ranks
    assert r0[0] == 11.0 and r0[1] == 1.0 and r0[2] == 4.0 and r0[3] == 0.5
    # work: sum over ranks of the per-rank pair counts (the replicas differ: different seeds)
    assert r0[4] == r0[6] + r1[6]
    assert r0[6] > 0 and r1[6] > 0


def test_single_rank_reduction_is_identity():
    import bench
    t, w = bench.reduce_over_ranks(torch.tensor([3.0, 4.0], dtype=torch.float64),
                                   torch.tensor([5.0], dtype=torch.float64), 1)
    assert t == [3.0, 4.0] and w == [5.0]


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    import bench
    from workloads import tables

    class Args:
        steps, warmup, gpus = 1, 0, 2

    monkeypatch.setenv("RANK", "1")
    bench.run_reference(Args(), tables.CONFIGS["tiny"])
    assert capsys.readouterr().out == ""


def test_gpus_flag_starts_the_ranks_itself(monkeypatch):
    """`python bench.py --gpus 4` without a launcher re-executes itself under torch.distributed.run with four
    ranks on the loopback address; under a launcher (WORLD_SIZE set) it does not."""
    import bench
    seen = {}

    def fake_run(cmd):
        seen["cmd"] = cmd
        return 0

    assert bench.spawn_ranks(["--gpus", "4", "--steps", "5"], 4, run=fake_run) == 0
    cmd = seen["cmd"]
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"]
    assert cmd[cmd.index("--nproc-per-node") + 1] == "4"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert os.path.basename(cmd[cmd.index("--master-port") + 2]) == "bench.py"
    assert cmd[-4:] == ["--gpus", "4", "--steps", "5"]

    # main(): spawns only when no launcher has set WORLD_SIZE
    calls = []
    monkeypatch.setattr(bench, "spawn_ranks", lambda argv, n, run=None: calls.append((argv, n)) or 0)
    monkeypatch.setattr(bench, "run_mate", lambda args, cfg: calls.append("run_mate"))
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2"])
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    try:
        bench.main()
    except SystemExit as e:
        assert e.code == 0
    assert calls == [(["--gpus", "2"], 2)]
    calls.clear()
    monkeypatch.setenv("WORLD_SIZE", "2")
    bench.main()
    assert calls == ["run_mate"]
