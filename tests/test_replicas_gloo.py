"""The N > 1 measurement protocol (barrier, max over ranks, whole-job rate) on CPU with gloo, world size 2."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2512_22195_b200 import replicas
    replicas.barrier()
    ms = 10.0 * (rank + 1)                       # rank 1 is the slow one
    worst = replicas.max_over_ranks(ms)
    rate = replicas.whole_job_rate(units_per_rank=128.0, ms_per_rank=ms)
    out.put((rank, replicas.world(), worst, rate))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_rate_world2():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, world, worst, rate in got:
        assert world == 2 and worst == 20.0
        assert abs(rate - 2 * 128.0 / 0.020) < 1e-6       # both ranks' tokens over the slowest rank's time


def test_single_process_is_identity():
    from paper_2512_22195_b200 import replicas
    assert replicas.world() == 1 and replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_rate(100.0, 50.0) == 2000.0


def _launched_rank(rank, out_dir):
    """What a rank started by `replicas.launch` does in the benchmark, with gloo in place of NCCL and no GPU."""
    from paper_2512_22195_b200 import replicas
    assert int(os.environ["RANK"]) == rank and int(os.environ["LOCAL_RANK"]) == rank
    assert os.environ["WORLD_SIZE"] == "2" and os.environ["MASTER_ADDR"] == "127.0.0.1"
    replicas.init_from_env("gloo")
    replicas.barrier()
    rate = replicas.whole_job_rate(units_per_rank=256.0, ms_per_rank=100.0 * (rank + 1))
    with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
        f.write(f"{replicas.world()} {rate}")
    dist.destroy_process_group()


def test_launch_starts_the_ranks_itself_world2(tmp_path):
    """`bench.py --gpus N` outside torchrun starts its N ranks through `replicas.launch`: the ranks find the rendezvous
    in their environment, join, and report the whole-job rate over the slowest rank's time."""
    from paper_2512_22195_b200 import replicas
    replicas.launch(2, _launched_rank, str(tmp_path))
    for rank in range(2):
        world, rate = open(tmp_path / f"rank{rank}.txt").read().split()
        assert int(world) == 2 and abs(float(rate) - 2 * 256.0 / 0.2) < 1e-6
