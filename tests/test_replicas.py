"""The multi-GPU path is replicas only; its rank plumbing is exercised here with two gloo ranks on CPU."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2607_21624_b200.replicas import Replicas
    rep = Replicas(backend="gloo")
    rep.barrier()
    ms, ms_e2e = rep.max_over_ranks([1.0 + rank, 5.0 - rank])      # rank 1 is slower on the first, rank 0 on the second
    rate = rep.whole_job_rate(1000.0, ms)
    rep.barrier()
    out.put((rank, ms, ms_e2e, rate, rep.world))
    rep.close()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_whole_job_rate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, ms_e2e, rate, world in got:
        assert world == 2
        assert ms == 2.0 and ms_e2e == 5.0                 # maxima over ranks, identical on both ranks
        assert rate == 2 * 1000.0 / 2.0e-3                 # both replicas' units over the slowest rank's time


def test_single_process_needs_no_process_group():
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    from paper_2607_21624_b200.replicas import Replicas
    rep = Replicas(backend="gloo")
    assert rep.world == 1 and rep.dist is None
    assert rep.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]
    assert rep.whole_job_rate(10.0, 1.0) == 10.0 / 1e-3
    rep.barrier()
    rep.close()


def _self_spawned(path):
    from paper_2607_21624_b200.replicas import Replicas
    rep = Replicas(backend="gloo")
    ms, = rep.max_over_ranks([10.0 * (rep.rank + 1)])
    with open(f"{path}.{rep.rank}", "w") as f:
        f.write(f"{rep.world} {rep.local_rank} {ms} {rep.whole_job_rate(7.0, ms)}")
    rep.barrier()
    rep.close()


def test_replicas_started_without_a_launcher(tmp_path):
    # `bench.py --gpus N` outside torchrun starts its own ranks through spawn_replicas; here with two gloo ranks
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        os.environ.pop(k, None)
    from paper_2607_21624_b200.replicas import spawn_replicas
    base = str(tmp_path / "out")
    spawn_replicas(2, _self_spawned, base)
    for rank in range(2):
        world, local_rank, ms, rate = open(f"{base}.{rank}").read().split()
        assert int(world) == 2 and int(local_rank) == rank
        assert float(ms) == 20.0 and float(rate) == 2 * 7.0 / 20.0e-3
    assert "WORLD_SIZE" not in os.environ            # the parent's environment is left alone
