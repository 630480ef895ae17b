"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The hot path has no exchange step (every
(layer, sequence, KV head) unit is independent), so several GPUs run replicas; what the ranks share is the timing
rule -- the slowest rank's time counts, and the value is the whole job's."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group(backend="gloo", rank=rank, world_size=world)
    mine = [10.0 + 5.0 * rank, 7.0 - rank]                  # rank 1 is slower on the first, faster on the second
    got = bench.max_over_ranks(mine, dist, torch.device("cpu"))
    dist.barrier()
    q.put((rank, got, bench.whole_job_value(16, 576, world, got[0])))
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time_and_the_whole_job_value():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, value in res:
        assert got == [15.0, 7.0]
        assert value == pytest.approx(2 * 16 * 576 / 15e-3)


def _stub_replica(args):
    """What a replica does around its measurement, without a GPU: join the job from the environment that
    spawn_replicas prepared, agree on the slowest time, and let rank 0 write the line."""
    sys.path.insert(0, ROOT)
    import json
    import bench
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert int(os.environ["LOCAL_RANK"]) == rank
    dist.init_process_group(backend="gloo")
    ms = bench.max_over_ranks([100.0 + 50.0 * rank], dist, torch.device("cpu"))[0]
    dist.barrier()
    if rank == 0:
        with open(args["out"], "w") as f:
            json.dump({"n_gpus": world, "ms_per_step": ms, "value": bench.whole_job_value(16, 576, world, ms)}, f)
    dist.destroy_process_group()


def test_gpus_flag_without_a_launcher_starts_the_replicas(tmp_path):
    sys.path.insert(0, ROOT)
    import json
    import bench
    out = tmp_path / "line.json"
    bench.spawn_replicas(2, _stub_replica, {"out": str(out)})
    line = json.loads(out.read_text())
    assert line["n_gpus"] == 2 and line["ms_per_step"] == 150.0
    assert line["value"] == pytest.approx(2 * 16 * 576 / 0.150)


def test_single_process_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.5, 1.0], None, torch.device("cpu")) == [3.5, 1.0]
    assert bench.whole_job_value(16, 576, 1, 339.0) == pytest.approx(16 * 576 / 0.339)
