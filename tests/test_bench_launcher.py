"""Host logic of bench.py: what `--gpus N` does before any device is touched (argv in, command out)."""
import os
import sys

import bench


def test_single_gpu_runs_in_this_process():
    assert bench.launch_command(1, {}, ["--steps", "3"], device_count=1, port=1234) == ("run", None)
    assert bench.launch_command(1, {}, [], device_count=8, port=1234) == ("run", None)


def test_n_gpus_start_n_ranks_on_this_file():
    what, cmd = bench.launch_command(4, {}, ["--gpus", "4", "--steps", "7", "--warmup", "3"], device_count=8, port=29511)
    assert what == "exec"
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nnodes=1" in cmd and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "29511"
    i = cmd.index(os.path.abspath(bench.__file__))
    assert cmd[i + 1:] == ["--gpus", "4", "--steps", "7", "--warmup", "3"]       # every rank sees the same arguments


def test_too_few_devices_is_refused_with_the_count():
    what, msg = bench.launch_command(2, {}, ["--gpus", "2"], device_count=1, port=1)
    assert what == "error" and "--gpus 2" in msg and "1 CUDA device" in msg


def test_inside_a_launcher_the_rank_count_must_match():
    env = {"WORLD_SIZE": "4", "RANK": "1", "LOCAL_RANK": "1"}
    assert bench.launch_command(4, env, [], device_count=4, port=1) == ("run", None)   # already a rank: no second launch
    what, msg = bench.launch_command(8, env, [], device_count=8, port=1)
    assert what == "error" and "WORLD_SIZE=4" in msg
    assert bench.launch_command(1, {"WORLD_SIZE": "1"}, [], device_count=1, port=1) == ("run", None)


def test_free_port_is_usable():
    p = bench.free_port()
    assert 1024 < p < 65536


def _rank_worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # what a rank contributes: its own timed interval and its own token count
        ms = bench.reduce_over_ranks(dist, "cpu", 7.0 + rank, "max")
        tokens = bench.reduce_over_ranks(dist, "cpu", 1000.0 * (rank + 1), "sum")
        out.put((rank, ms, tokens))
    finally:
        dist.destroy_process_group()


def test_timing_is_the_maximum_and_tokens_the_sum_over_ranks():
    """Two ranks (gloo, CPU): the step time of the job is the slowest rank's, the tokens are everyone's."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = bench.free_port()
    procs = [ctx.Process(target=_rank_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 8.0, 3000.0), (1, 8.0, 3000.0)]
    assert bench.reduce_over_ranks(None, "cpu", 5.5, "max") == 5.5
