"""World-size-2 check (gloo, CPU) of the benchmark's multi-rank host logic: the path has no exchange step, so
ranks are independent replicas and only the timing is reduced (max over ranks) and the value aggregated."""
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank),
                      WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    bench.barrier(world)
    t = bench.max_over_ranks(local_ms, world, torch.device("cpu"))
    # every rank restores its own copy of the workload: whole-job value = world * per-rank bytes / max time
    value = bench.aggregate_value(1.0e9, t, world)
    out[rank] = (t, value)
    dist.destroy_process_group()


def test_two_ranks_reduce_time_by_max_and_scale_value_by_world_size():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0] == out[1]
    t, value = out[0]
    assert t == 15.0
    assert abs(value - 2 * 1.0e9 / 15.0e-3 / 1e9) < 1e-9


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5
    assert abs(bench.aggregate_value(2.0e9, 4.0, 1) - 0.5e3) < 1e-9


def test_both_arms_print_the_same_config_object():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.workload_config(429, 1) == bench.workload_config(429, 1)
    assert bench.workload_config(429, 1)["workload"] == bench.WORKLOAD
    assert "PROFILING SLICE" in bench.workload_config(429, 1, layers=4)["workload"]


def test_traffic_figure_comes_from_the_committed_capture():
    sys.path.insert(0, ROOT)
    import bench
    kv = dict(x.split(" = ") for x in open(bench.TRAFFIC_FILE).read().splitlines() if " = " in x and not x.startswith("#"))
    n = int(kv["block_layers"])
    got, src = bench.captured_traffic(n, int(kv["algorithmic_bytes_written"]))
    # on the captured slice itself the figure is the capture's own read + write bytes
    assert abs(got - (int(kv["dram_bytes_read_per_launch"]) + int(kv["dram_bytes_write_per_launch"]))) <= 1
    assert kv["capture"] in src


def test_clock_samples_are_binned_by_block():
    sys.path.insert(0, ROOT)
    import bench
    s = bench.ClockSampler(0)
    s.proc = None
    s.lines = [(100.0, "0, 1965, 1965, 400.0, 0x0, Not Active, Not Active, Not Active, Not Active"),
               (100.5, "0, 1800, 1965, 900.0, 0x4, Not Active, Not Active, Not Active, Active")]
    rows = s.rows(99.9, 100.6)
    assert [r[1] for r in rows] == [1965.0, 1800.0] and rows[1][3] == ["sw_power_cap"]
