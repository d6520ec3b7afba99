"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job value,
independent replicas (different seeds, no data-path collective)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import workloads as W
    w = bench.rank_workload(W.CONFIGS["c1"], rank, 40)
    k, _ = W.kv_tokens(w, 0, 0, 0, 8)
    # each rank "measures" a different time; everyone must end up with the slowest one
    elapsed, other = bench.allreduce_max([10.0 + 5.0 * rank, 3.0 - rank])
    dist.barrier()
    out[rank] = (w.seed, w.steps, float(k.float().sum()), elapsed, other,
                 bench.aggregate_value(8 * 128, world, elapsed))
    dist.destroy_process_group()


def test_two_gloo_ranks_max_timing_and_replica_seeds():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] != r1[0] and r0[1] == r1[1] == 40          # own seed per replica, same shape
    assert r0[2] != r1[2]                                    # so the replicas hold different data
    assert r0[3] == r1[3] == 15.0 and r0[4] == r1[4] == 3.0  # max over ranks, on every rank
    assert r0[5] == r1[5] == 8 * 128 * 2 / 15e-3             # units of all ranks / slowest time


def test_single_process_is_identity():
    import bench
    assert bench.allreduce_max([1.5, 2.5]) == [1.5, 2.5]
    assert bench.aggregate_value(100, 1, 1000.0) == 100.0


def test_cpu_list_parsing_and_binding_is_a_no_op_without_locality(tmp_path):
    """The NUMA helper: cpulist syntax; a device whose local CPUs are all of the allowed ones (a
    single-node host) or whose sysfs entry is missing leaves the affinity alone."""
    import os
    import types
    import bench
    assert bench.parse_cpulist("0-3,8,10-11\n") == [0, 1, 2, 3, 8, 10, 11]
    assert bench.parse_cpulist("5") == [5]
    before = os.sched_getaffinity(0)
    props = types.SimpleNamespace(pci_domain_id=0, pci_bus_id=0x1b, pci_device_id=0)
    r = bench.bind_near_gpu(props, sysfs=str(tmp_path))                      # no such device
    assert r["bound"] is False and os.sched_getaffinity(0) == before
    d = tmp_path / "0000:1b:00.0"
    d.mkdir()
    (d / "local_cpulist").write_text(",".join(str(c) for c in sorted(before)) + "\n")
    r = bench.bind_near_gpu(props, sysfs=str(tmp_path))                      # every allowed CPU is local
    assert r["bound"] is False and os.sched_getaffinity(0) == before
    if len(before) > 1:
        keep = sorted(before)[:1]
        (d / "local_cpulist").write_text(str(keep[0]) + "\n")
        try:
            r = bench.bind_near_gpu(props, sysfs=str(tmp_path))
            assert r == {"bound": True, "local_cpus": 1} and os.sched_getaffinity(0) == set(keep)
        finally:
            os.sched_setaffinity(0, before)
