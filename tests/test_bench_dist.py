"""N > 1 path of the bench (replicas, no data-path collective): the aggregation over ranks is
max of the times and sum of the bytes.  Two gloo ranks on CPU."""
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
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, e2e, nbytes = bench.aggregate_over_ranks(dist, torch.device("cpu"), 10.0 + rank, 20.0 - rank,
                                                 1000.0 * (rank + 1))
    q.put((rank, ms, e2e, nbytes))
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, e2e, nbytes in res:
        assert ms == 11.0 and e2e == 20.0 and nbytes == 3000.0


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(None, None, 1.5, 2.5, 7.0) == (1.5, 2.5, 7.0)


def test_workload_table_matches_the_benchmark_definition():
    sys.path.insert(0, ROOT)
    import bench
    import synth
    s = bench.workload_shape(bench.DEFAULT_WORKLOAD)
    assert (s.H, s.I, s.E, s.top_k, s.n_shared) == (7168, 2048, 256, 8, 1)
    assert s.bytes_per_expert() == 44050944
    assert bench.WORKLOADS[bench.DEFAULT_WORKLOAD][1] == 64
    for name in bench.WORKLOADS:
        assert bench.workload_shape(name).name in synth.SHAPES
