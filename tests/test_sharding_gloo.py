"""Multi-rank host logic on CPU: two gloo ranks take their matrices and agree on the max time."""
import os
import socket

import torch.multiprocessing as mp

from paper_2503_13089_b200 import sharding
from paper_2503_13089_b200 import workloads as wl


def test_assign_matrices_balances_and_covers():
    w = wl.WORKLOADS["cfg5_layer7b_g16_k65536"]
    sizes = [w.n_subvectors(m) for m in w.matrices]
    for world in (1, 2, 3, 8):
        parts = sharding.assign_matrices(sizes, world)
        assert sorted(i for p in parts for i in p) == list(range(7))
        loads = [sum(sizes[i] for i in p) for p in parts]
        assert max(loads) <= sum(sizes) / world + max(sizes)
    assert sharding.matrices_for_rank(w, 0) == w.matrices
    r1 = sharding.matrices_for_rank(w, 1)
    assert [m.name for m in r1] == [m.name for m in w.matrices]
    assert all(a.data_seed != b.data_seed for a, b in zip(r1, w.matrices))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import torch
    from paper_2503_13089_b200 import binding as cc
    w = wl.WORKLOADS["cfg1_256x512_g4_k256"]
    specs = sharding.matrices_for_rank(w, rank)
    W = wl.make_matrix(specs[0])
    t = sharding.max_over_ranks(10.0 + rank)          # a stand-in for the rank's device time
    # the benchmark's split of a job over the ranks: `world` copies of a 7B layer's matrices through the
    # library's scheduler; the ranks exchange their shares and each checks that they partition the job
    layer = wl.WORKLOADS["cfg5_layer7b_g16_k65536"]
    job = [m for r in range(world) for m in sharding.matrices_for_rank(layer, r)]
    sizes = [layer.n_subvectors(m) for m in job]
    mine = cc.cc_schedule_matrices(sizes, world, rank)
    flags = torch.zeros(len(job), dtype=torch.int64)
    flags[mine] = 1
    dist.all_reduce(flags)
    load = torch.tensor([float(sum(sizes[i] for i in mine))], dtype=torch.float64)
    loads = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(loads, load)
    out.put((rank, specs[0].data_seed, float(W.astype("float32").sum()), t, bool((flags == 1).all()),
             [float(v) for v in loads], float(sum(sizes))))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_different_matrices_and_share_max_time():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] != res[1][1] and res[0][2] != res[1][2]      # different seeds, different data
    assert res[0][3] == res[1][3] == 11.0                          # both see the slower rank's time
    assert res[0][4] and res[1][4]                                 # every matrix of the job went to exactly one rank
    loads, total = res[0][5], res[0][6]
    assert res[1][5] == loads and sum(loads) == total
    assert max(loads) - min(loads) <= 2818048                      # balanced to within the largest matrix
