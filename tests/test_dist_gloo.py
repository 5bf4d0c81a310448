"""World-size-2 coverage (gloo, CPU) of the benchmark's multi-GPU plumbing: every rank draws its own
microbatch, nothing is exchanged on the data path, times reduce by max and work by sum."""
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
    import bench
    from paper_2607_03229_b200 import dist as D
    r, lr, w = D.init("gloo")
    assert (r, lr, w) == (rank, rank, world)
    wl = bench.workload_for(rank)
    D.barrier()
    (t_max, e_max), (flops, launches) = D.reduce_max_sum([1.0 + rank, 5.0 - rank], [wl.flops(), 5.0])
    # the number of timed regions (each ends in a barrier) must be the same on every rank although their own first
    # regions differ: it is derived from the slowest rank's time
    ms0 = 1.9 if rank == 0 else 2.3
    (ms0_all,), _ = D.reduce_max_sum([ms0], [0.0])
    regions = bench.repeat_count(ms0_all, 200, 2.0)
    assert bench.repeat_count(1.9, 200, 2.0) != bench.repeat_count(2.3, 200, 2.0)   # the local values would disagree
    for _ in range(regions):
        D.barrier()
    out.put((rank, wl.seed, wl.total_tokens, wl.flops(), t_max, e_max, flops, launches, regions))
    D.shutdown()


def test_two_ranks_shard_by_microbatch_and_reduce():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, t0, f0, mx0, ex0, fl0, l0, n0), (r1, s1, t1, f1, mx1, ex1, fl1, l1, n1) = res
    assert n0 == n1 == 5
    assert s0 != s1 and (t0, f0) != (t1, f1)          # different microbatches per rank
    assert mx0 == mx1 == 2.0 and ex0 == ex1 == 5.0    # max over ranks
    assert abs(fl0 - (f0 + f1)) < 1e-3 * fl0 and fl0 == fl1 and l0 == l1 == 10.0   # work sums


def test_single_process_defaults():
    from paper_2607_03229_b200 import dist as D
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert D.env_world() == (0, 0, 1)
    assert D.reduce_max_sum([3.0], [4.0]) == ([3.0], [4.0])
    assert D.rank_seed(7, 0) == 7 and D.rank_seed(7, 3) == 3007


def test_seam_targets_route_every_microbatch_to_the_first_stage():
    from paper_2607_03229_b200 import dist as D
    ship, local = D.seam_targets([3, 0, 1, 3, 0, 2], first_stage_rank=0)
    assert local == [1, 4] and ship == {0: [], 1: [2], 2: [5], 3: [0, 3]}
    ship, local = D.seam_targets([], first_stage_rank=0)
    assert local == [] and ship == {0: []}
    # every microbatch is either local to the first stage or shipped by exactly its owner
    owner = [1, 1, 0, 2]
    ship, local = D.seam_targets(owner, first_stage_rank=1)
    assert sorted(local + [m for v in ship.values() for m in v]) == list(range(len(owner)))
    assert all(owner[m] == r for r, v in ship.items() for m in v) and all(owner[m] == 1 for m in local)


def _reduce_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import torch
    from paper_2607_03229_b200 import dist as D
    D.init("gloo")
    flat, layers = D.alloc_grad_bucket(2, 16, 48, device="cpu")
    # every view is a window of the bucket: writing through the views fills it
    for l, views in enumerate(layers):
        for i, (name, t) in enumerate(views.items()):
            t.fill_(float((rank + 1) * (10 * l + i + 1)))
    before = flat.clone()
    D.dp_reduce(flat)                      # DpReduce(enc, ReplicaGroup): sum over the two replicas
    ok = bool(torch.equal(flat, before * 3 / (rank + 1))) and all(t.data_ptr() % 16 == 0 for v in layers for t in v.values())
    shapes = {k: tuple(v.shape) for k, v in layers[0].items()}
    out.put((rank, ok, shapes["w_qkv"], shapes["w_fc2"], int(flat.numel())))
    D.shutdown()


def test_dp_reduce_sums_the_gradient_bucket_over_replicas():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_reduce_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ok, s_qkv, s_fc2, n in res:
        assert ok and s_qkv == (48, 16) and s_fc2 == (16, 48)
        assert n >= 2 * (4 * 16 * 16 + 2 * 16 * 48)
