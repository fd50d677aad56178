"""The multi-rank path of the benchmark on CPU: two gloo ranks agree on the max time, the
summed units and a disjoint, complete sharding of the work."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2008_12260_b200 import dist as pdist


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, lr, w = pdist.init("gloo")
    assert (r, w) == (rank, world)
    pdist.barrier()
    b, e = pdist.shard_range(4097, rank, world)
    thr, t, u = pdist.throughput(100.0 * (rank + 1), e - b)
    pdist.barrier()
    out.put((rank, b, e, thr, t, u))
    torch.distributed.destroy_process_group()


def test_two_ranks_gloo():
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
    (r0, b0, e0, thr0, t0, u0), (r1, b1, e1, thr1, t1, u1) = res
    assert (b0, e0, b1, e1) == (0, 2049, 2049, 4097)
    assert t0 == t1 == 200.0 and u0 == u1 == 4097.0
    assert thr0 == thr1 == 4097.0 / 0.2


def test_shard_range_properties():
    for total in (0, 1, 7, 512, 4096, 4099):
        for world in (1, 2, 3, 8):
            prev = 0
            for r in range(world):
                b, e = pdist.shard_range(total, r, world)
                assert b == prev and e >= b and (e - b) in (total // world, total // world + 1)
                prev = e
            assert prev == total


def test_single_process_passthrough():
    assert pdist.aggregate(12.5, 7) == (12.5, 7.0)
    assert pdist.throughput(500.0, 10)[0] == 20.0


def _fake_children(pop, fit, first, count, g):
    """A stand-in for the GPU generation: child c depends on its index, the generation, and all
    parents (as the real one does), so a wrong gather or slice shows."""
    P = pop.shape[0]
    idx = torch.arange(first, first + count)
    pa = (idx * 7 + g) % P
    pb = torch.argsort(fit, descending=True)[(idx + g) % P]
    return pop[pa] + 2 * pop[pb] + (idx[:, None, None] + g).to(pop.dtype)


def _fake_fitness(children):
    return children.to(torch.float32).sum(dim=(1, 2)) % 101.0


def _evolve_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    pdist.init("gloo")
    g = torch.Generator().manual_seed(5)
    pop = torch.randint(0, 5, (11, 3, 4), generator=g, dtype=torch.int16)      # 11 candidates: uneven slices
    fit = _fake_fitness(pop)
    p, f = pdist.evolve_sharded(_fake_children, _fake_fitness, pop, fit, 4, rank, world)
    out.put((rank, p.numpy().tolist(), f.numpy().tolist()))
    torch.distributed.destroy_process_group()


def test_population_evolved_by_two_ranks_equals_one_process():
    g = torch.Generator().manual_seed(5)
    pop = torch.randint(0, 5, (11, 3, 4), generator=g, dtype=torch.int16)
    fit = _fake_fitness(pop)
    want_p, want_f = pdist.evolve_sharded(_fake_children, _fake_fitness, pop, fit, 4, 0, 1)
    ctx = mp.get_context("spawn")
    for world in (2, 3):
        q = ctx.Queue()
        port = _free_port()
        procs = [ctx.Process(target=_evolve_worker, args=(r, world, port, q)) for r in range(world)]
        for p in procs:
            p.start()
        res = sorted(q.get(timeout=120) for _ in procs)
        for p in procs:
            p.join(timeout=60)
            assert p.exitcode == 0
        for rank, p, f in res:
            assert p == want_p.numpy().tolist() and f == want_f.numpy().tolist()
