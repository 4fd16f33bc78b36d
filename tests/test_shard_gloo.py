"""The multi-rank plumbing on CPU: world_size 2 over gloo (no GPU, no NCCL)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_26842_b200 import shard, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, shapes, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert shard.env_rank() == (rank, rank, world)
        mine = shard.partition(shapes, world)[rank]
        gathered = [None] * world
        dist.all_gather_object(gathered, [(s.spec, s.start, s.count) for s in mine])
        # every rank derives the same global picture: each matrix owned exactly once
        owned = {}
        for r, lst in enumerate(gathered):
            for spec, start, count in lst:
                for b in range(start, start + count):
                    assert (spec, b) not in owned
                    owned[(spec, b)] = r
        assert len(owned) == sum(s[0] for s in shapes)
        # slowest rank's time decides; whole-job rate counts every rank's units
        slow = shard.max_over_ranks(10.0 + rank, dist)
        assert slow == 10.0 + world - 1
        rate = shard.whole_job_rate(1.0, world, slow)
        dist.barrier()
        q.put((rank, rate, len(mine)))
    finally:
        dist.destroy_process_group()


def test_partition_and_timing_over_two_gloo_ranks():
    wl = synth.workload(2, layers=2)
    shapes = [(s.batch, s.rows, s.cols) for s in wl.specs]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, shapes, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    res = sorted(q.get(timeout=5) for _ in range(2))
    assert [r[0] for r in res] == [0, 1]
    assert res[0][1] == res[1][1] == pytest.approx(2.0 / 11.0)


def _toy_step(w, g):
    """A stand-in for the optimizer step with its one relevant property: every matrix is updated from its own
    weight and gradient only.  (The real step needs a GPU; what is tested here is the sharding around it.)"""
    for b in range(w.shape[0]):
        u = g[b] @ g[b].T @ w[b] if w.shape[1] <= w.shape[2] else w[b] @ (g[b].T @ g[b])
        w[b].mul_(0.999).sub_(u, alpha=0.01)


def _sharded_worker(rank, world, port, shapes, steps, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        gen = torch.Generator().manual_seed(11)             # every rank starts from the same full parameter set
        params = [torch.randn(s, generator=gen) * 0.02 for s in shapes]
        all_shares = shard.partition(shapes, world)
        mine = all_shares[rank]
        assert shard.share_shapes(shapes, mine) == [(sh.count, shapes[sh.spec][1], shapes[sh.spec][2]) for sh in mine]
        received = 0
        for k in range(steps):
            ggen = torch.Generator().manual_seed(100 + k)   # the full gradient; a rank only looks at its share of it
            grads = [torch.randn(s, generator=ggen) * 1e-1 for s in shapes]
            for w, g in zip(shard.local_views(params, mine), shard.local_views(grads, mine)):
                _toy_step(w, g)
            received += shard.exchange(params, all_shares, dist)
        q.put((rank, [p.clone() for p in params], received))
    finally:
        dist.destroy_process_group()


def test_a_partitioned_run_reassembles_to_the_unpartitioned_result():
    """Two gloo ranks each step the matrices `partition()` gives them and exchange the updated slices; after every
    step both hold the same full parameter set, bit-identical to one process stepping everything."""
    shapes = [(5, 8, 12), (3, 12, 8), (1, 16, 16), (1, 4, 16), (2, 8, 8)]
    steps, world = 3, 2
    gen = torch.Generator().manual_seed(11)
    ref = [torch.randn(s, generator=gen) * 0.02 for s in shapes]
    for k in range(steps):
        ggen = torch.Generator().manual_seed(100 + k)
        grads = [torch.randn(s, generator=ggen) * 1e-1 for s in shapes]
        for w, g in zip(ref, grads):
            _toy_step(w, g)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_sharded_worker, args=(r, world, port, shapes, steps, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=120) for _ in range(world)), key=lambda t: t[0])
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    total_bytes = sum(s[0] * s[1] * s[2] * 4 for s in shapes)
    owned = [sum(c * r * cc * 4 for c, r, cc in shard.share_shapes(shapes, sh)) for sh in shard.partition(shapes, world)]
    for rank, params, received in res:
        for got, want in zip(params, ref):
            assert torch.equal(got, want)
        assert received == steps * (total_bytes - owned[rank])


def test_exchange_is_a_no_op_for_one_process():
    shapes = [(2, 4, 4)]
    p = [torch.ones(shapes[0])]
    assert shard.exchange(p, shard.partition(shapes, 1), None) == 0
    assert shard.local_views(p, shard.partition(shapes, 1)[0])[0].data_ptr() == p[0].data_ptr()


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("config", [1, 2, 3])
def test_partition_is_complete_disjoint_and_balanced(world, config):
    wl = synth.workload(config)
    shapes = [(s.batch, s.rows, s.cols) for s in wl.specs]
    shares = shard.partition(shapes, world)
    seen = set()
    for rank in shares:
        for sh in rank:
            assert sh.count >= 1 and 0 <= sh.start and sh.start + sh.count <= shapes[sh.spec][0]
            for b in range(sh.start, sh.start + sh.count):
                assert (sh.spec, b) not in seen
                seen.add((sh.spec, b))
    assert len(seen) == wl.n_matrices
    ld = shard.loads(shapes, shares)
    biggest = max(shard.step_cost(r, c) for _, r, c in shapes)
    assert max(ld) - min(ld) <= biggest * 1.0000001
    assert sum(ld) == pytest.approx(sum(b * shard.step_cost(r, c) for b, r, c in shapes))


def test_single_process_timing_needs_no_process_group():
    assert shard.max_over_ranks(3.5) == 3.5
    assert shard.whole_job_rate(2.0, 4, 0.5) == 16.0
