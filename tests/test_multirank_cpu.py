"""The N > 1 path on CPU: two gloo ranks shard a set of layers, run the host-side bookkeeping of the benchmark
(partition, max-over-ranks of the time, gather of per-layer results) and agree on the outcome.  The GPU work
itself needs no exchange (layers are independent problems), so nothing else crosses ranks."""
import os
import socket

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist  # noqa: E402
import torch.multiprocessing as mp  # noqa: E402


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, n_layers, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2511_19705_b200 import shard
    mine = shard.layers_of_rank(n_layers, world, rank)
    local = {layer: dict(rank=rank, loss=float(layer) * 0.5) for layer in mine}
    t = shard.max_over_ranks(10.0 + rank)               # rank 1 is the slower one
    everything = shard.gather_results(local)
    dist.barrier()
    q.put((rank, mine, t, sorted(everything.keys()), everything[n_layers - 1]["rank"]))
    dist.destroy_process_group()


def test_two_ranks_shard_layers_and_reduce_time():
    world, n_layers = 2, 7
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n_layers, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, l0, t0, k0, o0), (r1, l1, t1, k1, o1) = got
    assert l0 == [0, 2, 4, 6] and l1 == [1, 3, 5]            # disjoint, complete
    assert t0 == t1 == 11.0                                  # the slowest rank's time, on both ranks
    assert k0 == k1 == list(range(n_layers))
    assert o0 == o1 == (n_layers - 1) % world


def test_partition_properties():
    from paper_2511_19705_b200 import shard
    for world in (1, 2, 3, 8):
        seen = []
        for r in range(world):
            seen += shard.layers_of_rank(42, world, r)
        assert sorted(seen) == list(range(42))
    with pytest.raises(ValueError):
        shard.layers_of_rank(4, 2, 2)
    assert shard.max_over_ranks(3.5) == 3.5                  # no process group: identity
