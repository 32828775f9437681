"""Head-sharded budgets on two gloo ranks (CPU): each rank has the energy sums of its own KV heads
(computed here by the oracle), one all-reduce makes them whole, and both ranks arrive at the
budgets of the unsharded pass."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

L, H, D, LENS = 3, 4, 8, (40, 0, 25)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _layers():
    rng = np.random.default_rng(3)
    T = sum(LENS)
    Ks = [rng.standard_normal((T, H, D)) * (1.0 + l) for l in range(L)]
    Vs = [rng.standard_normal((T, H, D)) for l in range(L)]
    Ks[1][7] += 20.0
    return Ks, Vs


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from oracle import flashcache_oracle as O
    from paper_2511_16786_b200 import head_shard, replicas
    dist = replicas.init("gloo")
    h0, h1 = head_shard.shard_heads(H, world, rank)
    cu = [0] + [int(x) for x in np.cumsum(LENS)]
    Ks, Vs = _layers()
    energy = torch.zeros((L, len(LENS), 4), dtype=torch.float64)
    for l in range(L):
        _, e = O.score_layer(Ks[l][:, h0:h1], Vs[l][:, h0:h1], cu, 0.25, "literal")
        energy[l] = torch.from_numpy(e)
    head_shard.allreduce_energy(energy, dist)
    budgets, offsets = O.allocate_budgets(energy.numpy(), list(LENS), 0.4, 1)
    out.put((rank, (h0, h1), energy.numpy().tolist(), budgets.tolist()))
    replicas.barrier(dist)
    dist.destroy_process_group()


def test_head_sharded_budgets_equal_the_unsharded_ones():
    from oracle import flashcache_oracle as O
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cu = [0] + [int(x) for x in np.cumsum(LENS)]
    Ks, Vs = _layers()
    energy = np.stack([O.score_layer(Ks[l], Vs[l], cu, 0.25, "literal")[1] for l in range(L)])
    budgets, _ = O.allocate_budgets(energy, list(LENS), 0.4, 1)
    assert [r[1] for r in res] == [(0, 2), (2, 4)]
    for _, _, e, b in res:
        np.testing.assert_allclose(np.array(e), energy, rtol=1e-12)
        assert b == budgets.tolist()
    assert res[0][2] == res[1][2]                      # bit-identical on both ranks


def test_shard_heads_partitions_the_heads():
    from paper_2511_16786_b200 import head_shard
    for heads, world in ((4, 2), (32, 8), (7, 3), (3, 3), (2, 4)):
        blocks = [head_shard.shard_heads(heads, world, r) for r in range(world)]
        assert blocks[0][0] == 0 and blocks[-1][1] == heads
        for (a0, a1), (b0, b1) in zip(blocks, blocks[1:]):
            assert a1 == b0
        sizes = [b - a for a, b in blocks]
        assert max(sizes) - min(sizes) <= 1
    assert head_shard.allreduce_energy(torch.ones(2), None).tolist() == [1.0, 1.0]
