"""Token sharding across ranks: host logic on CPU with the gloo backend, world size 2.

Each rank runs the path on its shard (the CPU oracle stands in for the device library here: the
test is about the plumbing) and the pieces must reproduce the unsharded result: outputs by
concatenation, weight gradients by the all-reduce."""
import os
import socket

import numpy as np
import pytest

from paper_2204_00595_b200.sharding import shard_tokens


@pytest.mark.parametrize("tokens", [0, 1, 63, 64, 65, 128, 200, 8192, 8200])
@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_shards_tile_the_batch(tokens, world):
    pos = 0
    for r in range(world):
        start, count = shard_tokens(tokens, world, r)
        assert start == pos and count >= 0
        pos += count
    assert pos == tokens
    counts = [shard_tokens(tokens, world, r)[1] for r in range(world)]
    assert max(counts) - min(counts) <= 64 + 63           # balanced to one tile plus the ragged tail


def test_shard_argument_errors():
    with pytest.raises(ValueError):
        shard_tokens(10, 2, 2)
    with pytest.raises(ValueError):
        shard_tokens(-1, 2, 0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, T, m, out):
    import torch
    import torch.distributed as dist
    from oracle import monarch_oracle as O
    from paper_2204_00595_b200.sharding import allreduce_grads, shard_tokens
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(5)              # same full batch on every rank
        n = m * m
        x, dy = rng.standard_normal((T, n)), rng.standard_normal((T, n))
        L, R = rng.standard_normal((m, m, m)) / np.sqrt(m), rng.standard_normal((m, m, m)) / np.sqrt(m)
        s, c = shard_tokens(T, world, rank)
        y = O.fwd(x[s:s + c], L, R)
        g = O.bwd(x[s:s + c], dy[s:s + c], L, R)
        dL, dR = torch.from_numpy(g["dL"]).float(), torch.from_numpy(g["dR"]).float()
        allreduce_grads(dL, dR)
        ys = [None] * world
        dist.all_gather_object(ys, (s, y, g["dx"]))
        if rank == 0:
            full = O.bwd(x, dy, L, R)
            y_cat = np.concatenate([p[1] for p in sorted(ys, key=lambda p: p[0])])
            dx_cat = np.concatenate([p[2] for p in sorted(ys, key=lambda p: p[0])])
            out.put({
                "y": float(np.max(np.abs(y_cat - O.fwd(x, L, R)))),
                "dx": float(np.max(np.abs(dx_cat - full["dx"]))),
                "dL": float(np.max(np.abs(dL.numpy() - full["dL"])) / np.max(np.abs(full["dL"]))),
                "dR": float(np.max(np.abs(dR.numpy() - full["dR"])) / np.max(np.abs(full["dR"]))),
            })
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
def test_two_ranks_reproduce_the_unsharded_step():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    T, m = 200, 16                                  # ranks get 128 and 72 tokens
    procs = [ctx.Process(target=_worker, args=(r, 2, port, T, m, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=240)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert res["y"] == 0.0 and res["dx"] == 0.0     # per-token work: sharding changes nothing
    assert res["dL"] < 1e-6 and res["dR"] < 1e-6    # fp32 all-reduce of fp64 partial sums
