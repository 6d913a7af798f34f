"""The N>1 path (replicas, max-over-ranks time, summed tokens) on CPU with the gloo backend, world size 2."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_26779_b200 import inputs, replicas


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, tok = replicas.reduce_job(10.0 + 5.0 * rank, 100.0 * (rank + 1), dist)
    # weight refresh: every rank ends up with rank 0's bytes, arenas of odd sizes, several chunks
    g = torch.Generator().manual_seed(100 + rank)
    arenas = [torch.randint(0, 256, (n,), dtype=torch.uint8, generator=g) for n in (1000, 37, 4096)]
    sent = replicas.broadcast_weights(arenas, dist, src=0, chunk_bytes=300)
    g0 = torch.Generator().manual_seed(100)
    same = all(torch.equal(a, torch.randint(0, 256, (n,), dtype=torch.uint8, generator=g0)) for a, n in zip(arenas, (1000, 37, 4096)))
    dist.barrier()
    out[rank] = (ms, tok, replicas.replica_seed(rank), sent, same)
    dist.destroy_process_group()


def test_reduce_job_two_ranks():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
        assert out[0][:2] == (15.0, 300.0) and out[1][:2] == (15.0, 300.0)      # max time, summed tokens, on every rank
        assert out[0][2] != out[1][2] and out[0][2] == inputs.sub_seed(3, 0)
        assert out[0][3] == out[1][3] == 1000 + 37 + 4096 and out[0][4] and out[1][4]


def test_shard_by_tokens_balances_long_tail():
    lens = inputs.make_seq_lens_lognormal(512, 4096, np.log(2.0), 16, 32768, seed=4)
    for world in (2, 4, 8):
        groups = replicas.shard_by_tokens(lens, world)
        assert sorted(i for g in groups for i in g) == list(range(512))
        loads = [int(lens[g].sum()) for g in groups]
        assert max(loads) - min(loads) <= int(lens.max())
    assert replicas.reduce_job(3.0, 7.0) == (3.0, 7.0)
