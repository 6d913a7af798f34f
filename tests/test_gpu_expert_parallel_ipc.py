"""The expert-parallel block as it runs in production - one process per rank, windows shared through inter-process
memory handles, host barriers between the phases - here with two processes on ONE GPU (no kernel waits on another
process: each phase is finished and synchronised before the barrier).  Every rank's output must be bit-identical to the
same block computed with both ranks inside one process."""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu

E, TOP_K, D, FE = 16, 4, 512, 128
ROWS = [90, 41]


def _case():
    rng = np.random.default_rng(55)
    bf = lambda a: torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16)
    lw = dict(router=bf(rng.standard_normal((E, D)) / np.sqrt(D) * 4),
              experts_gate=bf(rng.standard_normal((E, FE, D)) / np.sqrt(D)),
              experts_up=bf(rng.standard_normal((E, FE, D)) / np.sqrt(D)),
              experts_down=bf(rng.standard_normal((E, D, FE)) / np.sqrt(FE)))
    hs = [bf(rng.standard_normal((n, D))) for n in ROWS]
    xs = [torch.from_numpy(rng.standard_normal((n, D)).astype(np.float32)) for n in ROWS]
    return lw, hs, xs


def _worker(rank, world, port, out, w8):
    from paper_2604_26779_b200 import expert_parallel as ep
    from paper_2604_26779_b200.engine import stack_gate_up
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    lw, hs, xs = _case()
    per = E // world
    me = ep.EpRank(world, rank, E, TOP_K, D, FE, max(ROWS))
    try:
        ep.exchange_windows(me, dist)
    except Exception as exc:                                   # no inter-process handles in this environment
        out[rank] = ("no-ipc", repr(exc))
        dist.barrier()
        dist.destroy_process_group()
        return
    gu = stack_gate_up(lw["experts_gate"][rank * per : (rank + 1) * per], lw["experts_up"][rank * per : (rank + 1) * per]).contiguous().cuda()
    dn = lw["experts_down"][rank * per : (rank + 1) * per].contiguous().cuda()
    x = xs[rank].clone().cuda()
    quant = lambda g_, d_: _quantised(g_, d_) if w8 else (g_, d_, None)      # 8-bit experts and 8-bit dispatch through the same windows
    gu, dn, sc = quant(gu, dn)
    me.route(hs[rank].cuda(), lw["router"].cuda(), rows8=w8)
    ep.stream_barrier(dist)
    me.experts(gu, dn, scales=sc)
    ep.stream_barrier(dist)
    me.combine(x)
    ep.stream_barrier(dist)
    me.check_status()
    # the same block with both ranks in this process
    ranks = [ep.EpRank(world, r, E, TOP_K, D, FE, max(ROWS)) for r in range(world)]
    gus = [stack_gate_up(lw["experts_gate"][r * per : (r + 1) * per], lw["experts_up"][r * per : (r + 1) * per]).contiguous().cuda() for r in range(world)]
    dns = [lw["experts_down"][r * per : (r + 1) * per].contiguous().cuda() for r in range(world)]
    xd = [t.clone().cuda() for t in xs]
    scs = None
    if w8:
        trip = [_quantised(g_, d_) for g_, d_ in zip(gus, dns)]
        gus, dns, scs = [t[0] for t in trip], [t[1] for t in trip], [t[2] for t in trip]
    ep.run_block_single_process(ranks, [h.cuda() for h in hs], lw["router"].cuda(), gus, dns, xd, scales=scs)
    torch.cuda.synchronize()
    out[rank] = ("ok", bool(torch.equal(x, xd[rank])), bool(torch.equal(x.cpu(), xs[rank])))
    dist.barrier()
    dist.destroy_process_group()


def _quantised(gu, dn):
    """Expert weights as e4m3 codes + one scale per row, by the library's quantiser."""
    from paper_2604_26779_b200 import binding as api
    g8, d8 = torch.empty(gu.shape, dtype=torch.uint8, device="cuda"), torch.empty(dn.shape, dtype=torch.uint8, device="cuda")
    gs = torch.empty(gu.shape[0] * gu.shape[1], dtype=torch.float32, device="cuda")
    ds = torch.empty(dn.shape[0] * dn.shape[1], dtype=torch.float32, device="cuda")
    api.spec_quantize_rows(gu.view(-1, gu.shape[-1]), g8.view(-1, gu.shape[-1]), gs)
    api.spec_quantize_rows(dn.view(-1, dn.shape[-1]), d8.view(-1, dn.shape[-1]), ds)
    torch.cuda.synchronize()
    return g8, d8, (gs, ds)


@pytest.mark.parametrize("w8", [False, True])
def test_two_processes_one_gpu(w8):
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, port, out, w8), nprocs=2, join=True)
        res = dict(out)
    if any(v[0] == "no-ipc" for v in res.values()):
        pytest.skip(f"inter-process memory handles are not available here: {[v for v in res.values() if v[0] == 'no-ipc'][0][1]}")
    for r in range(2):
        assert res[r] == ("ok", True, False), res[r]
