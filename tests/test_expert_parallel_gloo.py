"""Host side of the expert-parallel block with two gloo ranks on CPU: the window-address exchange (with stand-ins for
the inter-process handle calls) and the cross-rank index arithmetic of the protocol itself - each rank holds only its
own experts' weights, rows are addressed exactly as the kernels address them (owner's receive offset of (expert,
source) + the entry's rank among the source's entries of that expert) - checked against the unsharded block."""
import os
import socket
import types

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import model
from paper_2604_26779_b200 import expert_parallel as ep
from paper_2604_26779_b200 import inputs


def _case():
    d, E, Fe, topk = 32, 8, 16, 3
    cfg = dict(inputs.model_config("c5"), d_model=d, n_experts=E, d_expert_ffn=Fe, experts_top_k=topk,
               n_q_heads=2, n_kv_heads=1, head_dim=16, dtype="f32")
    lw = inputs.make_layer_weights(cfg, np.random.default_rng(21), std=0.2)
    lw["router"] = (lw["router"] * 8).astype(np.float32)
    rng = np.random.default_rng(22)
    ms = [rng.standard_normal((n, d)) for n in (6, 9)]
    return lw, ms, topk, E


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # 1. address exchange: stand-ins for the handle calls (a handle names its rank; "opening" it yields a fake base)
    fake = types.SimpleNamespace(cfg=types.SimpleNamespace(ep_rank=rank, ep_size=world), window=torch.zeros(64, dtype=torch.uint8), peers=None)
    fake.set_peers = lambda a: setattr(fake, "peers", list(a))
    addrs = ep.exchange_windows(fake, dist, export=lambda w: (bytes([rank]) * 64, 128 + rank),
                                open_=lambda h: 1_000_000 * (h[0] + 1))
    ok_addr = addrs[rank] == fake.window.data_ptr() and all(
        addrs[r] == 1_000_000 * (r + 1) + 128 + r for r in range(world) if r != rank) and fake.peers == addrs
    # 2. the protocol with real exchanges: publish (ids, per-expert entry lists, rows), pull, compute local experts, pull back
    lw, ms, topk, E = _case()
    per = E // world
    m = ms[rank]
    ids, wts = model.moe_route(m @ np.asarray(lw["router"], np.float64).T, topk)
    flat = ids.reshape(-1)
    rank_in = np.zeros(flat.size, np.int64)                   # entry's rank among this source's entries of its expert
    for e in range(E):
        idx = np.nonzero(flat == e)[0]
        rank_in[idx] = np.arange(idx.size)
    counts = np.bincount(flat, minlength=E)
    published = [None] * world
    dist.all_gather_object(published, dict(counts=counts, ids=ids, rows=m))
    # destination side: runs in (local expert, source) order; only the local experts' weights are touched
    recv_off = np.zeros((per, world), np.int64)
    y = []
    for el in range(per):
        e = rank * per + el
        g, u, dn = (np.asarray(lw[k][e], np.float64) for k in ("experts_gate", "experts_up", "experts_down"))
        for s in range(world):
            recv_off[el, s] = len(y)
            sid = published[s]["ids"]
            for t in range(sid.shape[0]):
                for j in range(topk):
                    if sid[t, j] == e:
                        x = published[s]["rows"][t]
                        y.append((model.silu(g @ x) * (u @ x)) @ dn.T)
    _, off_o = model.ep_receive_layout([p["ids"] for p in published], E, world)
    ok_layout = np.array_equal(recv_off, off_o[rank])
    back = [None] * world
    dist.all_gather_object(back, dict(recv_off=recv_off, y=y))
    # source side: row = owner's recv_off[(expert, me)] + rank of the entry
    res = np.zeros_like(m)
    for t in range(m.shape[0]):
        for j in range(topk):
            e = ids[t, j]
            owner, el = e // per, e % per
            row = back[owner]["recv_off"][el, rank] + rank_in[t * topk + j]
            res[t] += wts[t, j] * back[owner]["y"][row]
    err = float(np.max(np.abs(res - model.moe_mlp(lw, m, topk))))
    dist.barrier()
    out[rank] = (ok_addr, ok_layout, err)
    dist.destroy_process_group()


def test_exchange_and_protocol_two_ranks():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
        for r in range(2):
            ok_addr, ok_layout, err = out[r]
            assert ok_addr and ok_layout and err < 1e-12


def test_safe_capacity():
    assert ep.safe_cap_rows(8, 128, 8, 1024) == 8 * 1024 * 8
    assert ep.safe_cap_rows(64, 128, 8, 16) == 64 * 16 * 2          # two local experts: a row can land here at most twice
