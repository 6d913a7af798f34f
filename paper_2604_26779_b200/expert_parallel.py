"""Expert-parallel mixture-of-experts MLP on top of the library's three spec_ep_* calls.

The paper's largest configuration (Qwen3-235B-A22B, Section 5.1) spans the GPUs of an NVLink domain: every GPU keeps its own
sequences, the experts of a block are split over the GPUs.  One block is route -> barrier -> experts -> barrier -> combine;
rows move between ranks by peer-memory loads inside the library's gather and combine kernels.  This module only owns the
buffers, exchanges the window addresses and places the barriers; it does no arithmetic.

Two ways to run it:
  * one process per GPU (`EpRank` + `exchange_windows` + `stream_barrier` over a torch.distributed group): windows are shared
    through CUDA inter-process handles;
  * several ranks inside one process on one GPU (`run_block_single_process`): the ranks' calls are issued in phase order on
    one stream, which is all the barrier they need - used by the tests and the single-GPU benchmark.
"""
from __future__ import annotations

import torch

from . import binding as api


def safe_cap_rows(ep_size, n_experts, top_k, max_rows):
    """Rows a rank can receive in the worst case: every row of every rank picks as many local experts as it can."""
    return ep_size * max_rows * min(top_k, n_experts // ep_size)


class EpRank:
    """Buffers and calls of one rank.  Every rank of a group is built with the same arguments except ep_rank."""

    def __init__(self, ep_size, ep_rank, n_experts, top_k, d, d_expert_ffn, max_rows, cap_rows=None, device="cuda"):
        if cap_rows is None:
            cap_rows = safe_cap_rows(ep_size, n_experts, top_k, max_rows)
        self.cfg = api.spec_ep_config(ep_size, ep_rank, n_experts, top_k, d, d_expert_ffn, max_rows, cap_rows)
        sizes = api.spec_ep_query_sizes(self.cfg)
        self.window = torch.zeros(sizes.window_bytes, dtype=torch.uint8, device=device)
        self.scratch = torch.zeros(sizes.scratch_bytes, dtype=torch.uint8, device=device)
        self.status = torch.zeros(4, dtype=torch.int32, device=device)
        self.peers = None
        self.M = 0

    def set_peers(self, addresses):
        """addresses[r]: where this process sees rank r's window (a device address or a tensor)."""
        assert len(addresses) == self.cfg.ep_size
        self.peers = [a if isinstance(a, int) else a.data_ptr() for a in addresses]
        assert self.peers[self.cfg.ep_rank] == self.window.data_ptr()

    def route(self, h, router_w, stream=None, rows8=False):
        """rows8: also publish the rows as e4m3 codes + scales (what experts(..., scales=...) pulls)."""
        assert h.dtype == torch.bfloat16 and router_w.dtype == torch.bfloat16 and h.shape[1] == self.cfg.d
        self.M = int(h.shape[0])
        fn = api.spec_ep_route_e4m3 if rows8 else api.spec_ep_route
        fn(self.cfg, self.window, self.scratch, self.M, h if self.M else None, router_w, stream)

    def experts(self, w_gateup, w_down, stream=None, scales=None):
        """scales: None for 16-bit expert weights, or (gate/up scales, down scales) with the weights as e4m3 codes."""
        assert self.peers is not None, "set_peers first"
        if scales is None:
            api.spec_ep_experts(self.cfg, self.peers, self.scratch, w_gateup, w_down, self.status, stream)
        else:
            assert w_gateup.dtype == torch.uint8 and w_down.dtype == torch.uint8
            api.spec_ep_experts_e4m3(self.cfg, self.peers, self.scratch, w_gateup, scales[0], w_down, scales[1], self.status, stream)

    def combine(self, x, stream=None):
        assert x.dtype == torch.float32 and tuple(x.shape) == (self.M, self.cfg.d)
        api.spec_ep_combine(self.cfg, self.peers, self.M, x if self.M else None, stream)

    def tensor(self, name):
        """A view of one piece of the window / scratch (names: the SPEC_EP_T_* ids without the prefix)."""
        ptr, nbytes = api.spec_ep_tensor(self.cfg, self.window, self.scratch, api.EP_T[name])
        for buf in (self.window, self.scratch):
            off = ptr - buf.data_ptr()
            if 0 <= off < buf.numel():
                raw = buf[off : off + nbytes]
                break
        c, n = self.cfg, self.cfg.max_rows * self.cfg.top_k
        if name in ("IDS", "COUNTS", "RECV_OFF", "RECV_TOTAL"):
            t = raw.view(torch.int32)
            return t.view(c.max_rows, c.top_k) if name == "IDS" else (t.view(c.n_experts // c.ep_size, c.ep_size) if name == "RECV_OFF" else t)
        if name == "WTS":
            return raw.view(torch.float32).view(c.max_rows, c.top_k)
        if name == "EXPERT_OUT":
            return raw.view(torch.float32).view(c.cap_rows, c.d)
        return raw.view(torch.bfloat16).view(c.cap_rows, c.d)

    def check_status(self):
        s = self.status.cpu().tolist()
        if s[0] != 0:
            raise api.SpecError(s[0], f"expert-parallel block (detail {s[1]})")


def exchange_windows(rank: EpRank, dist, group=None, export=None, open_=None):
    """Every rank publishes an inter-process handle of its window; returns the addresses under which this process sees
    all windows (its own: the local address).  `export` / `open_` default to the library's spec_ipc_* calls."""
    export = export or api.spec_ipc_export
    open_ = open_ or api.spec_ipc_open
    me, size = rank.cfg.ep_rank, rank.cfg.ep_size
    assert dist.get_world_size(group) == size and dist.get_rank(group) == me
    mine = export(rank.window)
    everyone = [None] * size
    dist.all_gather_object(everyone, mine, group=group)
    addresses = []
    for r, (handle, offset) in enumerate(everyone):
        addresses.append(rank.window.data_ptr() if r == me else open_(handle) + offset)
    rank.set_peers(addresses)
    return addresses


def stream_barrier(dist, group=None, device_tensor=None):
    """Barrier between two phases.  With a device tensor (NCCL group): an all-reduce on the current stream, so the next
    phase's kernels are ordered behind every rank's previous phase without a host round trip.  Otherwise: finish the
    local work, then a host barrier."""
    if device_tensor is not None:
        dist.all_reduce(device_tensor, group=group)
        return
    torch.cuda.synchronize()
    dist.barrier(group=group)


def run_block_single_process(ranks, hs, router_w, w_gateups, w_downs, xs, stream=None, scales=None):
    """All ranks of a group inside one process (their windows on one GPU): phase by phase on one stream."""
    addresses = [r.window.data_ptr() for r in ranks]
    for r in ranks:
        if r.peers is None:
            r.set_peers(addresses)
    for r, h in zip(ranks, hs):
        r.route(h, router_w, stream, rows8=scales is not None)
    for i, (r, gu, dn) in enumerate(zip(ranks, w_gateups, w_downs)):
        r.experts(gu, dn, stream, None if scales is None else scales[i])
    for r, x in zip(ranks, xs):
        r.combine(x, stream)
