"""Hands the CPU oracle the exact bytes a device context holds (weights, cache contents), lazily and layer by layer,
so that large workloads can be checked and timed on a bounded sample without a second copy of the model in host
memory.  TEST INFRASTRUCTURE ONLY (tests, smoke check, the benchmark's CPU-baseline leg).  It does no arithmetic of
the method: it converts storage types and gathers cache rows through the block table; the oracle's own functions do
the rest.  The context object is duck-typed (`tensor(name, layer, dtype, shape)`), nothing of the product is imported.
"""
from __future__ import annotations

import time

import numpy as np

import oracle
from oracle import model


def _np(t):
    return t.float().cpu().numpy()


def _split_gate_up(gu):
    """The device stores gate and up stacked in 256-row groups (128 gate rows, then the matching 128 up rows)."""
    F2, d = gu.shape
    t = gu.reshape(F2 // 256, 256, d)
    return t[:, :128].reshape(F2 // 2, d), t[:, 128:].reshape(F2 // 2, d)


def _w8(eng):
    """True for a context that stores the target's projections as e4m3 codes with one scale per row."""
    return int(getattr(eng.sc, "weight_dtype", 0)) == 1


def _projection(eng, name, layer, shape):
    """A projection weight as the oracle takes it: fp32 copies of the 16-bit values, or the stored codes and scales."""
    import torch
    if not _w8(eng):
        return _np(eng.tensor(name, layer, eng.tdtype, shape))
    return model.QuantRows(eng.tensor(name, layer, torch.uint8, shape).cpu().numpy(),
                           eng.tensor(name + "_SCALE", layer, torch.float32, (shape[0],)).cpu().numpy())


class _LazyRows:
    """Per-expert weight matrices [E][rows][cols] fetched from the device one expert at a time; `part` picks the gate
    (0) or up (1) half of a stacked gate/up matrix, None the whole matrix."""

    def __init__(self, dev_tensor, part=None):
        self.t, self.part = dev_tensor, part

    def __getitem__(self, e):
        m = _np(self.t[int(e)])
        return m if self.part is None else _split_gate_up(m)[self.part]


class _LazyQuantRows:
    """Per-expert 8-bit weight matrices: codes [E][rows][cols] and scales [E][rows] on the device, fetched one expert at a
    time as a QuantRows; `part` picks the gate (0) or up (1) half of a stacked gate/up matrix."""

    def __init__(self, codes, scales, part=None):
        self.codes, self.scales, self.part = codes, scales, part

    def __getitem__(self, e):
        c, s = self.codes[int(e)].cpu().numpy(), self.scales[int(e)].cpu().numpy()
        if self.part is None:
            return model.QuantRows(c, s)
        return model.QuantRows(_split_gate_up(c)[self.part], _split_gate_up(s[:, None])[self.part][:, 0])


class LazyLayers:
    """Sequence of per-layer weight dicts fetched from the device on access (fp32 copies of the stored values)."""

    def __init__(self, eng, cfg, n_layers=None):
        self.eng, self.cfg = eng, cfg
        self.n = cfg["n_layers"] if n_layers is None else n_layers

    def __len__(self):
        return self.n

    def __iter__(self):
        for l in range(self.n):
            yield self[l]

    def __getitem__(self, l):
        import torch
        eng, cfg = self.eng, self.cfg
        d, F = cfg["d_model"], cfg["d_ffn"]
        qn = (cfg["n_q_heads"] + 2 * cfg["n_kv_heads"]) * cfg["head_dim"]
        od = cfg["n_q_heads"] * cfg["head_dim"]
        td = eng.tdtype
        lw = dict(attn_norm=_np(eng.tensor("ATTN_NORM", l, torch.float32, (d,))),
                  wqkv=_projection(eng, "WQKV", l, (qn, d)), wo=_projection(eng, "WO", l, (d, od)),
                  mlp_norm=_np(eng.tensor("MLP_NORM", l, torch.float32, (d,))))
        if cfg.get("n_experts", 0) > 0:
            E, Fe = cfg["n_experts"], cfg["d_expert_ffn"]
            lw.update(router=_np(eng.tensor("ROUTER", l, td, (E, d))))
            if _w8(eng):
                u8, f32 = torch.uint8, torch.float32
                gu, gs = eng.tensor("EXPERTS_GATEUP", l, u8, (E, 2 * Fe, d)), eng.tensor("EXPERTS_GATEUP_SCALE", l, f32, (E, 2 * Fe))
                dn, ds = eng.tensor("EXPERTS_DOWN", l, u8, (E, d, Fe)), eng.tensor("EXPERTS_DOWN_SCALE", l, f32, (E, d))
                lw.update(experts_gate=_LazyQuantRows(gu, gs, 0), experts_up=_LazyQuantRows(gu, gs, 1), experts_down=_LazyQuantRows(dn, ds))
            else:
                gu = eng.tensor("EXPERTS_GATEUP", l, td, (E, 2 * Fe, d))
                dn = eng.tensor("EXPERTS_DOWN", l, td, (E, d, Fe))
                lw.update(experts_gate=_LazyRows(gu, 0), experts_up=_LazyRows(gu, 1), experts_down=_LazyRows(dn))
        else:
            gu = _projection(eng, "WGATEUP", l, (2 * F, d))
            if isinstance(gu, model.QuantRows):
                (cg, cu), (sg, su) = _split_gate_up(gu.codes), _split_gate_up(gu.scales[:, None])
                gate, up = model.QuantRows(cg, sg[:, 0]), model.QuantRows(cu, su[:, 0])
            else:
                gate, up = _split_gate_up(gu)
            lw.update(wgate=gate, wup=up, wdown=_projection(eng, "WDOWN", l, (d, F)))
        return lw


class LazyPast:
    """Per-layer (K, V) [n_past][Hkv][dh] of one sequence, gathered from the paged pools through its block table."""

    def __init__(self, eng, cfg, block_row, n_past, kv_pools, n_layers=None):
        self.eng, self.cfg, self.blocks, self.n_past, self.G = eng, cfg, block_row, n_past, kv_pools
        self.n = cfg["n_layers"] if n_layers is None else n_layers

    def __getitem__(self, l):
        import torch
        nb = -(-self.n_past // 16)
        idx = torch.as_tensor(np.ascontiguousarray(self.blocks[:nb]), dtype=torch.long, device=self.eng.device)
        out = []
        for which in ("KV_K", "KV_V"):
            pool = self.eng.kv_pool(which, l % self.G)
            rows = pool[idx].permute(0, 2, 1, 3).reshape(nb * 16, pool.shape[1], pool.shape[3])[: self.n_past]
            if pool.dtype == torch.uint8:       # 8-bit cache: e4m3 codes times the scale (torch's cast reads the codes back exactly)
                sc = self.eng.sc
                rows = rows.contiguous().view(torch.float8_e4m3fn).float() * (sc.kv_scale_k if which.endswith("_K") else sc.kv_scale_v)
            out.append(_np(rows))
        return tuple(out)


def device_weights(eng, cfg, n_layers=None):
    import torch
    d, V, td = cfg["d_model"], cfg["vocab"], eng.tdtype
    return dict(embed=_np(eng.tensor("EMBED", 0, td, (V, d))), lm_head=_projection(eng, "LM_HEAD", 0, (V, d)),
                final_norm=_np(eng.tensor("FINAL_NORM", 0, torch.float32, (d,))), layers=LazyLayers(eng, cfg, n_layers))


def oracle_verify_sample(eng, cfg, W, seq, tokens_in, n_past, block_row, kv_pools, draft_logits, seed, step,
                         n_layers=None, temperature=1.0):
    """The oracle's verify forward and rejection sampling for one sequence of a device context.

    tokens_in = [last token, d_1..d_k]; the cache prefix (n_past positions per layer) is read from the device pools as
    they stand.  Returns dict(logits, p, q, out_tokens, n_emitted, margins, seconds_forward, seconds_sample)."""
    k = len(tokens_in) - 1
    t0 = time.perf_counter()
    cfg_run = cfg if n_layers is None else dict(cfg, n_layers=n_layers)
    out = model.target_forward(cfg_run, W, tokens_in, past=LazyPast(eng, cfg, block_row, n_past, kv_pools, n_layers),
                               start_pos=n_past)
    t1 = time.perf_counter()
    logits = out["logits"].astype(np.float32)
    p = oracle.softmax(logits, temperature)
    q = oracle.softmax(np.asarray(draft_logits, np.float32), temperature) if k > 0 else np.zeros((0, p.shape[1]), np.float32)
    u = oracle.uniforms(seed, step, 0, seq + 1, k + 1)[seq]
    toks, n_emit, flags, margins = oracle.reject_sample_seq(p, q, np.asarray(tokens_in[1:], np.int32), u)
    t2 = time.perf_counter()
    return dict(logits=logits, p=p, q=q, out_tokens=toks, n_emitted=n_emit, margins=margins, final=out["final"],
                seconds_forward=t1 - t0, seconds_sample=t2 - t1)
