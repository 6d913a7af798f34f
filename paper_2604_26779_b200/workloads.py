"""Builds the synthetic 8B-shaped workload on the device: random-init weights, a cache already filled with N(0,1)
values for sequences of seeded lengths, a permuted block order.  Used by bench.py, the smoke check and the full-size
parity test.  Data only; every number comes from seeded generators (torch's Philox on the device for the bulk
tensors, numpy's PCG64 for lengths, tokens and block order)."""
from __future__ import annotations

import numpy as np
import torch

from . import binding, engine, inputs


def _fill_normal(t: torch.Tensor, std: float, gen: torch.Generator):
    """In-place N(0, std) fill of a (possibly huge) bf16/fp32 view, in slices to keep temporaries small."""
    flat = t.reshape(-1)
    step = 1 << 28
    for i in range(0, flat.numel(), step):
        flat[i : i + step].normal_(0.0, std, generator=gen)


def _fill_normal_e4m3(t: torch.Tensor, std: float, scale: float, gen: torch.Generator):
    """In-place fill of a uint8 view with the e4m3 codes of N(0, std) / scale (input data for the 8-bit cache)."""
    flat = t.reshape(-1)
    step = 1 << 27
    for i in range(0, flat.numel(), step):
        n = min(step, flat.numel() - i)
        x = torch.empty(n, dtype=torch.float32, device=flat.device).normal_(0.0, std, generator=gen) / scale
        flat[i : i + n].copy_(x.to(torch.float8_e4m3fn).view(torch.uint8))


def build_dense_workload(name="c3", *, B=256, k=3, n_layers=None, len_lo=1024, len_hi=16384, lens=None, draft="eagle3",
                         kv_pools=None, steps_budget=64, seed=None, device="cuda:0", vocab=None, mem_fraction=0.92,
                         cfg_over=None):
    """Returns (SpecStep, info dict).  The cache of layer l lives in pool l mod G; G < n_layers (chosen so that the
    arenas fit the device) is the aliased, timing-only mode: bytes moved per layer are unchanged because one pool
    (gigabytes) is far larger than L2."""
    cfg = inputs.model_config(name)
    if n_layers is not None:
        cfg = dict(cfg, n_layers=n_layers, tap_layers=inputs.default_tap_layers(n_layers) if draft == "eagle3" else (n_layers,))
    if vocab is not None:
        cfg = dict(cfg, vocab=vocab)
    if cfg_over:
        cfg = dict(cfg, **cfg_over)
    seed = inputs.sub_seed(3, 0) if seed is None else seed
    if lens is None:
        lens = inputs.make_seq_lens_uniform(B, len_lo, len_hi, seed + 1)
    lens = np.ascontiguousarray(lens, np.int32)
    B = lens.shape[0]
    bt = 16
    grow = steps_budget * (k + 1) + k + 2
    per_seq = [-(-(int(l) + grow) // bt) for l in lens]
    max_blocks = max(per_seq) + 1
    num_blocks = int(sum(per_seq)) + 16
    L = cfg["n_layers"]

    def sizes_for(G):
        sc = engine.make_spec_config(cfg, draft_kind=draft, k_max=k, max_batch=B, kv_num_blocks=num_blocks,
                                     max_blocks_per_seq=max_blocks, kv_layer_pools=G, seed=seed,
                                     draft_vocab=int(cfg.get("draft_vocab") or 0), draft_greedy=bool(cfg.get("draft_greedy")),
                                     kv_fp8=cfg.get("kv_fp8"), w_fp8=bool(cfg.get("w_fp8")))
        from . import binding as Bd
        import ctypes as C
        s = Bd.spec_sizes()
        Bd._check(Bd.lib().spec_query_sizes(C.byref(sc), C.byref(s)), "spec_query_sizes")
        total = s.weights_bytes + s.draft_weights_bytes + s.kv_bytes + s.draft_kv_bytes + s.workspace_bytes + s.state_bytes
        return sc, total

    free, _total = torch.cuda.mem_get_info(torch.device(device))
    G = L if kv_pools is None else min(kv_pools, L)
    sc, need = sizes_for(G)
    while need > free * mem_fraction and G > 1:
        G -= 1
        sc, need = sizes_for(G)
    if need > free * mem_fraction:
        raise RuntimeError(f"workload needs {need / 1e9:.1f} GB, device has {free / 1e9:.1f} GB free")
    eng = engine.SpecStep(sc, device=device)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    bf = eng.tdtype
    f32 = torch.float32
    w8 = bool(cfg.get("w_fp8"))

    def fill_projection(name, layer, rows, k):
        # N(0, 0.02) weights; with 8-bit weights they are drawn in bf16 and quantised row by row on the device by the library
        if not w8:
            return _fill_normal(eng.tensor(name, layer, bf), 0.02, gen)
        tmp = torch.empty((rows, k), dtype=torch.bfloat16, device=device)
        _fill_normal(tmp, 0.02, gen)
        binding.spec_quantize_rows(tmp, eng.tensor(name, layer, torch.uint8, (rows, k)), eng.tensor(name + "_SCALE", layer, f32, (rows,)))
        torch.cuda.synchronize()

    d_, qn_, od_ = cfg["d_model"], (cfg["n_q_heads"] + 2 * cfg["n_kv_heads"]) * cfg["head_dim"], cfg["n_q_heads"] * cfg["head_dim"]
    _fill_normal(eng.tensor("EMBED", 0, bf), 0.02, gen)
    fill_projection("LM_HEAD", 0, cfg["vocab"], d_)
    eng.tensor("FINAL_NORM", 0, f32).fill_(1.0)
    for l in range(L):
        eng.tensor("ATTN_NORM", l, f32).fill_(1.0)
        eng.tensor("MLP_NORM", l, f32).fill_(1.0)
        if cfg.get("n_experts", 0) > 0:
            E_, Fe_ = cfg["n_experts"], cfg["d_expert_ffn"]
            fill_projection("WQKV", l, qn_, d_)
            fill_projection("WO", l, d_, od_)
            fill_projection("EXPERTS_GATEUP", l, E_ * 2 * Fe_, d_)
            fill_projection("EXPERTS_DOWN", l, E_ * d_, Fe_)
            # router rows ~ N(0, 1/d): unit-RMS inputs give router logits ~ N(0, 1)
            _fill_normal(eng.tensor("ROUTER", l, bf), float(cfg["d_model"]) ** -0.5, gen)
        else:
            fill_projection("WQKV", l, qn_, d_)
            fill_projection("WO", l, d_, od_)
            fill_projection("WGATEUP", l, 2 * cfg["d_ffn"], d_)
            fill_projection("WDOWN", l, d_, cfg["d_ffn"])
    if draft != "none":
        for nm in ("D_NORM_E", "D_NORM_G", "D_MLP_NORM") + (("D_NORM_F",) if draft == "eagle3" else ("D_ATTN_NORM",)):
            eng.tensor(nm, 0, f32).fill_(1.0)
        for nm in ("D_WQKV", "D_WO", "D_WGATEUP", "D_WDOWN") + (("D_WFC", "D_LM_HEAD") if draft == "eagle3" else ("D_WPROJ",)):
            _fill_normal(eng.tensor(nm, 0, bf), 0.02, gen)
        if draft == "eagle3" and cfg.get("draft_vocab"):      # the head's id set: a seeded subset of the vocabulary, increasing
            rng = np.random.Generator(np.random.PCG64(seed + 4))
            d2t = np.sort(rng.choice(cfg["vocab"], size=int(cfg["draft_vocab"]), replace=False)).astype(np.int32)
            eng.tensor("D_D2T", 0, torch.int32).copy_(torch.from_numpy(d2t).to(device))
        if cfg.get("kv_fp8"):
            _fill_normal_e4m3(eng.kv_pool("DRAFT_KV_K", 0), 1.0, cfg["kv_fp8"][0], gen)
            _fill_normal_e4m3(eng.kv_pool("DRAFT_KV_V", 0), 1.0, cfg["kv_fp8"][1], gen)
        else:
            _fill_normal(eng.tensor("DRAFT_KV_K", 0, bf), 1.0, gen)
            _fill_normal(eng.tensor("DRAFT_KV_V", 0, bf), 1.0, gen)
    for p in range(G):
        if cfg.get("kv_fp8"):
            _fill_normal_e4m3(eng.kv_pool("KV_K", p), 1.0, cfg["kv_fp8"][0], gen)
            _fill_normal_e4m3(eng.kv_pool("KV_V", p), 1.0, cfg["kv_fp8"][1], gen)
        else:
            _fill_normal(eng.tensor("KV_K", p, bf), 1.0, gen)
            _fill_normal(eng.tensor("KV_V", p, bf), 1.0, gen)
    last = inputs.make_prompts(B, 1, cfg["vocab"], seed + 2)[:, 0]
    order = inputs.make_block_order(num_blocks, seed + 3)
    torch.cuda.synchronize()
    info = dict(cfg=cfg, lens=lens, last_token=last, block_order=order, kv_pools=G, aliased=G < L, bytes=need,
                num_blocks=num_blocks, max_blocks=max_blocks, B=B, k=k, draft=draft, seed=seed)
    eng.seq_init(lens, last, order)
    return eng, info


def bootstrap(eng):
    """One plain decode step (k = 0) so that the draft head has a committed position to draft from."""
    eng.verify(0)
    eng.reject_sample(0)
    eng.kv_commit()


def spec_step(eng, k, with_draft=True):
    if with_draft:
        eng.draft(k)
    eng.verify(k)
    eng.reject_sample(k)
    eng.kv_commit()
