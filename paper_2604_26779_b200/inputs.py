"""Seeded synthetic inputs: model shapes, weights, prompts, logits, KV lengths and block orders.

This module is data only.  It serves both the CUDA path and the CPU oracle and therefore holds none of the
method's arithmetic (no softmax, no sampling, no attention): it draws numbers from numpy's PCG64 generator
and shapes them.  The shapes are those of the five workloads the build is measured on:

  C1  tiny chain speculation  (2-layer d=256 target, one-layer EAGLE-3-style draft, fp32, B=4, k=3)
  C2  rejection-sampling micro-benchmark (B=1024, V=151936, k in {1,3,5,7})
  C3  8B-shaped dense verify (32 layers, d=4096, 32 q / 8 KV heads, FFN 14336, V=128256, bf16) + EAGLE-3 head
  C4  the same target with an MTP head, B=512, long-tailed KV lengths
  C5  one mixture-of-experts decoder layer of 235B-A22B shape + LM head over V=151936
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 2604026779


def sub_seed(config_index: int, tensor_id: int) -> int:
    return BASE_SEED + 1000 * config_index + tensor_id


# ---- shapes --------------------------------------------------------------------------------------------------

def model_config(name: str) -> dict:
    if name == "c1":
        return dict(name="c1", n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=4, head_dim=64, d_ffn=1024,
                    vocab=1024, rms_eps=1e-5, rope_theta=10000.0, n_experts=0, experts_top_k=0, d_expert_ffn=0,
                    dtype="f32", tap_layers=(0, 1, 2), temperature=1.0)
    if name in ("c3", "c4"):
        return dict(name=name, n_layers=32, d_model=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, d_ffn=14336,
                    vocab=128256, rms_eps=1e-5, rope_theta=500000.0, n_experts=0, experts_top_k=0,
                    d_expert_ffn=0, dtype="bf16", tap_layers=(2, 16, 29) if name == "c3" else (32,),
                    temperature=1.0)
    if name == "c5":
        return dict(name="c5", n_layers=1, d_model=4096, n_q_heads=64, n_kv_heads=4, head_dim=128, d_ffn=0,
                    vocab=151936, rms_eps=1e-5, rope_theta=500000.0, n_experts=128, experts_top_k=8,
                    d_expert_ffn=1536, dtype="bf16", tap_layers=(), temperature=1.0)
    raise KeyError(name)


def scaled_config(base: str, **over) -> dict:
    """A workload's shape with some dimensions shrunk, for parity cases the oracle finishes in seconds."""
    cfg = model_config(base)
    cfg.update(over)
    return cfg


def default_tap_layers(n_layers: int) -> tuple:
    """Residual-stream taps fed to the EAGLE-3-style head: after 2, L/2 and L-3 layers (small models: 0, ceil(L/2), L)."""
    if n_layers >= 6:
        return (2, n_layers // 2, n_layers - 3)
    return (0, (n_layers + 1) // 2, n_layers)


# ---- number formats ------------------------------------------------------------------------------------------

def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """fp32 array whose values are the nearest-even bf16 values of `a` (still stored as fp32)."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns of an fp32 array that already holds bf16-representable values."""
    return (np.ascontiguousarray(a, np.float32).view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def _normal(rng, shape, std, dtype):
    w = rng.standard_normal(shape, dtype=np.float32) * np.float32(std)
    return round_to_bf16(w) if dtype == "bf16" else w


# ---- weights -------------------------------------------------------------------------------------------------

def make_layer_weights(cfg: dict, rng, std=0.02, qkv_in=None) -> dict:
    d, Hq, Hkv, dh = cfg["d_model"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    dt = cfg["dtype"]
    lw = dict(attn_norm=np.ones(d, np.float32),
              wqkv=_normal(rng, ((Hq + 2 * Hkv) * dh, qkv_in or d), std, dt),
              wo=_normal(rng, (d, Hq * dh), std, dt),
              mlp_norm=np.ones(d, np.float32))
    if cfg.get("n_experts", 0) > 0:
        E, Fe = cfg["n_experts"], cfg["d_expert_ffn"]
        # router rows ~ N(0, 1/d): with unit-RMS inputs the router logits come out ~ N(0, 1)
        lw["router"] = _normal(rng, (E, d), 1.0 / np.sqrt(d), dt)
        lw["experts_gate"] = _normal(rng, (E, Fe, d), std, dt)
        lw["experts_up"] = _normal(rng, (E, Fe, d), std, dt)
        lw["experts_down"] = _normal(rng, (E, d, Fe), std, dt)
    else:
        F = cfg["d_ffn"]
        lw["wgate"] = _normal(rng, (F, d), std, dt)
        lw["wup"] = _normal(rng, (F, d), std, dt)
        lw["wdown"] = _normal(rng, (d, F), std, dt)
    return lw


def make_target_weights(cfg: dict, seed: int, std=0.02) -> dict:
    rng = np.random.Generator(np.random.PCG64(seed))
    d, V, dt = cfg["d_model"], cfg["vocab"], cfg["dtype"]
    return dict(embed=_normal(rng, (V, d), std, dt),
                layers=[make_layer_weights(cfg, rng, std) for _ in range(cfg["n_layers"])],
                final_norm=np.ones(d, np.float32),
                lm_head=_normal(rng, (V, d), std, dt))


def make_eagle3_weights(cfg: dict, seed: int, std=0.02) -> dict:
    """One-layer EAGLE-3-style head: W_fc (3d->d), a layer whose QKV reads 2d inputs, its own LM head."""
    rng = np.random.Generator(np.random.PCG64(seed))
    d, V, dt = cfg["d_model"], cfg["vocab"], cfg["dtype"]
    dense = dict(cfg, n_experts=0, d_ffn=cfg["d_ffn"] or 4 * d)
    H = make_layer_weights(dense, rng, std, qkv_in=2 * d)
    del H["attn_norm"]
    Vd = int(cfg.get("draft_vocab") or 0)
    H.update(wfc=_normal(rng, (d, len(cfg["tap_layers"]) * d), std, dt),
             norm_e=np.ones(d, np.float32), norm_g=np.ones(d, np.float32), norm_f=np.ones(d, np.float32),
             lm_head=_normal(rng, (Vd or V, d), std, dt))
    if Vd:      # the head's own vocabulary: a seeded subset of the target's ids, in increasing order
        H["d2t"] = np.sort(rng.choice(V, size=Vd, replace=False)).astype(np.int32)
    return H


def make_mtp_weights(cfg: dict, seed: int, std=0.02) -> dict:
    """MTP-style head: W_proj (2d->d) and one ordinary decoder layer; norm and LM head are the target's."""
    rng = np.random.Generator(np.random.PCG64(seed))
    d, dt = cfg["d_model"], cfg["dtype"]
    dense = dict(cfg, n_experts=0, d_ffn=cfg["d_ffn"] or 4 * d)
    H = make_layer_weights(dense, rng, std)
    H.update(wproj=_normal(rng, (d, 2 * d), std, dt),
             norm_e=np.ones(d, np.float32), norm_g=np.ones(d, np.float32))
    return H


# ---- tokens, logits, lengths, block orders -------------------------------------------------------------------

def make_prompts(B: int, length: int, vocab: int, seed: int) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(0, vocab, size=(B, length), dtype=np.int64).astype(np.int32)


def make_sampler_logits(B: int, k: int, V: int, sigma: float, tau: float, seed: int):
    """Micro-benchmark logits: target rows N(0, sigma^2) [B][k+1][V]; draft rows = target + N(0, tau^2) [B][k][V]."""
    rng = np.random.Generator(np.random.PCG64(seed))
    t = rng.standard_normal((B, k + 1, V), dtype=np.float32) * np.float32(sigma)
    d = t[:, :k, :] + rng.standard_normal((B, k, V), dtype=np.float32) * np.float32(tau)
    return t, d.astype(np.float32)


def make_seq_lens_uniform(B: int, lo: int, hi: int, seed: int) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(lo, hi + 1, size=B, dtype=np.int64).astype(np.int32)


def make_seq_lens_lognormal(B: int, median: int, sigma: float, lo: int, hi: int, seed: int) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed))
    z = rng.standard_normal(B)
    return np.clip(np.rint(median * np.exp(sigma * z)), lo, hi).astype(np.int32)


def make_block_order(num_blocks: int, seed: int) -> np.ndarray:
    """Initial free stack: a seeded permutation of the physical block ids (no contiguity to exploit)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.permutation(num_blocks).astype(np.int32)


def make_kv_values(shape, seed: int, dtype="bf16") -> np.ndarray:
    """Synthetic cache contents ~ N(0,1) for workloads that start from a filled cache (no prefill is run)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return _normal(rng, shape, 1.0, dtype)
