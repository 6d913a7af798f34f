"""Pins for the CPU oracle's model side (oracle/model.py, oracle/chain.py).

The target forward is checked against library implementations of the same architecture (the transformers
package's Llama model and its Qwen3 mixture-of-experts block, torch's attention and RMSNorm), the rotary
embedding through its invariants, and the cached forward against the cache-free one.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import model
from oracle.chain import ChainOracle
from paper_2604_26779_b200 import inputs


def _tiny_cfg(**over):
    cfg = inputs.model_config("c1")
    cfg.update(over)
    return cfg


def test_target_forward_matches_transformers_llama():
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg = _tiny_cfg(n_kv_heads=2)                      # grouped-query attention: 4 q heads on 2 KV heads
    W = inputs.make_target_weights(cfg, seed=11, std=0.05)
    rng = np.random.default_rng(0)
    for lw in W["layers"]:                             # non-trivial norm weights
        lw["attn_norm"] = (1 + 0.1 * rng.standard_normal(cfg["d_model"])).astype(np.float32)
        lw["mlp_norm"] = (1 + 0.1 * rng.standard_normal(cfg["d_model"])).astype(np.float32)
    W["final_norm"] = (1 + 0.1 * rng.standard_normal(cfg["d_model"])).astype(np.float32)
    hf = LlamaConfig(vocab_size=cfg["vocab"], hidden_size=cfg["d_model"], intermediate_size=cfg["d_ffn"],
                     num_hidden_layers=cfg["n_layers"], num_attention_heads=cfg["n_q_heads"],
                     num_key_value_heads=cfg["n_kv_heads"], head_dim=cfg["head_dim"], rms_norm_eps=cfg["rms_eps"],
                     rope_theta=cfg["rope_theta"], attention_bias=False, mlp_bias=False,
                     tie_word_embeddings=False, max_position_embeddings=512)
    m = LlamaForCausalLM(hf).double().eval()
    Hq, Hkv, dh = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    sd = {"model.embed_tokens.weight": W["embed"], "model.norm.weight": W["final_norm"], "lm_head.weight": W["lm_head"]}
    for l, lw in enumerate(W["layers"]):
        pre = f"model.layers.{l}."
        sd[pre + "self_attn.q_proj.weight"] = lw["wqkv"][: Hq * dh]
        sd[pre + "self_attn.k_proj.weight"] = lw["wqkv"][Hq * dh : (Hq + Hkv) * dh]
        sd[pre + "self_attn.v_proj.weight"] = lw["wqkv"][(Hq + Hkv) * dh :]
        sd[pre + "self_attn.o_proj.weight"] = lw["wo"]
        sd[pre + "mlp.gate_proj.weight"] = lw["wgate"]
        sd[pre + "mlp.up_proj.weight"] = lw["wup"]
        sd[pre + "mlp.down_proj.weight"] = lw["wdown"]
        sd[pre + "input_layernorm.weight"] = lw["attn_norm"]
        sd[pre + "post_attention_layernorm.weight"] = lw["mlp_norm"]
    missing = m.load_state_dict({k: torch.tensor(np.asarray(v, np.float64)) for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k] and not missing.unexpected_keys
    toks = inputs.make_prompts(1, 23, cfg["vocab"], seed=3)[0]
    with torch.no_grad():
        out = m(torch.tensor(toks[None].astype(np.int64)), output_hidden_states=True)
    got = model.target_forward(cfg, W, toks, tap_layers=(0, 1, 2))
    # the library evaluates its rotary cos/sin tables in fp32 even in a double model: agreement stops near 1e-6,
    # four orders of magnitude below what any structural mistake (pairing, sign, norm, head order) produces
    assert np.max(np.abs(got["logits"] - out.logits[0].numpy())) < 5e-6
    assert np.max(np.abs(out.logits[0].numpy())) > 0.5
    d = cfg["d_model"]
    # residual stream after 0 and 1 layers = the library's hidden_states[0], [1]
    assert np.max(np.abs(got["taps"][:, :d] - out.hidden_states[0][0].numpy())) < 1e-12
    assert np.max(np.abs(got["taps"][:, d : 2 * d] - out.hidden_states[1][0].numpy())) < 5e-6


def test_attention_matches_torch_sdpa():
    rng = np.random.default_rng(1)
    T, n_past, Hq, Hkv, dh = 5, 37, 8, 2, 32
    q = rng.standard_normal((T, Hq, dh))
    k = rng.standard_normal((n_past + T, Hkv, dh))
    v = rng.standard_normal((n_past + T, Hkv, dh))
    got = model.attention(q, k, v, n_past)
    mask = torch.tril(torch.ones(T, n_past + T, dtype=torch.bool), diagonal=n_past)
    qt = torch.tensor(q).permute(1, 0, 2)[None]
    kt = torch.tensor(k).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    vt = torch.tensor(v).permute(1, 0, 2)[None].repeat_interleave(Hq // Hkv, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=mask)[0].permute(1, 0, 2).numpy()
    assert np.max(np.abs(got - ref)) < 1e-12


def test_rmsnorm_matches_torch():
    rng = np.random.default_rng(2)
    x, w = rng.standard_normal((6, 96)), rng.standard_normal(96)
    ref = torch.nn.functional.rms_norm(torch.tensor(x), (96,), torch.tensor(w), eps=1e-5).numpy()
    assert np.max(np.abs(model.rmsnorm(x, w, 1e-5) - ref)) < 1e-13


def test_rope_invariants():
    rng = np.random.default_rng(3)
    q, k = rng.standard_normal((1, 2, 64)), rng.standard_normal((1, 2, 64))
    theta = 10000.0
    assert np.allclose(model.rope(q, [0], theta), q)                                   # position 0 is the identity
    assert np.allclose(np.linalg.norm(model.rope(q, [123], theta), axis=-1), np.linalg.norm(q, axis=-1))
    # scores depend on the position difference only
    a = np.sum(model.rope(q, [40], theta) * model.rope(k, [33], theta))
    b = np.sum(model.rope(q, [1007], theta) * model.rope(k, [1000], theta))
    assert abs(a - b) < 1e-9
    # the first pair (j = 0, partner j + dh/2) turns by exactly `pos` radians
    e = np.zeros((1, 1, 64))
    e[0, 0, 0] = 1.0
    r = model.rope(e, [0.5], theta)[0, 0]
    assert np.isclose(r[0], np.cos(0.5)) and np.isclose(r[32], np.sin(0.5)) and np.count_nonzero(r) == 2
    # the last pair turns by pos * theta^(-(dh-2)/dh)
    e = np.zeros((1, 1, 64))
    e[0, 0, 31] = 1.0
    r = model.rope(e, [100.0], theta)[0, 0]
    assert np.isclose(r[31], np.cos(100.0 * theta ** (-62 / 64))) and np.isclose(r[63], np.sin(100.0 * theta ** (-62 / 64)))


def test_forward_with_past_equals_recompute():
    cfg = _tiny_cfg()
    W = inputs.make_target_weights(cfg, seed=5, std=0.05)
    toks = inputs.make_prompts(1, 20, cfg["vocab"], seed=8)[0]
    full = model.target_forward(cfg, W, toks, tap_layers=(0, 1, 2))
    head = model.target_forward(cfg, W, toks[:16])
    tail = model.target_forward(cfg, W, toks[16:], past=head["new_kv"], start_pos=16, tap_layers=(0, 1, 2))
    assert np.max(np.abs(tail["logits"] - full["logits"][16:])) < 1e-10
    assert np.max(np.abs(tail["taps"] - full["taps"][16:])) < 1e-10
    # k = 0: a one-token verify is plain decode
    one = model.target_forward(cfg, W, toks[19:], past=[(np.concatenate([a, c[:3]]), np.concatenate([b, e[:3]]))
                                                       for (a, b), (c, e) in zip(head["new_kv"], tail["new_kv"])],
                               start_pos=19)
    assert np.max(np.abs(one["logits"][0] - full["logits"][19])) < 1e-10


def test_moe_matches_transformers_block():
    from transformers.models.qwen3_moe import modeling_qwen3_moe as mq
    d, E, Fe, topk = 64, 16, 32, 4
    cfg = dict(inputs.model_config("c5"), d_model=d, n_experts=E, d_expert_ffn=Fe, experts_top_k=topk,
               n_q_heads=2, n_kv_heads=1, head_dim=32, dtype="f32")
    lw = inputs.make_layer_weights(cfg, np.random.default_rng(4), std=0.2)
    lw["router"] = (lw["router"] * 8).astype(np.float32)
    hf = mq.Qwen3MoeConfig(hidden_size=d, moe_intermediate_size=Fe, num_experts=E, num_experts_per_tok=topk,
                           norm_topk_prob=True)
    blk = mq.Qwen3MoeSparseMoeBlock(hf).double().eval()
    names = dict(blk.named_parameters())
    with torch.no_grad():
        names["gate.weight"].copy_(torch.tensor(lw["router"].astype(np.float64)))
        names["experts.gate_up_proj"].copy_(torch.tensor(
            np.concatenate([lw["experts_gate"], lw["experts_up"]], axis=1).astype(np.float64)))
        names["experts.down_proj"].copy_(torch.tensor(lw["experts_down"].astype(np.float64)))
        x = np.random.default_rng(5).standard_normal((9, d))
        out = blk(torch.tensor(x)[None])
        ref = (out[0] if isinstance(out, tuple) else out).reshape(9, d).numpy()
    got = model.moe_mlp(lw, x, topk)
    # the library's router takes its softmax in fp32, so the mixture weights agree to fp32 rounding only
    assert np.max(np.abs(got - ref)) < 1e-5 and np.max(np.abs(ref)) > 0.5
    # ties go to the lower expert index
    ids, wts = model.moe_route(np.array([[1.0, 3.0, 3.0, 0.0, 3.0]]), 2)
    assert ids[0].tolist() == [1, 2] and np.allclose(wts[0], 0.5)


@pytest.mark.parametrize("kind", ["eagle3", "mtp"])
def test_draft_head_consistency(kind):
    """The heads are this build's own definitions; what can be pinned is structural: proposing k tokens in one
    call equals proposing them slot by slot through the cached path, and the true-slot part is causal."""
    cfg = _tiny_cfg(tap_layers=(0, 1, 2) if kind == "eagle3" else (2,))
    W = inputs.make_target_weights(cfg, seed=5, std=0.05)
    H = (inputs.make_eagle3_weights if kind == "eagle3" else inputs.make_mtp_weights)(cfg, seed=6, std=0.05)
    toks = inputs.make_prompts(1, 12, cfg["vocab"], seed=2)[0]
    feats = model.target_forward(cfg, W, toks[:-1], tap_layers=cfg["tap_layers"])["taps"]
    u = oracle.uniforms(7, 0, 1, 1, 3)[0]

    def sample_fn(i, lg):
        q = oracle.softmax(np.asarray(lg, np.float32)[None])[0]
        return oracle.invcdf(q, u[i])[0], q

    d_all, q_all, _ = model.draft_propose(cfg, W, H, kind, feats, toks[1:], 3, sample_fn)
    # the same with the first 8 true slots served from a cache built by an earlier call
    if kind == "eagle3":
        g = feats[:8] @ H["wfc"].astype(np.float64).T
        _, pk, pv = model.eagle3_slots(cfg, W, H, g, toks[1:9], np.arange(8))
    else:
        _, pk, pv = model.mtp_slots(cfg, W, H, feats[:8], toks[1:9], np.arange(8))
    d_inc, q_inc, _ = model.draft_propose(cfg, W, H, kind, feats[8:], toks[9:], 3, sample_fn, pk, pv, first_slot=8)
    assert d_all.tolist() == d_inc.tolist() and np.max(np.abs(q_all - q_inc)) < 1e-7
    assert np.allclose(q_all.sum(-1), 1.0, atol=1e-5)


def test_chain_oracle_emits_between_1_and_k_plus_1_tokens():
    cfg = _tiny_cfg()
    W = inputs.make_target_weights(cfg, seed=inputs.sub_seed(1, 0))
    H = inputs.make_eagle3_weights(cfg, seed=inputs.sub_seed(1, 1))
    prompt = inputs.make_prompts(1, 16, cfg["vocab"], seed=inputs.sub_seed(1, 2))[0]
    ch = ChainOracle(cfg, W, H, "eagle3", seed=inputs.BASE_SEED, seq_index=0, prompt=prompt)
    for _ in range(4):
        L = len(ch.tokens)
        rec = ch.step_once(3)
        assert 1 <= rec["n_emitted"] <= 4 and len(ch.tokens) == L + rec["n_emitted"]
        assert np.all(rec["out_tokens"][rec["n_emitted"]:] == -1)
    # draft == target (the head replaced by forced drafts with q = p): every draft token is accepted
    ch2 = ChainOracle(cfg, W, H, "eagle3", seed=1, seq_index=0, prompt=prompt)
    toks = list(prompt)
    drafts, qs = [], []
    for i in range(3):
        lg = model.target_forward(cfg, W, toks + drafts)["logits"][-1].astype(np.float32)
        q = oracle.softmax(lg[None])[0]
        drafts.append(oracle.invcdf(q, 0.37 + 0.1 * i)[0])
        qs.append(q)
    rec = ch2.step_once(3, forced_drafts=(drafts, np.stack(qs)))
    assert rec["n_emitted"] == 4


def test_ngram_propose_worked_examples():
    # trailing [1,2,3] last seen at positions 4..6, followed by 9, 1, 2, 3
    assert model.ngram_propose([1, 2, 3, 4, 1, 2, 3, 9, 1, 2, 3], 3, 4).tolist() == [9, 1, 2, 3]
    # the most recent earlier occurrence wins, not the first
    assert model.ngram_propose([1, 2, 7, 1, 2, 8, 1, 2], 2, 1).tolist() == [8]
    # no 3- or 2-gram match: falls back to the single token 5 (seen at position 0, followed by 6), then runs off the end
    assert model.ngram_propose([5, 6, 5], 3, 3).tolist() == [6, 5, 5]
    # nothing matches: repeat the last token
    assert model.ngram_propose([5, 6, 7], 3, 3).tolist() == [7, 7, 7]
    assert model.ngram_propose([7], 3, 2).tolist() == [7, 7]
    # brute force on random short strings over a tiny alphabet: the proposal continues an occurrence of the longest matching suffix
    rng = np.random.default_rng(0)
    for _ in range(300):
        t = rng.integers(0, 3, rng.integers(2, 12)).tolist()
        d = model.ngram_propose(t, 3, 1)[0]
        best = None
        for n in (3, 2, 1):
            if n > len(t) - 1:
                continue
            hits = [s for s in range(len(t) - n) if t[s : s + n] == t[len(t) - n :]]
            if hits:
                best = t[max(hits) + n]
                break
        assert d == (best if best is not None else t[-1])


def test_ep_receive_layout_hand_worked():
    # 2 ranks, 4 experts (rank 0 owns 0 and 1, rank 1 owns 2 and 3), top-2.
    # rank 0 tokens: t0 -> (2, 0), t1 -> (1, 2), t2 -> (0, 1);   rank 1 tokens: t0 -> (3, 0), t1 -> (2, 3)
    ids = [np.array([[2, 0], [1, 2], [0, 1]]), np.array([[3, 0], [2, 3]])]
    rows, off = model.ep_receive_layout(ids, 4, 2)
    # worked by hand: expert 0 gets (r0,t0,slot1), (r0,t2,slot0), then (r1,t0,slot1); expert 1 gets (r0,t1,slot0), (r0,t2,slot1)
    assert rows[0] == [(0, 0, 0, 1), (0, 0, 2, 0), (0, 1, 0, 1), (1, 0, 1, 0), (1, 0, 2, 1)]
    # expert 2 gets (r0,t0,slot0), (r0,t1,slot1), then (r1,t1,slot0); expert 3 gets (r1,t0,slot0), (r1,t1,slot1)
    assert rows[1] == [(2, 0, 0, 0), (2, 0, 1, 1), (2, 1, 1, 0), (3, 1, 0, 0), (3, 1, 1, 1)]
    assert off[0].tolist() == [[0, 2], [3, 5]] and off[1].tolist() == [[0, 2], [3, 3]]
    # every (rank, token, slot) entry is received exactly once, by the owner of its expert
    seen = sorted((s, t, j) for r in rows for (_, s, t, j) in r)
    assert seen == sorted((s, t, j) for s in range(2) for t in range(ids[s].shape[0]) for j in range(2))
    assert all(e // 2 == d for d in range(2) for (e, _, _, _) in rows[d])


@pytest.mark.parametrize("ep_size", [1, 2, 4])
def test_ep_moe_equals_unsharded_moe(ep_size):
    # sharding invariance: what a token gets back does not depend on where its experts live or who else is in the batch
    d, E, Fe, topk = 32, 8, 16, 3
    cfg = dict(inputs.model_config("c5"), d_model=d, n_experts=E, d_expert_ffn=Fe, experts_top_k=topk,
               n_q_heads=2, n_kv_heads=1, head_dim=16, dtype="f32")
    lw = inputs.make_layer_weights(cfg, np.random.default_rng(14), std=0.2)
    lw["router"] = (lw["router"] * 8).astype(np.float32)
    rng = np.random.default_rng(15)
    ms = [rng.standard_normal((n, d)) for n in [5, 0, 7, 3][:ep_size]]
    got = model.ep_moe_mlp(lw, ms, topk, ep_size)
    worst = 0.0
    for s in range(ep_size):
        ref = model.moe_mlp(lw, ms[s], topk)
        assert got[s].shape == ref.shape
        if ref.size:
            worst = max(worst, float(np.max(np.abs(got[s] - ref))))
    assert worst < 1e-12


def test_e4m3_row_quantisation_hand_worked():
    import oracle
    x = np.array([[448.0, -224.0, 1.0, 0.0],          # amax 448: scale 1, the values are their own codes' values
                  [1.0, 0.5, -0.25, 0.0],             # amax 1: scale 1/448; x / scale = 448, 224, -112: all exact e4m3 values
                  [0.0, 0.0, 0.0, 0.0],               # zero row: scale 1, codes 0
                  [3.0, 1.0, 0.1, -3.0]], np.float32)
    codes, scales = oracle.e4m3_quantize_rows(x)
    assert scales[0] == 1.0 and scales[1] == np.float32(1.0) / np.float32(448.0) and scales[2] == 1.0
    assert scales[3] == np.float32(3.0) / np.float32(448.0)
    back = oracle.e4m3_rows_roundtrip(x)
    assert np.array_equal(back[0], x[0]) and np.array_equal(back[2], x[2])
    assert np.allclose(back[1], x[1], rtol=1e-6, atol=0)
    # a general row: every element within half an e4m3 step (2^-4 relative for normal values) of the original, the extreme exact
    assert abs(back[3][0] - 3.0) < 1e-6 and abs(back[3][3] + 3.0) < 1e-6
    assert abs(back[3][1] - 1.0) <= 1.0 * 2.0 ** -4 and abs(back[3][2] - 0.1) <= 0.1 * 2.0 ** -4
    # the codes are those of the per-tensor routine called row by row with the row's scale
    for r in range(4):
        assert np.array_equal(codes[r], oracle.e4m3_quantize(x[r], float(scales[r])))


def test_fp8_projection_error_is_what_the_format_allows():
    # a random projection through the 8-bit path stays within the few-percent error two 4-bit-significand operands allow,
    # and is exact when both operands are representable with a power-of-two scale: every row holds 14 = 448 * 2^-5 (so its
    # scale is exactly 2^-5) and powers of two between 1/8 and 4 (codes 4 .. 128 after scaling).  With any other row maximum
    # the fp32 scale amax / 448 is itself rounded, and the represented value code * scale is 2^-24-relative off the input:
    # that rounding belongs to the format and the product of the represented values carries it.
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 256)).astype(np.float32)
    W = (rng.standard_normal((7, 256)) * 0.05).astype(np.float32)
    ref = x.astype(np.float64) @ W.astype(np.float64).T
    got = model.proj({"w_fp8": True}, x, W)
    assert np.max(np.abs(got - ref)) / np.max(np.abs(ref)) < 0.06
    assert np.max(np.abs(got - ref)) > 0
    xp = np.ldexp(1.0, rng.integers(-3, 3, (4, 64))).astype(np.float32) * rng.choice([-1.0, 1.0], (4, 64)).astype(np.float32)
    Wp = np.ldexp(1.0, rng.integers(-3, 3, (6, 64))).astype(np.float32)
    xp[:, 0], Wp[:, 5] = 14.0, 14.0
    assert np.array_equal(model.proj({"w_fp8": True}, xp, Wp), xp.astype(np.float64) @ Wp.astype(np.float64).T)
    assert np.array_equal(model.proj({}, xp, Wp), xp.astype(np.float64) @ Wp.astype(np.float64).T)
    # stored codes and scales are taken as they stand: the same product as quantising the 16-bit matrix here
    codes, scales = oracle.e4m3_quantize_rows(W)
    assert np.array_equal(model.proj({"w_fp8": True}, x, model.QuantRows(codes, scales)), got)
    # recording returns the rows as quantised; forcing them back reproduces the product; forcing other rows replaces x
    rec = {}
    assert np.array_equal(model.proj({"w_fp8": True, "record": rec}, x, W, "qkv"), got)
    xc, xs = oracle.e4m3_quantize_rows(model._bf16_round(x))      # activations enter as 16-bit values
    assert np.array_equal(rec["qkv"].codes, xc) and np.array_equal(rec["qkv"].scales, xs)
    assert np.array_equal(model.proj({"w_fp8": True, "forced": {"qkv": rec["qkv"]}}, np.zeros_like(x), W, "qkv"), got)
    assert np.array_equal(model.proj({"w_fp8": True, "forced": {"o": rec["qkv"]}}, np.zeros_like(x), W, "qkv"), np.zeros_like(got))
    one = model.QuantRows(np.full((1, 256), 0x38, np.uint8), np.array([2.0], np.float32))      # 0x38 = 1.0: a row of twos
    assert np.allclose(model.proj({"w_fp8": True, "forced": {"qkv": one}}, x[:1], W, "qkv")[0], 2.0 * model.rows_8bit(W).sum(-1), rtol=1e-12)


def test_8bit_expert_block_reduces_to_the_dense_8bit_mlp():
    # one expert, top-1: the mixture weight is 1 and the block is the dense SwiGLU MLP through the same 8-bit projections;
    # with several experts, forcing back the rows the block itself quantised reproduces it, and the router is untouched
    rng = np.random.default_rng(11)
    d, Fe, T = 64, 48, 5
    m = rng.standard_normal((T, d))
    g, u, dn = (rng.standard_normal((Fe, d)) * 0.2).astype(np.float32), (rng.standard_normal((Fe, d)) * 0.2).astype(np.float32), \
        (rng.standard_normal((d, Fe)) * 0.2).astype(np.float32)
    cfg = {"w_fp8": True}
    one = dict(router=np.zeros((1, d), np.float32), experts_gate=[g], experts_up=[u], experts_down=[dn])
    # (row-at-a-time against whole-matrix products: equal up to the fp64 summation order of the library matmul)
    assert np.allclose(model.moe_mlp(one, m, 1, cfg=cfg), model.dense_mlp(dict(wgate=g, wup=u, wdown=dn), m, cfg), rtol=1e-12, atol=1e-14)
    E, topk = 4, 2
    lw = dict(router=rng.standard_normal((E, d)).astype(np.float32),
              experts_gate=[(rng.standard_normal((Fe, d)) * 0.2).astype(np.float32) for _ in range(E)],
              experts_up=[(rng.standard_normal((Fe, d)) * 0.2).astype(np.float32) for _ in range(E)],
              experts_down=[(rng.standard_normal((d, Fe)) * 0.2).astype(np.float32) for _ in range(E)])
    rec = {}
    a = model.moe_mlp(lw, m, topk, cfg=dict(cfg, record_moe=rec))
    assert set(rec) == {(t, j) for t in range(T) for j in range(topk)} and all(set(v) == {"gateup", "down"} for v in rec.values())
    b = model.moe_mlp(lw, np.zeros_like(m), topk, router_logits=m @ lw["router"].astype(np.float64).T,
                      cfg=dict(cfg, forced_moe=lambda t, j: rec[(t, j)]))
    assert np.array_equal(a, b)
    assert np.max(np.abs(a - model.moe_mlp(lw, m, topk))) / np.max(np.abs(a)) < 0.1 and not np.array_equal(a, model.moe_mlp(lw, m, topk))
