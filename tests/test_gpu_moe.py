"""GPU parity of the mixture-of-experts decoder layer (router top-k, permutation, grouped expert GEMMs, combination)
inside a verify forward, against the CPU oracle.  The top-k choice is an integer decision taken from floating point, so
both sides take it on the same numbers: the oracle is handed the device's fp32 router logits.  Bars: selected experts
identical (order included), mixture weights within 1e-5, hidden state and logits within 2e-2 of the row maximum (bf16).
"""
import numpy as np
import pytest

from oracle import harness, model
from paper_2604_26779_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def check_moe_layer(eng, info, drafts, pre_len, pre_last, rows_of=(0,)):
    cfg = info["cfg"]
    B, k = eng.B, drafts.shape[1]
    R = k + 1
    E, tk, d = cfg["n_experts"], cfg["experts_top_k"], cfg["d_model"]
    table = eng.block_table().cpu().numpy()
    g_rl = eng.tensor("MOE_LOGITS", 0, torch.float32, (B * R, E)).cpu().numpy()
    g_ids = eng.tensor("MOE_IDS", 0, torch.int32, (B * R, tk)).cpu().numpy()
    g_w = eng.tensor("MOE_WTS", 0, torch.float32, (B * R, tk)).cpu().numpy()
    # routing on the device's own router logits
    ids, wts = model.moe_route(g_rl, tk)
    assert np.array_equal(ids, g_ids)
    assert np.max(np.abs(wts - g_w)) < 1e-5
    assert np.allclose(g_w.sum(-1), 1.0, atol=1e-5)
    # router logits themselves are ~N(0,1) as the recipe asks (only meaningful at full width)
    W = harness.device_weights(eng, cfg)
    hid = eng.tensor("HIDDEN", 0, torch.float32, (B, R, d)).cpu().numpy()
    logits = eng.logits(k).cpu().numpy()
    worst_h = worst_l = 0.0
    for b in rows_of:
        toks = [int(pre_last[b])] + [int(x) for x in drafts[b]]
        out = model.target_forward(cfg, W, toks, past=harness.LazyPast(eng, cfg, table[b], int(pre_len[b]), info["kv_pools"]),
                                   start_pos=int(pre_len[b]), router_logits=[g_rl[b * R : (b + 1) * R]] * cfg["n_layers"])
        worst_h = max(worst_h, float((np.abs(hid[b] - out["final"]).max(-1) / np.abs(out["final"]).max(-1)).max()))
        worst_l = max(worst_l, float((np.abs(logits[b] - out["logits"]).max(-1) / np.abs(out["logits"]).max(-1)).max()))
    return worst_h, worst_l, g_rl


def run_case(cfg_over, lens, vocab, rows_of):
    from paper_2604_26779_b200 import workloads
    eng, info = workloads.build_dense_workload("c5", lens=np.array(lens, np.int32), k=3, draft="none", steps_budget=2,
                                               vocab=vocab, cfg_over=cfg_over)
    B = eng.B
    drafts = torch.from_numpy(inputs.make_prompts(B, 3, info["cfg"]["vocab"], seed=77)).cuda()
    pre_len = eng.seq_len().cpu().numpy().copy()
    pre_last = eng.tensor("LAST_TOKEN", 0, torch.int32, (B,)).cpu().numpy().copy()
    eng.verify(3, drafts)
    assert eng.status().device_status == 0
    r = check_moe_layer(eng, info, drafts.cpu().numpy(), pre_len, pre_last, rows_of)
    eng.close()
    return r


def test_moe_layer_small_shapes():
    # 16 experts, top-4, expert FFN 128, d=512, 8 q / 2 KV heads of 64; ragged lengths; every row recomputed
    over = dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, n_experts=16, experts_top_k=4, d_expert_ffn=128)
    wh, wl, _ = run_case(over, [3, 40, 100, 300, 20, 1], 1024, rows_of=range(6))
    print(f"small MoE layer: hidden {wh:.2e}, logits {wl:.2e}")
    assert wh < 2e-2 and wl < 2e-2


def test_moe_layer_235b_shape_sampled():
    # the 235B-A22B layer shape: d=4096, 64 q / 4 KV heads, 128 experts top-8, expert FFN 1536, LM head over 151936
    wh, wl, rl = run_case(None, [8192, 700, 33, 2500, 8192, 1200, 64, 5000], None, rows_of=(1, 2))
    print(f"235B-shape MoE layer: hidden {wh:.2e}, logits {wl:.2e}; router logits std {rl.std():.3f}")
    assert wh < 2e-2 and wl < 2e-2
    assert 0.8 < rl.std() < 1.25
