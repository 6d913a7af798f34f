"""GPU parity of a verify pass with 8-bit (e4m3) projections, projection by projection.

Quantising an activation row is a step function (a row maximum that rounds to the neighbouring 16-bit value moves the
row's scale and with it many codes), so logits of two whole forwards that differ in the last place of one activation
drift apart by about the format's own noise; an end-to-end bar would say nothing.  Instead the context keeps the rows every
projection of its last layer (and the LM head) consumed, and each stage is checked with those rows forced into the oracle:

  product     forced rows x stored weight codes, exact in the oracle: cache entries (after the rotary embedding) to bf16
              rounding, residual stream and logits to fp32 accumulation error
  quantiser   what the oracle quantises from ITS result of the stage before against the device's rows of the next stage:
              scales within one 16-bit step, nearly all codes equal, none further than one code step
"""
import numpy as np
import pytest

import oracle
from oracle import harness, model

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def act_rows(eng, slot, M, K):
    codes = eng.tensor("ACT_CODES", slot, torch.uint8)[: M * K].view(M, K).cpu().numpy()
    scales = eng.tensor("ACT_SCALES", slot, torch.float32)[:M].cpu().numpy()
    return model.QuantRows(codes, scales)


def rows_of(qr, r0, r1):
    return model.QuantRows(qr.codes[r0:r1], qr.scales[r0:r1])


def compare_rows(dev, ref, what, min_equal, abs_rms=0.0):
    """Device rows against the oracle's: scales within one bf16 step of the row maximum, values within one e4m3 step of
    the element (at most 2^-3 of it; sub-normal codes: 2^-9 of the scale) plus the effect of that scale difference, plus
    abs_rms times the row's RMS where the 16-bit input itself carries an absolute error: the attention output, whose
    probabilities and queries are bf16 on the device (each about 2^-9 relative, together about 3e-3 of the row's RMS as a
    standard deviation; the bar of 2e-2 is six of those, for the maximum over tens of thousands of elements)."""
    assert np.all(np.abs(dev.scales - ref.scales) <= 2.0 ** -7 * ref.scales), what
    a, b = dev.values(), ref.values()
    tol = 0.135 * np.abs(b) + 2.0 ** -9 * ref.scales[:, None] + abs_rms * np.sqrt(np.mean(b * b, -1, keepdims=True))
    assert np.all(np.abs(a - b) <= tol), (what, float(np.max(np.abs(a - b) - tol)))
    same = float(np.mean(dev.codes == ref.codes))
    assert same >= min_equal, (what, same)
    return same


@pytest.mark.parametrize("n_layers,head_dim,kv_fp8", [(1, 128, None), (3, 128, None), (1, 64, None), (2, 128, (0.25, 0.25))])
def test_w_fp8_verify_projection_by_projection(n_layers, head_dim, kv_fp8):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26779_b200 import workloads
    k = 3
    over = dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=head_dim, d_ffn=1024, w_fp8=True)
    if kv_fp8:
        over["kv_fp8"] = kv_fp8
    lens = np.array([5, 40, 100, 17, 300, 64, 33], np.int32)
    eng, info = workloads.build_dense_workload("c3", lens=lens, k=k, draft="eagle3", steps_budget=8, n_layers=n_layers,
                                               vocab=2048, cfg_over=over)
    cfg = dict(info["cfg"], n_layers=n_layers)
    B, d, V, F = eng.B, cfg["d_model"], cfg["vocab"], cfg["d_ffn"]
    Hq, Hkv, dh = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    W = harness.device_weights(eng, cfg)
    assert isinstance(W["lm_head"], model.QuantRows)
    lw = W["layers"][n_layers - 1]
    workloads.bootstrap(eng)
    eng.draft(k); eng.verify(k); eng.reject_sample(k); eng.kv_commit()      # one whole step first: state past the bootstrap
    seq_len = eng.seq_len().cpu().numpy().copy()
    last = eng.tensor("LAST_TOKEN", 0, torch.int32, (B,)).cpu().numpy().copy()
    eng.draft(k)
    drafts = eng.draft_tokens().cpu().numpy()[:, :k].copy()
    eng.verify(k)
    assert eng.status().device_status == 0
    table = eng.block_table().cpu().numpy().copy()
    R, M = k + 1, B * (k + 1)
    dev = {"qkv": act_rows(eng, 0, M, d), "o": act_rows(eng, 1, M, Hq * dh), "gateup": act_rows(eng, 2, M, d),
           "down": act_rows(eng, 3, M, F), "lm_head": act_rows(eng, 4, M, d)}
    hidden = eng.tensor("HIDDEN", 0, torch.float32, (M, d)).cpu().numpy().astype(np.float64)
    logits = eng.logits(k).cpu().numpy().reshape(M, V).astype(np.float64)
    stats = eng.tensor("ROW_STATS", 0, torch.float32, (M, 2)).cpu().numpy()
    embed = W["embed"]
    worst_kv = worst_x = worst_l = 0.0
    equal = {"qkv": 1.0, "o": 1.0, "gateup": 1.0, "down": 1.0, "lm_head": 1.0}
    for b in range(B):
        r0, r1 = b * R, (b + 1) * R
        n_past = int(seq_len[b])
        tokens = [int(last[b])] + [int(t) for t in drafts[b]]
        pos = np.arange(n_past, n_past + R)
        record = {}
        cfg_f = dict(cfg, forced={s: rows_of(q, r0, r1) for s, q in dev.items()}, record=record)
        past = harness.LazyPast(eng, cfg, table[b], n_past, info["kv_pools"], n_layers)[n_layers - 1]
        # a one-layer model starts from the embedding rows, which the oracle knows exactly; deeper ones: the layer's input is
        # not kept, so what depends on it (the residual stream) is left to the one-layer cases
        x_in = embed[tokens].astype(np.float64) if n_layers == 1 else np.zeros((R, d))
        x_out, k_new, v_new = model.decoder_layer(cfg_f, lw, x_in, pos, past[0] if n_past else None, past[1] if n_past else None)
        # -- QKV product + rotary embedding + cache append: the device's cache entries of the new positions
        got = harness.LazyPast(eng, cfg, table[b], n_past + R, info["kv_pools"], n_layers)[n_layers - 1]
        for g_, ref in ((got[0][n_past:], k_new), (got[1][n_past:], v_new)):
            if kv_fp8:      # the oracle's values are already rounded to the cache format: one code step where fp32 and fp64 results straddle a boundary
                assert np.all(np.abs(g_ - ref) <= 0.126 * np.abs(ref) + 2.0 ** -9 * kv_fp8[0])
                assert np.mean(g_ == ref.astype(np.float32)) > 0.97
            else:
                err = np.abs(g_ - ref) / (np.abs(ref) + 1e-3 * np.abs(ref).max())
                worst_kv = max(worst_kv, float(err.max()))
        # -- attention output as the O projection consumed it (q went through the same epilogue as k)
        equal["o"] = min(equal["o"], compare_rows(rows_of(dev["o"], r0, r1), record["o"], "o", 0.80, abs_rms=2e-2))
        # -- SwiGLU of the forced gate/up input, as the down projection consumed it
        equal["down"] = min(equal["down"], compare_rows(rows_of(dev["down"], r0, r1), record["down"], "down", 0.97))
        if n_layers == 1:
            equal["qkv"] = min(equal["qkv"], compare_rows(rows_of(dev["qkv"], r0, r1), record["qkv"], "qkv", 0.99))
            equal["gateup"] = min(equal["gateup"], compare_rows(rows_of(dev["gateup"], r0, r1), record["gateup"], "gateup", 0.99))
            # -- O and down products with their residual adds: the fp32 residual stream after the layer
            worst_x = max(worst_x, float(np.abs(hidden[r0:r1] - x_out).max() / np.abs(x_out).max()))
        # -- final norm of the device's residual stream, quantised, then the LM head product and its row statistics
        rec2 = {}
        cfg_l = dict(cfg, forced={"lm_head": rows_of(dev["lm_head"], r0, r1)}, record=rec2)
        ref_logits = model.proj(cfg_l, model.rmsnorm(hidden[r0:r1], W["final_norm"], cfg["rms_eps"]), W["lm_head"], "lm_head")
        equal["lm_head"] = min(equal["lm_head"], compare_rows(rows_of(dev["lm_head"], r0, r1), rec2["lm_head"], "lm_head", 0.99))
        worst_l = max(worst_l, float((np.abs(logits[r0:r1] - ref_logits).max(-1) / np.abs(ref_logits).max(-1)).max()))
        for j in range(R):
            m_o, z_o = oracle.softmax_stats(logits[r0 + j].astype(np.float32), 1.0)
            assert stats[r0 + j, 0] == m_o and abs(stats[r0 + j, 1] - z_o) <= 1e-4 * z_o
    print(f"w_fp8 L={n_layers} dh={head_dim} kv_fp8={kv_fp8}: cache entries {worst_kv:.2e}, residual stream {worst_x:.2e}, "
          f"logits {worst_l:.2e}, equal codes {equal}")
    assert worst_kv < 2.0 ** -7          # bf16 rounding of the stored value (2^-9 .. 2^-8) plus fp32 accumulation
    assert worst_x < 1e-5 and worst_l < 1e-5
    eng.close()


def test_w_fp8_full_size_sampled():
    """The benchmark's configuration with 8-bit projections (8B shape, 32 layers, B = 256, cache lengths ~U[1024,16384], k = 3):
    sampled sequences, the last layer and the LM head, with the device's own quantised rows forced into the oracle."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 60e9:
        pytest.skip("needs a device with > 60 GB free")
    from paper_2604_26779_b200 import workloads
    k, B = 3, 256
    eng, info = workloads.build_dense_workload("c3", B=B, k=k, steps_budget=8, cfg_over=dict(w_fp8=True))
    cfg = info["cfg"]
    L, d, V, F = cfg["n_layers"], cfg["d_model"], cfg["vocab"], cfg["d_ffn"]
    Hq, dh = cfg["n_q_heads"], cfg["head_dim"]
    assert L == 32 and d == 4096 and V == 128256 and cfg.get("w_fp8")
    workloads.bootstrap(eng)
    workloads.spec_step(eng, k)
    seq_len = eng.seq_len().cpu().numpy().copy()
    eng.draft(k)
    eng.verify(k)
    assert eng.status().device_status == 0
    table = eng.block_table().cpu().numpy().copy()
    R, M = k + 1, B * (k + 1)
    W = harness.device_weights(eng, cfg)
    lw = W["layers"][L - 1]
    worst_kv = worst_l = 0.0
    low = {"o": 1.0, "down": 1.0, "lm_head": 1.0}
    for b in (0, 101, 255):
        r0, r1 = b * R, (b + 1) * R
        n_past = int(seq_len[b])
        forced = {}
        for s, (slot, K) in {"qkv": (0, d), "o": (1, Hq * dh), "gateup": (2, d), "down": (3, F), "lm_head": (4, d)}.items():
            codes = eng.tensor("ACT_CODES", slot, torch.uint8)[: M * K].view(M, K)[r0:r1].cpu().numpy()
            scales = eng.tensor("ACT_SCALES", slot, torch.float32)[r0:r1].cpu().numpy()
            forced[s] = model.QuantRows(codes, scales)
        record = {}
        cfg_f = dict(cfg, forced=forced, record=record)
        past = harness.LazyPast(eng, cfg, table[b], n_past, info["kv_pools"], L)[L - 1]
        pos = np.arange(n_past, n_past + R)
        _, k_new, v_new = model.decoder_layer(cfg_f, lw, np.zeros((R, d)), pos, past[0], past[1])
        got = harness.LazyPast(eng, cfg, table[b], n_past + R, info["kv_pools"], L)[L - 1]
        for g_, ref in ((got[0][n_past:], k_new), (got[1][n_past:], v_new)):
            worst_kv = max(worst_kv, float((np.abs(g_ - ref) / (np.abs(ref) + 1e-3 * np.abs(ref).max())).max()))
        low["o"] = min(low["o"], compare_rows(forced["o"], record["o"], "o", 0.80, abs_rms=2e-2))
        low["down"] = min(low["down"], compare_rows(forced["down"], record["down"], "down", 0.97))
        hidden = eng.tensor("HIDDEN", 0, torch.float32, (M, d))[r0:r1].cpu().numpy().astype(np.float64)
        rec2 = {}
        ref_logits = model.proj(dict(cfg, forced={"lm_head": forced["lm_head"]}, record=rec2),
                                model.rmsnorm(hidden, W["final_norm"], cfg["rms_eps"]), W["lm_head"], "lm_head")
        low["lm_head"] = min(low["lm_head"], compare_rows(forced["lm_head"], rec2["lm_head"], "lm_head", 0.99))
        logits = eng.logits(k)[b].cpu().numpy().reshape(R, V).astype(np.float64)
        worst_l = max(worst_l, float((np.abs(logits - ref_logits).max(-1) / np.abs(ref_logits).max(-1)).max()))
    print(f"w_fp8 full size: cache entries {worst_kv:.2e}, logits {worst_l:.2e}, equal codes {low}")
    assert worst_kv < 2.0 ** -7 and worst_l < 1e-5
    eng.close()


def test_w_fp8_mtp_head_scores_with_the_8bit_lm_head():
    """The MTP head's logits are the target's LM head applied to its own hidden state: with 8-bit projections that product
    takes the head's rows quantised per row; the last pass's rows stay in slot 4 until the verify pass overwrites them."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26779_b200 import workloads
    k = 3
    over = dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=128, d_ffn=1024, w_fp8=True)
    lens = np.array([5, 40, 100, 17, 300, 64, 33], np.int32)
    eng, info = workloads.build_dense_workload("c3", lens=lens, k=k, draft="mtp", steps_budget=8, n_layers=2, vocab=2048, cfg_over=over)
    cfg = dict(info["cfg"], n_layers=2)
    B, d, V = eng.B, cfg["d_model"], cfg["vocab"]
    W = harness.device_weights(eng, cfg)
    workloads.bootstrap(eng)
    workloads.spec_step(eng, k)
    eng.draft(k)
    assert eng.status().device_status == 0
    rows = act_rows(eng, 4, B, d)
    dlog = eng.draft_logits(k).cpu().numpy().astype(np.float64)[:, k - 1]
    ref = model.proj(dict(cfg, forced={"lm_head": rows}), np.zeros((B, d)), W["lm_head"], "lm_head")
    err = float((np.abs(dlog - ref).max(-1) / np.abs(ref).max(-1)).max())
    print(f"w_fp8 MTP head: last pass logits {err:.2e}")
    assert err < 1e-5
    eng.close()


@pytest.mark.parametrize("shape", ["small", "235b"])
def test_w_fp8_moe_layer_projection_by_projection(shape):
    """One mixture-of-experts decoder layer + LM head with 8-bit projections (the router stays 16-bit and decides on the
    device's own fp32 logits): the rows every expert entry consumed - in expert order, found through MOE_INV - are forced into
    the oracle; products to fp32 accumulation error, quantiser decisions compared where the oracle reproduces the input."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26779_b200 import inputs, workloads
    k = 3
    if shape == "small":
        over = dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, n_experts=16, experts_top_k=4, d_expert_ffn=128, w_fp8=True)
        lens, vocab, checked = [3, 40, 100, 300, 20, 1], 1024, range(6)
    else:           # d=4096, 64 q / 4 KV heads of 128, 128 experts top-8, expert FFN 1536, LM head over 151936
        over, lens, vocab, checked = dict(w_fp8=True), [8192, 700, 33, 2500, 8192, 1200, 64, 5000], None, (1, 2)
    eng, info = workloads.build_dense_workload("c5", lens=np.array(lens, np.int32), k=k, draft="none", steps_budget=2, vocab=vocab, cfg_over=over)
    cfg = info["cfg"]
    assert cfg["n_layers"] == 1 and cfg["n_experts"] > 0
    B, d, V, Fe, E, tk = eng.B, cfg["d_model"], cfg["vocab"], cfg["d_expert_ffn"], cfg["n_experts"], cfg["experts_top_k"]
    Hq, dh = cfg["n_q_heads"], cfg["head_dim"]
    R, M = k + 1, B * (k + 1)
    n = M * tk
    drafts = torch.from_numpy(inputs.make_prompts(B, k, V, seed=77)).cuda()
    seq_len = eng.seq_len().cpu().numpy().copy()
    last = eng.tensor("LAST_TOKEN", 0, torch.int32, (B,)).cpu().numpy().copy()
    eng.verify(k, drafts)
    assert eng.status().device_status == 0
    drafts = drafts.cpu().numpy()
    table = eng.block_table().cpu().numpy().copy()
    W = harness.device_weights(eng, cfg)
    lw = W["layers"][0]
    rl = eng.tensor("MOE_LOGITS", 0, torch.float32, (M, E)).cpu().numpy()
    ids = eng.tensor("MOE_IDS", 0, torch.int32, (M, tk)).cpu().numpy()
    o_ids, _ = model.moe_route(rl, tk)
    assert np.array_equal(o_ids, ids)
    inv = eng.tensor("MOE_INV", 0, torch.int32, (M, tk)).cpu().numpy()
    assert np.array_equal(np.sort(inv.reshape(-1)), np.arange(n))                 # a permutation of the entries
    dev = {"qkv": act_rows(eng, 0, M, d), "o": act_rows(eng, 1, M, Hq * dh), "gateup": act_rows(eng, 2, n, d),
           "down": act_rows(eng, 3, n, Fe), "lm_head": act_rows(eng, 4, M, d)}
    hidden = eng.tensor("HIDDEN", 0, torch.float32, (M, d)).cpu().numpy().astype(np.float64)
    worst_x = worst_l = 0.0
    low = {"gateup": 1.0, "down": 1.0}
    for b in checked:
        r0, r1 = b * R, (b + 1) * R
        n_past = int(seq_len[b])
        tokens = [int(last[b])] + [int(t) for t in drafts[b]]
        rec = {}
        entry = lambda t, j: {s: rows_of(dev[s], int(inv[r0 + t, j]), int(inv[r0 + t, j]) + 1) for s in ("gateup", "down")}
        cfg_f = dict(cfg, forced={s: rows_of(dev[s], r0, r1) for s in ("qkv", "o")}, forced_moe=entry, record_moe=rec)
        past = harness.LazyPast(eng, cfg, table[b], n_past, info["kv_pools"], 1)[0]
        x_out, _, _ = model.decoder_layer(cfg_f, lw, W["embed"][tokens].astype(np.float64), np.arange(n_past, n_past + R),
                                          past[0] if n_past else None, past[1] if n_past else None, router_logits=rl[r0:r1])
        worst_x = max(worst_x, float(np.abs(hidden[r0:r1] - x_out).max() / np.abs(x_out).max()))
        for (t, j), rr in rec.items():
            p = int(inv[r0 + t, j])
            low["gateup"] = min(low["gateup"], compare_rows(rows_of(dev["gateup"], p, p + 1), rr["gateup"], "gateup", 0.98))
            low["down"] = min(low["down"], compare_rows(rows_of(dev["down"], p, p + 1), rr["down"], "down", 0.90))
        ref_logits = model.proj(dict(cfg, forced={"lm_head": rows_of(dev["lm_head"], r0, r1)}), np.zeros((R, d)), W["lm_head"], "lm_head")
        logits = eng.logits(k)[b].cpu().numpy().reshape(R, V).astype(np.float64)
        worst_l = max(worst_l, float((np.abs(logits - ref_logits).max(-1) / np.abs(ref_logits).max(-1)).max()))
    print(f"w_fp8 MoE layer ({shape}): residual stream {worst_x:.2e}, logits {worst_l:.2e}, equal codes {low}")
    assert worst_x < 1e-5 and worst_l < 1e-5
    eng.close()
