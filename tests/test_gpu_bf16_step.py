"""GPU parity of whole speculation steps on the bf16 path (tcgen05 GEMMs with fused epilogues, tensor-core attention,
draft heads), at a size the oracle recomputes in seconds.  bf16 trajectories diverge from an fp64 oracle as soon as one
decision flips, so every stage is checked with teacher forcing on the device's own state:
  draft   oracle head run on the device's tapped hidden states / committed tokens / draft cache -> draft logits
  verify  oracle target forward on the device's tokens and cache bytes -> logits
  sample  oracle rejection rule on the device's logits -> decisions, lengths, tokens
  commit  lengths and block tables
Bars: logits within 2e-2 of the row maximum; sampler identical except inside the bands |u - min(1,p/q)| < 1e-4 and
|u - CDF edge| < 1e-6; integer state exact.
"""
import numpy as np
import pytest

import oracle
from oracle import harness, model
from paper_2604_26779_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def gather_pool(eng, which, blocks, n):
    pool = eng.kv_pool(which, 0)
    nb = -(-n // 16)
    idx = torch.as_tensor(np.ascontiguousarray(blocks[:nb]), dtype=torch.long, device="cuda")
    rows = pool[idx].permute(0, 2, 1, 3).reshape(nb * 16, pool.shape[1], pool.shape[3])[:n]
    if pool.dtype == torch.uint8:                # 8-bit cache: codes times the scale
        rows = rows.contiguous().view(torch.float8_e4m3fn).float() * (eng.sc.kv_scale_k if which.endswith("_K") else eng.sc.kv_scale_v)
    return rows.float().cpu().numpy()


def draft_head_weights(eng, cfg, kind):
    d, F = cfg["d_model"], cfg["d_ffn"]
    qn = (cfg["n_q_heads"] + 2 * cfg["n_kv_heads"]) * cfg["head_dim"]
    od = cfg["n_q_heads"] * cfg["head_dim"]
    td, f32 = eng.tdtype, torch.float32
    g = lambda name, shape, dt=td: eng.tensor(name, 0, dt, shape).float().cpu().numpy()
    gate, up = harness._split_gate_up(g("D_WGATEUP", (2 * F, d)))
    H = dict(norm_e=g("D_NORM_E", (d,), f32), norm_g=g("D_NORM_G", (d,), f32), mlp_norm=g("D_MLP_NORM", (d,), f32),
             wo=g("D_WO", (d, od)), wgate=gate, wup=up, wdown=g("D_WDOWN", (d, F)))
    if kind == "eagle3":
        H.update(wfc=g("D_WFC", (d, len(cfg["tap_layers"]) * d)), norm_f=g("D_NORM_F", (d,), f32),
                 wqkv=g("D_WQKV", (qn, 2 * d)), lm_head=g("D_LM_HEAD", (cfg["vocab"], d)))
    else:
        H.update(wproj=g("D_WPROJ", (d, 2 * d)), attn_norm=g("D_ATTN_NORM", (d,), f32), wqkv=g("D_WQKV", (qn, d)))
    return H


@pytest.mark.parametrize("kind,k,head_dim,kv_fp8,w_fp8", [("eagle3", 3, 64, None, False), ("mtp", 2, 64, None, False),
                                                           ("eagle3", 2, 128, None, "72 sequences"), ("mtp", 1, 64, None, "100 sequences"),
                                                           ("eagle3", 7, 64, None, False), ("eagle3", 5, 128, None, False),
                                                           ("mtp", 7, 128, None, False), ("eagle3", 3, 128, (1.0, 1.0), False),
                                                           ("mtp", 3, 128, (0.05, 0.03), False), ("eagle3", 3, 128, None, True),
                                                           ("eagle3", 3, 128, (1.0, 1.0), True),
                                                           ("mtp", 2, 128, None, True)])
def test_bf16_steps_stage_by_stage(kind, k, head_dim, kv_fp8, w_fp8):
    """head_dim 64: 16 or 32 query rows per KV head on the register-fragment attention kernel; head_dim 128 with k = 5 / 7:
    24 / 32 rows on the tcgen05 kernel, including the draft head's first pass, whose rows past the committed count carry
    position -1."""
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26779_b200 import workloads
    over = dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=head_dim, d_ffn=1024)
    # "N sequences": 65..256 rows per pass - two row tiles, the second ragged, few tiles per projection (split-K for the O and
    # down projections, fused epilogues on one or two tiles per CTA); every 9th sequence is checked
    many = int(w_fp8.split()[0]) if isinstance(w_fp8, str) else 0
    w_fp8 = w_fp8 is True
    if kv_fp8:                 # 8-bit cache: the oracle rounds every key and value to e4m3 exactly where the device stores it
        over["kv_fp8"] = kv_fp8
    if w_fp8:
        # 8-bit projections.  Quantising an activation row is a step function (a row maximum that rounds to the neighbouring
        # 16-bit value moves the whole row's codes), so two forwards that differ in one last place drift apart by about the
        # format's own noise: on the oracle alone, a 2^-12 relative perturbation of the activations moves the logits of this
        # model by 7 % of the row maximum, and the 8-bit forward sits 11 % from the 16-bit one.  The whole-forward logit bar
        # below therefore only catches gross errors; the products and quantisers are checked exactly, projection by projection
        # with the device's own rows, in test_gpu_w_fp8.py.  Draft, sampler and bookkeeping bars are unchanged.
        over["w_fp8"] = True
    logit_bar = 0.25 if w_fp8 else 2e-2
    draft_bar = 0.25 if (w_fp8 and kind == "mtp") else 2e-2      # the MTP head scores with the 8-bit LM head: the same step-function drift
    n_layers = 3
    lens = np.array([5, 40, 100, 17, 300], np.int32)
    if many:
        lens = np.random.default_rng(many).integers(3, 90, many).astype(np.int32)
    eng, info = workloads.build_dense_workload("c3", lens=lens, k=k, draft=kind, steps_budget=8, n_layers=n_layers,
                                               vocab=2048, cfg_over=over)
    cfg = info["cfg"]
    cfg = dict(cfg, tap_layers=inputs.default_tap_layers(n_layers) if kind == "eagle3" else (n_layers,))
    B, d, V = eng.B, cfg["d_model"], cfg["vocab"]
    W = harness.device_weights(eng, cfg)
    H = draft_head_weights(eng, cfg, kind)
    workloads.bootstrap(eng)
    worst_d = worst_v = 0.0
    boundary = 0
    k_prev = 0
    for step in range(4):
        # ---- state the draft starts from -------------------------------------------------------------------------
        seq_len = eng.seq_len().cpu().numpy().copy()
        n_prev = eng.n_emitted().cpu().numpy().copy()
        toks_prev = eng.out_tokens(k_prev).cpu().numpy().copy()
        table = eng.block_table().cpu().numpy().copy()
        if kind == "eagle3":
            feats = eng.tensor("TAPS", 0, eng.tdtype, (B, k_prev + 1, len(cfg["tap_layers"]) * d)).float().cpu().numpy()
        else:
            feats = eng.tensor("HIDDEN", 0, torch.float32, (B, k_prev + 1, d)).cpu().numpy().copy()
        last = eng.tensor("LAST_TOKEN", 0, torch.int32, (B,)).cpu().numpy().copy()
        eng.draft(k)
        g_drafts = eng.draft_tokens().cpu().numpy()[:, :k].copy()
        g_dlog = eng.draft_logits(k).cpu().numpy().copy()
        draft_step = int(eng.status().steps)
        checked = range(0, B, 9) if many else range(B)
        for b in checked:
            base = int(seq_len[b] - n_prev[b])
            pk, pv = gather_pool(eng, "DRAFT_KV_K", table[b], base), gather_pool(eng, "DRAFT_KV_V", table[b], base)
            _, _, dlog = model.draft_propose(cfg, W, H, kind, feats[b, : n_prev[b]], toks_prev[b, : n_prev[b]], k,
                                             lambda i, lg: (int(g_drafts[b, i]), oracle.softmax(np.asarray(lg, np.float32)[None])[0]),
                                             pk if base > 0 else None, pv if base > 0 else None, first_slot=base)
            worst_d = max(worst_d, float((np.abs(g_dlog[b] - dlog).max(-1) / np.abs(dlog).max(-1)).max()))
            # the device's draft tokens are inverse-CDF draws from its own q with the stream-1 uniforms
            ud = oracle.uniforms(info["seed"], draft_step, 1, b + 1, k)[b]
            for i in range(k):
                t, mg = oracle.invcdf(oracle.softmax(g_dlog[b, i][None])[0], ud[i])
                assert t == g_drafts[b, i] or mg < 1e-5, (step, b, i, t, g_drafts[b, i], mg)
        # ---- verify + sample ---------------------------------------------------------------------------------------
        eng.verify(k)
        eng.reject_sample(k)
        g_logits = eng.logits(k).cpu().numpy().copy()
        g_out, g_n = eng.out_tokens(k).cpu().numpy().copy(), eng.n_emitted().cpu().numpy().copy()
        for b in checked:
            r = harness.oracle_verify_sample(eng, cfg, W, b, [int(last[b])] + [int(x) for x in g_drafts[b]], int(seq_len[b]),
                                             table[b], info["kv_pools"], g_dlog[b], info["seed"], draft_step)
            worst_v = max(worst_v, float((np.abs(g_logits[b] - r["logits"]).max(-1) / np.abs(r["logits"]).max(-1)).max()))
            if kv_fp8 and b == 1:
                # what the step appended to the 8-bit cache of the first layer: the oracle's keys and values of the k+1 new
                # positions, rounded to e4m3 by the oracle.  The device rounds fp32 results of bf16 GEMMs, the oracle fp64 ones,
                # so a value near a rounding boundary (small values above all) may land on the neighbouring code: most codes equal, none further
                # than one step (2^-3 relative) away.
                tokens_in = [int(last[b])] + [int(x) for x in g_drafts[b]]
                fw = model.target_forward(dict(cfg, n_layers=1), dict(W, layers=[W["layers"][0]]), tokens_in,
                                          past=harness.LazyPast(eng, cfg, table[b], int(seq_len[b]), info["kv_pools"], 1),
                                          start_pos=int(seq_len[b]))
                for which, ref in (("KV_K", fw["new_kv"][0][0]), ("KV_V", fw["new_kv"][0][1])):
                    n_all = int(seq_len[b]) + k + 1
                    dev = gather_pool(eng, which, eng.block_table().cpu().numpy()[b], n_all)[int(seq_len[b]):]
                    same = np.mean(dev == ref.astype(np.float32))
                    # one code step (2^-3 of the value) plus the absolute error of the bf16 computation that fed the rounding
                    step_ok = np.all(np.abs(dev - ref) <= 0.126 * np.abs(ref) + 8e-3 * np.sqrt(np.mean(ref ** 2)))
                    assert same > 0.85 and step_ok, (which, same)
            p, q = oracle.softmax(g_logits[b]), oracle.softmax(g_dlog[b])
            u = oracle.uniforms(info["seed"], draft_step, 0, b + 1, k + 1)[b]
            toks, n_o, _, mg = oracle.reject_sample_seq(p, q, g_drafts[b], u)
            if n_o != g_n[b] or not np.array_equal(toks, g_out[b]):
                assert np.any(mg[:k] < 1e-4) or mg[k] < 1e-6, (step, b, toks, g_out[b], mg)
                boundary += 1
        eng.kv_commit()
        assert eng.status().device_status == 0
        assert np.array_equal(eng.seq_len().cpu().numpy(), seq_len + g_n)
        k_prev = k
    print(f"bf16 {kind} k={k} dh={head_dim} kv_fp8={kv_fp8} w_fp8={w_fp8}: draft logits {worst_d:.2e}, verify logits {worst_v:.2e}, "
          f"boundary cases {boundary}")
    assert worst_d < draft_bar and worst_v < logit_bar and boundary <= 2
    eng.close()
