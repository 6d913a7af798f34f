"""CPU oracle for the model side of one speculation step: target forward, EAGLE-3-style and MTP-style
draft heads, in numpy fp64, one sequence at a time.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's CPU-baseline leg.
The CUDA path shares nothing with this file.

What it follows.  The paper names the pieces without giving formulas: a target model that verifies the
draft tokens in one forward (Introduction, third paragraph), decode phase only (Section 2.2), and two
drafting paths (Section 2.3): a general one-layer EAGLE-3 head driven by target hidden states and a native
multi-token-prediction head.  The architecture used is the reading chosen for this build:

* target: pre-norm decoder.  x = E[token]; per layer  h = RMSNorm(x), (q,k,v) = W_qkv h, rotary position
  embedding on q and k with the half-split pairing (j, j + dh/2) and angle pos * theta^(-2j/dh),
  scores q.k/sqrt(dh), causal softmax, x += W_o attn; then x += W_down(silu(W_gate m) * (W_up m)) with
  m = RMSNorm(x) (or the mixture-of-experts variant below); logits = W_lm RMSNorm(x).  No biases, no QK
  norm, separate E and W_lm.  A weight matrix is stored [out][in].
* mixture of experts: router logits W_r m, softmax over experts, the top_k largest (ties: lower index),
  weights renormalised to sum 1, output sum_e w_e Expert_e(m); no capacity limit.
* EAGLE-3-style head, slot j (input token t_{j+1}, predicts t_{j+2}): e = E[t_{j+1}];
  g = W_fc concat(taps_j) when the target has processed position j, else the head's own output of slot
  j-1; a = concat(RMSNorm_e(e), RMSNorm_g(g)); (q,k,v) = W_qkv a; rotary at position j; causal attention
  over the head's own slots; h1 = g + W_o attn; h2 = h1 + SwiGLU(RMSNorm_m(h1)); logits = W_lm' RMSNorm_f(h2).
* MTP-style head, same slots: h0 = W_proj concat(RMSNorm_g(g), RMSNorm_e(e)); one ordinary decoder layer;
  logits = the target's own final norm and LM head; g of a speculative slot = the layer's previous output.
* taps: the residual stream after a given number of layers (0 = the embedding output).

Pins (tests/test_oracle_model.py): the whole target forward against the transformers library's Llama
implementation with the same weights; softmax, attention and RMSNorm against scipy / torch library
routines; rotary invariants; forward-with-past equals the matching rows of a recompute-all forward; the
expert mixture against a brute-force dense evaluation.  The two draft heads are this build's own
definitions: PARITY UNPINNED by the paper for them beyond the layer function they share with the target.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def rmsnorm(x, w, eps):
    x = np.asarray(x, F64)
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * np.asarray(w, F64)


def rope(x, pos, theta):
    """x [T][H][dh], pos [T] absolute positions.  Pairs (j, j+dh/2) rotate by pos * theta^(-2j/dh)."""
    x = np.asarray(x, F64)
    T, H, dh = x.shape
    half = dh // 2
    j = np.arange(half, dtype=F64)
    inv = theta ** (-2.0 * j / dh)
    ang = np.asarray(pos, F64)[:, None] * inv[None, :]          # [T][half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def softmax_rows(z):
    z = np.asarray(z, F64)
    z = z - z.max(axis=-1, keepdims=True)
    e = np.exp(z)
    return e / e.sum(axis=-1, keepdims=True)


def attention(q, k_all, v_all, n_past):
    """q [T][Hq][dh]; k_all, v_all [n_past+T][Hkv][dh]; query t sees keys 0..n_past+t (causal)."""
    T, Hq, dh = q.shape
    Hkv = k_all.shape[1]
    group = Hq // Hkv
    out = np.zeros((T, Hq, dh), F64)
    for t in range(T):
        n_vis = n_past + t + 1
        for h in range(Hq):
            kh = k_all[:n_vis, h // group, :]
            vh = v_all[:n_vis, h // group, :]
            s = kh @ q[t, h] / np.sqrt(float(dh))
            out[t, h] = softmax_rows(s[None, :])[0] @ vh
    return out


def silu(x):
    return x / (1.0 + np.exp(-x))


def dense_mlp(lw, m, cfg=None):
    if cfg is None or not cfg.get("w_fp8"):
        return (silu(m @ np.asarray(lw["wgate"], F64).T) * (m @ np.asarray(lw["wup"], F64).T)) @ np.asarray(lw["wdown"], F64).T
    return proj(cfg, silu(proj(cfg, m, lw["wgate"], "gateup")) * proj(cfg, m, lw["wup"], "gateup"), lw["wdown"], "down")


def moe_route(router_logits, top_k):
    """Returns (expert ids [T][top_k], weights [T][top_k]); ties resolved towards the lower index."""
    probs = softmax_rows(router_logits)
    T, E = probs.shape
    ids = np.zeros((T, top_k), np.int64)
    wts = np.zeros((T, top_k), F64)
    for t in range(T):
        order = sorted(range(E), key=lambda e: (-probs[t, e], e))[:top_k]
        ids[t] = order
        wts[t] = probs[t, order] / probs[t, order].sum()
    return ids, wts


def moe_mlp(lw, m, top_k, router_logits=None, cfg=None):
    """router_logits, when given, replaces W_r m as the input of the top-k decision (used to take that integer
    decision on the same numbers as an implementation under test).

    With cfg["w_fp8"] the experts' three projections go through the 8-bit format (proj), the router does not.  For checks
    on given quantised rows, cfg["forced_moe"](t, j) returns the `forced` dict of token t's j-th expert entry, and
    cfg["record_moe"][(t, j)] receives what was quantised here."""
    ids, wts = moe_route(m @ np.asarray(lw["router"], F64).T if router_logits is None else np.asarray(router_logits, F64), top_k)
    out = np.zeros_like(m)
    w8 = cfg is not None and cfg.get("w_fp8")
    for t in range(m.shape[0]):
        for j, (e, w) in enumerate(zip(ids[t], wts[t])):
            if not w8:
                g = np.asarray(lw["experts_gate"][e], F64)
                u = np.asarray(lw["experts_up"][e], F64)
                d = np.asarray(lw["experts_down"][e], F64)
                out[t] += w * ((silu(g @ m[t]) * (u @ m[t])) @ d.T)
                continue
            c = dict(cfg, forced=cfg["forced_moe"](t, j) if cfg.get("forced_moe") else None, record={})
            row = m[t : t + 1]
            act = silu(proj(c, row, lw["experts_gate"][e], "gateup")) * proj(c, row, lw["experts_up"][e], "gateup")
            out[t] += w * proj(c, act, lw["experts_down"][e], "down")[0]
            if cfg.get("record_moe") is not None:
                cfg["record_moe"][(t, j)] = c["record"]
    return out


def ep_receive_layout(ids_by_rank, n_experts, ep_size):
    """Expert parallelism over ep_size ranks (the paper's 235B-A22B configuration spans many GPUs, Section 5.1): rank r
    owns the experts [r * E/ep_size, (r+1) * E/ep_size) and every rank routes its own tokens.  ids_by_rank[s] is the
    [M_s][top_k] expert choice of source rank s.  Returns, for every destination rank d, the rows it receives, in the
    order it stores them: its experts ascending; within an expert the source ranks ascending; within a source the
    entries (token, slot) in row-major order.  Each row is (expert, source rank, source token, slot).  Also returns
    recv_off[d][local expert][source] = index of the first row of that (expert, source) run."""
    assert n_experts % ep_size == 0
    per = n_experts // ep_size
    rows, recv_off = [], []
    for d in range(ep_size):
        r, off = [], np.zeros((per, ep_size), np.int64)
        for el in range(per):
            e = d * per + el
            for s in range(ep_size):
                off[el, s] = len(r)
                ids = np.asarray(ids_by_rank[s])
                for m in range(ids.shape[0]):
                    for j in range(ids.shape[1]):
                        if ids[m, j] == e:
                            r.append((e, s, m, j))
        rows.append(r)
        recv_off.append(off)
    return rows, recv_off


def ep_moe_mlp(lw, m_by_rank, top_k, ep_size, router_logits_by_rank=None):
    """The mixture-of-experts MLP computed the expert-parallel way: route locally, send every (token, slot) row to the
    rank that owns its expert, run each local expert on the rows it received, return the outputs to the source rank and
    add them there in slot order with the routing weights.  Returns the list of per-rank outputs [M_s][d]."""
    E = np.asarray(lw["router"]).shape[0]
    ids_by, wts_by = [], []
    for s in range(ep_size):
        m = np.asarray(m_by_rank[s], F64)
        lg = m @ np.asarray(lw["router"], F64).T if router_logits_by_rank is None else np.asarray(router_logits_by_rank[s], F64)
        ids, wts = moe_route(lg, top_k)
        ids_by.append(ids)
        wts_by.append(wts)
    rows, _ = ep_receive_layout(ids_by, E, ep_size)
    back = [dict() for _ in range(ep_size)]                  # per source rank: (token, slot) -> expert output row
    for d in range(ep_size):
        for (e, s, t, j) in rows[d]:
            x = np.asarray(m_by_rank[s], F64)[t]                                     # dispatch: the row crosses to rank d
            g = np.asarray(lw["experts_gate"][e], F64)
            u = np.asarray(lw["experts_up"][e], F64)
            dn = np.asarray(lw["experts_down"][e], F64)
            back[s][(t, j)] = (silu(g @ x) * (u @ x)) @ dn.T                          # combine: the row crosses back
    out = []
    for s in range(ep_size):
        m = np.asarray(m_by_rank[s], F64)
        o = np.zeros_like(m)
        for t in range(m.shape[0]):
            for j in range(top_k):
                o[t] += wts_by[s][t, j] * back[s][(t, j)]
        out.append(o)
    return out


def _bf16_round(x):
    """fp32 values rounded to bf16 (round to nearest even), as fp32."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)).view(np.float32)
    return r


class QuantRows:
    """A weight matrix that is already stored in the 8-bit format: e4m3 codes [rows][k] and one fp32 scale per row.  Its
    value is the exact product code x scale; proj() uses it as it stands instead of quantising 16-bit weights again."""

    def __init__(self, codes, scales):
        self.codes = np.ascontiguousarray(codes, np.uint8)
        self.scales = np.ascontiguousarray(scales, np.float32)
        assert self.codes.ndim == 2 and self.scales.shape == (self.codes.shape[0],)

    def values(self):
        import oracle
        return oracle.e4m3_dequantize(self.codes).reshape(self.codes.shape).astype(F64) * self.scales.astype(F64)[:, None]


def rows_8bit(x):
    """Every row of x as its 8-bit representation: e4m3 codes of x / scale times the row's scale amax / 448, in fp64."""
    import oracle
    codes, scales = oracle.e4m3_quantize_rows(np.asarray(x, np.float32))
    return QuantRows(codes, scales).values()


def proj(cfg, x, W, stage=None):
    """x W^T of a target projection.  With cfg["w_fp8"] both operands go through the 8-bit format first (the precision the
    paper's simulator assumes, Section 5.1): the activation rows as the 16-bit values the layer before produced, each row
    of x and each row of W with its own scale amax / 448; the product itself is exact.  W is either the 16-bit matrix
    (quantised here) or a QuantRows holding the stored codes and scales.

    Quantising is a step function of its input, so two computations whose activations differ in the last 16-bit place
    drift apart by whole code steps.  For checks that must not depend on that, `stage` names the projection ("qkv", "o",
    "gateup", "down", "lm_head"): cfg["record"][stage], when the dict is there, receives the rows as quantised here, and
    cfg["forced"][stage], when present, is a QuantRows that replaces them in the product (single-layer calls only: every
    layer of a multi-layer forward would see the same entry)."""
    if not cfg.get("w_fp8"):
        return x @ np.asarray(W, F64).T
    import oracle
    own = QuantRows(*oracle.e4m3_quantize_rows(_bf16_round(np.asarray(x, np.float32))))
    if stage is not None and cfg.get("record") is not None:
        cfg["record"][stage] = own
    forced = (cfg.get("forced") or {}).get(stage) if stage is not None else None
    xq = (own if forced is None else forced).values()
    wq = W.values() if isinstance(W, QuantRows) else rows_8bit(W)
    return xq @ wq.T


def kv_as_cached(cfg, k, v):
    """What the attention reads back for freshly computed keys and values: themselves, or, with an 8-bit cache
    (cfg["kv_fp8"] = (k_scale, v_scale)), their e4m3 codes times the scale - for the new positions as for the old ones,
    since every position is attended to through the cache."""
    if not cfg.get("kv_fp8"):
        return k, v
    import oracle
    ks, vs = cfg["kv_fp8"]
    return (oracle.e4m3_roundtrip(np.asarray(k, np.float32), ks).astype(F64),
            oracle.e4m3_roundtrip(np.asarray(v, np.float32), vs).astype(F64))


def decoder_layer(cfg, lw, x, pos, past_k=None, past_v=None, attn_in=None, router_logits=None):
    """One pre-norm decoder layer on rows x [T][d] at absolute positions pos.

    past_k / past_v [n_past][Hkv][dh] are cached (already rotated) keys and values, or None.
    attn_in, when given, replaces RMSNorm(x) as the input of the QKV projection (the EAGLE-3 head feeds a
    2d-wide concatenation there).  Returns (x_out, k_new, v_new)."""
    Hq, Hkv, dh = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    T = x.shape[0]
    h = rmsnorm(x, lw["attn_norm"], cfg["rms_eps"]) if attn_in is None else attn_in
    qkv = proj(cfg, h, lw["wqkv"], "qkv")
    q = qkv[:, : Hq * dh].reshape(T, Hq, dh)
    k = qkv[:, Hq * dh : (Hq + Hkv) * dh].reshape(T, Hkv, dh)
    v = qkv[:, (Hq + Hkv) * dh :].reshape(T, Hkv, dh)
    q = rope(q, pos, cfg["rope_theta"])
    k = rope(k, pos, cfg["rope_theta"])
    k, v = kv_as_cached(cfg, k, v)
    n_past = 0 if past_k is None else past_k.shape[0]
    k_all = k if n_past == 0 else np.concatenate([np.asarray(past_k, F64), k], axis=0)
    v_all = v if n_past == 0 else np.concatenate([np.asarray(past_v, F64), v], axis=0)
    att = attention(q, k_all, v_all, n_past).reshape(T, Hq * dh)
    x = x + proj(cfg, att, lw["wo"], "o")
    m = rmsnorm(x, lw["mlp_norm"], cfg["rms_eps"])
    if cfg.get("n_experts", 0) > 0:
        x = x + moe_mlp(lw, m, cfg["experts_top_k"], router_logits, cfg)
    else:
        x = x + dense_mlp(lw, m, cfg)
    return x, k, v


def target_forward(cfg, W, tokens, past=None, start_pos=0, tap_layers=(), router_logits=None):
    """Target forward over `tokens` placed at positions start_pos, start_pos+1, ...

    past: None (recompute-all, no cache) or a list, per layer, of (K [n_past][Hkv][dh], V likewise).
    Returns dict(logits [T][V], taps [T][len(tap_layers)*d], final [T][d] (residual before the final norm),
    new_kv = per layer (k, v) of the T new positions)."""
    tokens = np.asarray(tokens, np.int64)
    T = tokens.shape[0]
    pos = start_pos + np.arange(T)
    x = np.asarray(W["embed"], F64)[tokens]
    taps = {}
    if 0 in tap_layers:
        taps[0] = x
    new_kv = []
    for l, lw in enumerate(W["layers"]):
        pk, pv = (None, None) if past is None else past[l]
        x, k, v = decoder_layer(cfg, lw, x, pos, pk, pv, router_logits=None if router_logits is None else router_logits[l])
        new_kv.append((k, v))
        if (l + 1) in tap_layers:
            taps[l + 1] = x
    logits = proj(cfg, rmsnorm(x, W["final_norm"], cfg["rms_eps"]), W["lm_head"], "lm_head")
    tap_cat = np.concatenate([taps[t] for t in tap_layers], axis=-1) if tap_layers else np.zeros((T, 0))
    return {"logits": logits, "taps": tap_cat, "final": x, "new_kv": new_kv}


def _swiglu_block(cfg, hw, h1):
    m = rmsnorm(h1, hw["mlp_norm"], cfg["rms_eps"])
    return h1 + dense_mlp(hw, m)


def eagle3_slots(cfg, W, H, g, tokens_next, pos, past_k=None, past_v=None):
    """EAGLE-3-style head on consecutive slots.  g [T][d] feature rows (already W_fc-projected taps or the
    head's own previous outputs), tokens_next [T] = t_{j+1} of each slot, pos [T] slot indices.
    Returns (h2 [T][d], k_new, v_new)."""
    Hq, Hkv, dh = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    T = g.shape[0]
    e = np.asarray(W["embed"], F64)[np.asarray(tokens_next, np.int64)]
    a = np.concatenate([rmsnorm(e, H["norm_e"], cfg["rms_eps"]), rmsnorm(g, H["norm_g"], cfg["rms_eps"])], axis=-1)
    qkv = a @ np.asarray(H["wqkv"], F64).T
    q = rope(qkv[:, : Hq * dh].reshape(T, Hq, dh), pos, cfg["rope_theta"])
    k = rope(qkv[:, Hq * dh : (Hq + Hkv) * dh].reshape(T, Hkv, dh), pos, cfg["rope_theta"])
    v = qkv[:, (Hq + Hkv) * dh :].reshape(T, Hkv, dh)
    k, v = kv_as_cached(cfg, k, v)
    n_past = 0 if past_k is None else past_k.shape[0]
    k_all = k if n_past == 0 else np.concatenate([past_k, k], axis=0)
    v_all = v if n_past == 0 else np.concatenate([past_v, v], axis=0)
    att = attention(q, k_all, v_all, n_past).reshape(T, Hq * dh)
    h1 = g + att @ np.asarray(H["wo"], F64).T
    h2 = _swiglu_block(cfg, H, h1)
    return h2, k, v


def eagle3_logits(cfg, H, h2):
    return rmsnorm(h2, H["norm_f"], cfg["rms_eps"]) @ np.asarray(H["lm_head"], F64).T


def mtp_slots(cfg, W, H, g, tokens_next, pos, past_k=None, past_v=None):
    """MTP-style head on consecutive slots; returns (h_out [T][d], k_new, v_new)."""
    e = np.asarray(W["embed"], F64)[np.asarray(tokens_next, np.int64)]
    cat = np.concatenate([rmsnorm(g, H["norm_g"], cfg["rms_eps"]), rmsnorm(e, H["norm_e"], cfg["rms_eps"])], axis=-1)
    h0 = cat @ np.asarray(H["wproj"], F64).T
    return decoder_layer(cfg, H, h0, pos, past_k, past_v)


def mtp_logits(cfg, W, h):
    return proj(cfg, rmsnorm(h, W["final_norm"], cfg["rms_eps"]), W["lm_head"], "lm_head")     # the target's LM head, in its format


def draft_propose(cfg, W, H, kind, true_feat, tokens, k, sample_fn, past_k=None, past_v=None, first_slot=0):
    """Runs a draft head over the true slots first_slot..first_slot+S-1 and then k-1 speculative slots.

    true_feat [S][T*d]: tapped target hidden states of the true slots (EAGLE-3: three taps, projected here
    by W_fc; MTP: the last-layer residual).  tokens [S]: t_{j+1} of each true slot (the last one is the
    most recent committed token).  past_k/past_v: the head's cached keys/values of slots < first_slot, or
    None.  sample_fn(i, logits_row) -> (token d_{i+1}, q_{i+1} as the fp32 probabilities it was drawn from);
    the caller supplies it so that the softmax and the inverse CDF are the C oracle's.
    Returns (draft tokens [k], q [k][V] fp32 probabilities, logits [k][V or draft vocabulary] fp64)."""
    S = true_feat.shape[0]
    pos = first_slot + np.arange(S)
    if kind == "eagle3":
        g = np.asarray(true_feat, F64) @ np.asarray(H["wfc"], F64).T
        h, kk, vv = eagle3_slots(cfg, W, H, g, tokens, pos, past_k, past_v)
    else:
        g = np.asarray(true_feat, F64)
        h, kk, vv = mtp_slots(cfg, W, H, g, tokens, pos, past_k, past_v)
    k_all = kk if past_k is None else np.concatenate([past_k, kk], axis=0)
    v_all = vv if past_v is None else np.concatenate([past_v, vv], axis=0)
    drafts, q_rows, logit_rows = [], [], []
    h_last = h[-1:]
    slot = first_slot + S - 1
    for i in range(k):
        lg = eagle3_logits(cfg, H, h_last)[0] if kind == "eagle3" else mtp_logits(cfg, W, h_last)[0]
        d, q = sample_fn(i, lg)
        if H.get("d2t") is not None:        # the head's own vocabulary: row r scores target token d2t[r], q is zero elsewhere
            d2t = np.asarray(H["d2t"], np.int64)
            q_full = np.zeros(cfg["vocab"], np.float32)
            q_full[d2t] = q
            d, q = int(d2t[int(d)]), q_full
        drafts.append(int(d))
        q_rows.append(q)
        logit_rows.append(lg)
        if i == k - 1:
            break
        slot += 1
        if kind == "eagle3":
            h_last, kk, vv = eagle3_slots(cfg, W, H, h_last, [d], np.array([slot]), k_all, v_all)
        else:
            h_last, kk, vv = mtp_slots(cfg, W, H, h_last, [d], np.array([slot]), k_all, v_all)
        k_all = np.concatenate([k_all, kk], axis=0)
        v_all = np.concatenate([v_all, vv], axis=0)
    return np.array(drafts, np.int32), np.stack(q_rows), np.stack(logit_rows)


def ngram_propose(tokens, n_max, k):
    """Model-free drafting (the paper's n-gram baseline, Section 4.2): find the most recent earlier occurrence of the
    trailing n tokens of `tokens` (n = n_max down to 1; a match must be followed by at least one token), propose the k
    tokens that followed it, repeating the last proposed token once the sequence ends; without any match the last
    token is repeated.  The proposal distribution is one-hot."""
    t = [int(x) for x in tokens]
    L = len(t)
    start, n_found = -1, 0
    for n in range(min(n_max, L - 1), 0, -1):
        for s in range(L - 1 - n, -1, -1):
            if t[s : s + n] == t[L - n :]:
                start, n_found = s, n
                break
        if start >= 0:
            break
    out, prev = [], t[-1]
    for i in range(k):
        p = start + n_found + i
        prev = t[p] if (start >= 0 and p <= L - 1) else prev
        out.append(prev)
    return np.array(out, np.int32)
