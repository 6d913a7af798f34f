"""CPU oracle for a chain of speculation steps on one sequence, without any KV cache.

TEST INFRASTRUCTURE ONLY.  Every step recomputes the whole causal forward from the committed tokens, so a
stale or misplaced cache slot in the implementation under test shows up as a mismatch at the next step.

One step (paper: Introduction, third paragraph; Section 2.2 for "tokens produced per step"):
  state   committed tokens t[0..L-1]; the last one, x_last = t[L-1], has not been fed to the target yet
  draft   q_i = softmax(draft logits / T), d_i = invcdf(q_i, U(step, seq, i-1, stream 1)),  i = 1..k
  verify  p_i = softmax(target logits of [t, d_1..d_{i-1}] / T),  i = 1..k+1  (one causal forward)
  accept  rejection rule of spec_oracle.c with uniforms U(step, seq, 0..k, stream 0)
  commit  t <- t + [d_1..d_n, token]
"""
from __future__ import annotations

import numpy as np

import oracle
from oracle import model


class ChainOracle:
    def __init__(self, cfg, W, H, kind, seed, seq_index, prompt, step0=0):
        self.cfg, self.W, self.H, self.kind = cfg, W, H, kind
        self.seed, self.seq = int(seed), int(seq_index)
        self.tokens = [int(t) for t in prompt]
        self.step = int(step0)
        self.T = float(cfg.get("temperature", 1.0))

    def step_once(self, k, forced_drafts=None):
        cfg, W = self.cfg, self.W
        t = self.tokens
        L = len(t)
        taps_layers = tuple(cfg["tap_layers"])
        rec = {}
        if forced_drafts is None and self.kind == "ngram":
            drafts = model.ngram_propose(t, int(cfg.get("ngram_n", 3)), k)
            q = np.zeros((k, cfg["vocab"]), np.float32)
            q[np.arange(k), drafts] = 1.0
        elif forced_drafts is None:
            feats = model.target_forward(cfg, W, t[: L - 1], tap_layers=taps_layers)["taps"]   # positions 0..L-2
            u_draft = oracle.uniforms(self.seed, self.step, 1, self.seq + 1, max(k, 1))[self.seq]

            def sample_fn(i, logits_row):
                lg = np.asarray(logits_row, np.float32)
                if cfg.get("draft_greedy"):                 # deterministic draft: arg-max (lowest id among equals), q = one-hot
                    tok = int(np.argmax(lg))
                    q = np.zeros(lg.shape[0], np.float32)
                    q[tok] = 1.0
                    return tok, q
                q = oracle.softmax(lg[None, :], self.T)[0]
                tok, _ = oracle.invcdf(q, u_draft[i])
                return tok, q

            drafts, q, dlog = model.draft_propose(cfg, W, self.H, self.kind, feats, t[1:L], k, sample_fn)
            rec["draft_logits"] = dlog
        else:
            drafts, q = np.asarray(forced_drafts[0], np.int32), np.asarray(forced_drafts[1], np.float32)
        out = model.target_forward(cfg, W, t + [int(d) for d in drafts], tap_layers=taps_layers)
        tl = out["logits"][L - 1 : L + k].astype(np.float32)
        p = oracle.softmax(tl, self.T)
        u = oracle.uniforms(self.seed, self.step, 0, self.seq + 1, k + 1)[self.seq]
        toks, n_emit, flags, margins = oracle.reject_sample_seq(p, q, drafts, u)
        rec.update(drafts=drafts, q=q, p=p, target_logits=tl, out_tokens=toks, n_emitted=n_emit,
                   margins=margins, flags=flags, taps=out["taps"][L - 1 : L + k], len_before=L - 1)
        self.tokens = t + [int(x) for x in toks[:n_emit]]
        self.step += 1
        return rec
