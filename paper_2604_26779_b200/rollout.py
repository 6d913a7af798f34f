"""Multi-step rollout generation with continuous batching on top of the speculation step.

Responses of one rollout batch end at very different lengths (the long tail the paper's Section 5.1 describes), so a
fixed batch would run mostly empty towards the end.  Here every slot whose sequence is done takes the next prompt
(`spec_seq_replace`); the new prompt prefills through forced verify steps, k+1 prompt tokens per step, while the other
slots keep speculating; when no prompt is left the slot is retired, and once the queue is empty and few enough slots are
still running the batch is compacted (`spec_seq_compact`) so that the long tail does not drag the retired slots' rows through
every projection.  The draft length k may change from step to step
(`k_policy`), which is how a caller acts on the paper's observation that the useful k is narrow and depends on how
full the batch is (Section 4.2, Section 5.2).

Host code here only sequences calls of the C ABI and moves a few integers per step; all arithmetic runs in the library.
There are no end-of-sequence tokens in a synthetic workload, so a response ends after a given number of tokens.
"""
from __future__ import annotations

import dataclasses
from typing import Callable, Optional, Sequence

import numpy as np
import torch


def expected_tokens_per_step(alpha: float, k: int) -> float:
    """Tokens per step when each draft token is accepted independently with probability alpha:
    1 + alpha + ... + alpha^k (the accepted prefix plus the recovery / bonus token)."""
    a = min(max(float(alpha), 0.0), 1.0)
    return float(k + 1) if a >= 1.0 else (1.0 - a ** (k + 1)) / (1.0 - a)


def acceptance_rate(accepted_drafts: int, tried_drafts: int) -> float:
    """Estimate of alpha: accepted drafts over the draft positions that were tried (a step that accepted n < k drafts
    tried n+1 of them, one that accepted all k tried k)."""
    return float(accepted_drafts) / int(tried_drafts) if tried_drafts > 0 else 0.0


def choose_k(alpha: float, n_active: int, step_cost: Callable[[int, int], float], k_choices: Sequence[int]) -> int:
    """The k among k_choices with the highest modelled tokens per second: expected tokens per step (independent
    acceptance with rate alpha) over step_cost(n_active, k), the caller's model or measurement of one step's time."""
    best, best_rate = None, -1.0
    for k in k_choices:
        rate = expected_tokens_per_step(alpha, k) / float(step_cost(n_active, k))
        if rate > best_rate * (1.0 + 1e-12):
            best, best_rate = int(k), rate
    return best


@dataclasses.dataclass
class SequenceRecord:
    seq_id: int
    slot: int
    first_decode_step: int          # value of the step counter at this sequence's first sampled step
    tokens: list                    # response tokens (truncated to the requested length)
    ks: list                        # k of each of its decode steps
    slots: list = dataclasses.field(default_factory=list)   # slot it occupied at each decode step (compaction moves it)


@dataclasses.dataclass
class _Slot:
    seq_id: int = -1
    prompt: Optional[np.ndarray] = None
    cursor: int = 0                 # index in `prompt` of the slot's current last token while prefilling
    want: int = 0
    rec: Optional[SequenceRecord] = None

    @property
    def active(self):
        return self.seq_id >= 0

    @property
    def prefilling(self):
        return self.active and self.cursor < len(self.prompt) - 1


class Rollout:
    """Generates `response_lens[i]` tokens after `prompts[i]` for every i, with at most `eng.sc.max_batch` sequences in
    flight.  `k_policy(step, n_active, alpha_estimate) -> k` picks the draft length of each step (default: k_max)."""

    def __init__(self, eng, prompts, response_lens, free_stack, k_policy=None, compact_fraction=0.0, use_graphs=False):
        """compact_fraction: once the prompt queue is empty, the batch is compacted whenever the running sequences are
        at most this fraction of the slots (0 = never; 0.5 halves the batch at most log2(slots) times).
        use_graphs: steps in which no slot is prefilling replay a CUDA graph of the step (one per (batch size, k), captured
        on first use after a plain step of that kind; the key includes the previous step's k) - the thin tail is a chain of short kernels and replays ~10 % faster."""
        assert len(prompts) == len(response_lens) and len(prompts) > 0
        self.eng, self.sc = eng, eng.sc
        self.queue = [(i, np.ascontiguousarray(p, np.int32), int(w)) for i, (p, w) in enumerate(zip(prompts, response_lens))]
        assert all(len(p) >= 1 and w >= 1 for _, p, w in self.queue)
        self.k_policy = k_policy or (lambda step, n_active, alpha: self.sc.k_max)
        self.has_draft = self.sc.draft_kind != 0
        assert self.has_draft, "the rollout driver needs a draft kind (eagle3, mtp or ngram)"
        B = min(self.sc.max_batch, len(self.queue))
        self.slots = [_Slot() for _ in range(B)]
        first = []
        for s in self.slots:
            self._assign(s, self.queue.pop(0))
            first.append(int(s.prompt[0]))
        eng.seq_init(np.zeros(B, np.int32), np.asarray(first, np.int32), free_stack)
        for b, s in enumerate(self.slots):
            s.rec.slot = b
        self.done = {}
        self.step = 0
        self.k_trace, self.active_trace = [], []
        self._acc = [0, 0]          # accepted drafts, tried draft positions
        self.compact_fraction = float(compact_fraction)
        self.compactions = []       # (step, slots before, slots after)
        self.use_graphs = bool(use_graphs)
        self._graphs = {}           # (batch size, previous k, k) -> captured step; dropped when the batch is compacted
        self._plain_seen = set()    # keys that have run once the ordinary way
        self._last_k = None
        self.graph_steps = 0

    @staticmethod
    def _assign(slot, item):
        slot.seq_id, slot.prompt, slot.want = item
        slot.cursor = 0
        slot.rec = SequenceRecord(item[0], -1, -1, [], [])

    def _alpha(self):
        return acceptance_rate(*self._acc)

    def run_step(self):
        eng, B = self.eng, len(self.slots)
        n_active = sum(s.active for s in self.slots)
        first_step = self.step == 0
        needs_pending = self.sc.draft_kind in (1, 2)
        k = 0 if (first_step and needs_pending) else int(self.k_policy(self.step, n_active, self._alpha()))
        assert (k == 0 and first_step) or 1 <= k <= self.sc.k_max
        forced = {}
        for b, s in enumerate(self.slots):
            if s.prefilling:
                p, c = s.prompt, s.cursor
                r = len(p) - 1 - c                          # prompt tokens not yet fed
                d = np.zeros(k, np.int32)
                take = min(k, r)
                d[:take] = p[c + 1 : c + 1 + take]
                forced[b] = (d, k, int(p[c + k + 1])) if r > k else (d, r - 1, int(p[-1]))
        decoding = [b for b, s in enumerate(self.slots) if s.active and not s.prefilling]
        key = (B, self._last_k, k)                          # the draft head's first pass absorbs the previous step's k + 1 rows
        if self.use_graphs and k > 0 and not forced and decoding and key in self._plain_seen:
            if key not in self._graphs:
                self._graphs[key] = eng.capture_step(k)      # the capture itself executes nothing
            self._graphs[key].replay()
            self.graph_steps += 1
            self._finish_step(k, n_active, decoding, forced)
            return
        if k > 0:
            eng.draft(k)
        drafts = None
        if k > 0 and forced:
            drafts = eng.draft_tokens()[:, :k].clone().contiguous()
            idx = torch.as_tensor(sorted(forced), dtype=torch.long, device=drafts.device)
            rows = torch.as_tensor(np.stack([forced[b][0] for b in sorted(forced)]), dtype=torch.int32).to(drafts.device)
            drafts.index_copy_(0, idx, rows)
        eng.verify(k, drafts)
        if decoding:
            eng.reject_sample(k)
        if forced:
            fn = np.full(B, -1, np.int32)
            ft = np.zeros(B, np.int32)
            for b, (_, n, t) in forced.items():
                fn[b], ft[b] = n, t
            eng.kv_commit(torch.from_numpy(fn).to("cuda"), torch.from_numpy(ft).to("cuda"))
        else:
            eng.kv_commit()
            if k > 0 and decoding:
                self._plain_seen.add(key)
        self._finish_step(k, n_active, decoding, forced)

    def _finish_step(self, k, n_active, decoding, forced):
        eng = self.eng
        n_em = eng.n_emitted().cpu().numpy()
        out = eng.out_tokens(k).cpu().numpy()
        replace = []
        for b in decoding:
            s = self.slots[b]
            if s.rec.first_decode_step < 0:
                s.rec.first_decode_step = self.step
            s.rec.ks.append(k)
            s.rec.slots.append(b)
            s.rec.tokens += [int(t) for t in out[b, : n_em[b]]]
            self._acc[0] += int(n_em[b]) - 1
            self._acc[1] += min(int(n_em[b]), k)
            if len(s.rec.tokens) >= s.want:
                s.rec.tokens = s.rec.tokens[: s.want]
                self.done[s.seq_id] = s.rec
                replace.append(b)
        for b, (_, n, _) in forced.items():
            self.slots[b].cursor += n + 1
        if replace:
            lens, lasts = [], []
            for b in replace:
                if self.queue:
                    self._assign(self.slots[b], self.queue.pop(0))
                    self.slots[b].rec.slot = b
                    lens.append(0)
                    lasts.append(int(self.slots[b].prompt[0]))
                else:
                    self.slots[b] = _Slot()
                    lens.append(-1)
                    lasts.append(0)
            eng.seq_replace(replace, lens, lasts)
        if not self.queue and self.compact_fraction > 0.0:
            live = [b for b, s in enumerate(self.slots) if s.active]
            if 0 < len(live) <= self.compact_fraction * len(self.slots):
                eng.seq_compact(live)
                self.compactions.append((self.step, len(self.slots), len(live)))
                self.slots = [self.slots[b] for b in live]
                for j, s in enumerate(self.slots):
                    s.rec.slot = j
                self._graphs.clear()                         # graphs are tied to the batch size
                self._plain_seen.clear()
        self._last_k = k
        self.k_trace.append(k)
        self.active_trace.append(n_active)
        self.step += 1

    def run(self, max_steps=None):
        while any(s.active for s in self.slots):
            if max_steps is not None and self.step >= max_steps:
                break
            self.run_step()
        rep = self.eng.status()
        if rep.device_status != 0:
            raise RuntimeError(f"device status {rep.device_status} (detail {rep.device_detail})")
        return self.done
