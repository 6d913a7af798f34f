"""Batch compaction (spec_seq_compact) in the middle of a run: the kept sequences move to the front slots, everything
else is retired, and the run continues on the smaller batch in lock-step with the cache-free oracle chains (a moved
sequence draws from its NEW slot's Philox stream), with the block bookkeeping equal to the oracle's bit for bit.
fp32 tiny workload: tokens, accepted lengths and tables identical except at counted boundary cases."""
import numpy as np
import pytest

import oracle
from oracle.chain import ChainOracle
from paper_2604_26779_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def weights_for(cfg, kind, case):
    W = inputs.make_target_weights(cfg, seed=inputs.sub_seed(case, 0))
    if kind == "ngram":
        return W, None
    return W, (inputs.make_eagle3_weights if kind == "eagle3" else inputs.make_mtp_weights)(cfg, seed=inputs.sub_seed(case, 1))


@pytest.mark.parametrize("kind,keep", [("eagle3", [1, 3]), ("mtp", [0, 2, 3]), ("ngram", [2])])
def test_compaction_mid_run_stays_in_lockstep(kind, keep):
    from paper_2604_26779_b200 import engine
    cfg = dict(inputs.model_config("c1"))
    if kind == "mtp":
        cfg["tap_layers"] = (cfg["n_layers"],)
    if kind == "ngram":
        cfg["ngram_n"] = 3
    B, k, seed, bt = 4, 3, 777, 16
    R = k + 1
    W, H = weights_for(cfg, kind, 5)
    prompts = inputs.make_prompts(B, 16, cfg["vocab"], seed=inputs.sub_seed(5, 2))
    max_blocks = 8
    sc = engine.make_spec_config(cfg, draft_kind=kind, k_max=k, max_batch=B, kv_num_blocks=4 * max_blocks + 2,
                                 max_blocks_per_seq=max_blocks, seed=seed)
    eng = engine.SpecStep(sc)
    eng.load_target_weights(W)
    if H is not None:
        eng.load_draft_weights(H)
    order = inputs.make_block_order(sc.kv_num_blocks, inputs.sub_seed(5, 3))
    eng.seq_init(np.zeros(B, np.int32), prompts[:, 0], order)
    o_len, o_table = np.zeros(B, np.int32), np.full((B, max_blocks), -1, np.int32)
    o_free, o_top = order.copy(), np.array([sc.kv_num_blocks], np.int32)

    def books_equal():
        n = eng.B
        assert np.array_equal(eng.seq_len().cpu().numpy()[:n], o_len)
        assert np.array_equal(eng.block_table().cpu().numpy()[:n], o_table)
        top = int(eng.tensor("FREE_TOP", 0, torch.int32, (1,)).item())
        assert top == int(o_top[0])
        assert np.array_equal(eng.tensor("FREE_STACK", 0, torch.int32, (sc.kv_num_blocks,)).cpu().numpy()[:top], o_free[:top])

    def step(forced):
        n = eng.B
        if eng.status().steps > 0 or kind == "ngram":
            eng.draft(k)
        drafts = eng.draft_tokens()[:n, :k].clone().contiguous()
        fn = torch.full((n,), -1, dtype=torch.int32)
        ft = torch.zeros((n,), dtype=torch.int32)
        for b, (d, nn, t) in forced.items():
            drafts[b] = torch.as_tensor(np.asarray(d, np.int32)).cuda()
            fn[b], ft[b] = nn, int(t)
        eng.verify(k, drafts)
        if len(forced) < n:
            eng.reject_sample(k)
        eng.kv_commit(fn.cuda(), ft.cuda())
        assert eng.status().device_status == 0
        assert oracle.kv_reserve(k, bt, o_len, o_table, o_free, o_top) == 0
        n_dev = eng.n_emitted().cpu().numpy()[:n].copy()
        oracle.kv_commit(bt, n_dev, o_len, o_table, o_free, o_top)
        books_equal()
        return drafts.cpu().numpy(), eng.out_tokens(k).cpu().numpy()[:n].copy(), n_dev

    def prefill_chunk(p, c):
        last = c == len(p) // R - 1
        return (p[c * R + 1 : c * R + R], k - 1 if last else k, p[-1] if last else p[(c + 1) * R])

    for c in range(4):
        step({b: prefill_chunk(prompts[b], c) for b in range(B)})
    chains = [ChainOracle(cfg, W, H, kind, seed, b, prompts[b], step0=4) for b in range(B)]
    boundary = 0

    def lockstep():
        nonlocal boundary
        g_drafts, g_out, g_n = step({})
        for b, ch in enumerate(chains):
            rec = ch.step_once(k)
            same = (np.array_equal(rec["drafts"], g_drafts[b]) and rec["n_emitted"] == g_n[b] and np.array_equal(rec["out_tokens"], g_out[b]))
            if not same:
                mg = rec["margins"]
                assert np.any(mg[:k] < 1e-4) or mg[k] < 1e-6 or not np.array_equal(rec["drafts"], g_drafts[b]), (b, rec, g_out[b])
                boundary += 1
                ch.tokens = ch.tokens[: len(ch.tokens) - int(rec["n_emitted"])] + [int(t) for t in g_out[b, : g_n[b]]]

    for _ in range(3):
        lockstep()
    # the batch shrinks: the kept sequences move to slots 0.., the others' blocks go back in the oracle's order
    eng.seq_compact(keep)
    o_len, o_table = oracle.kv_compact(keep, bt, o_len, o_table, o_free, o_top)
    assert eng.B == len(keep) and eng.status().device_status == 0
    books_equal()
    chains = [chains[s] for s in keep]
    for j, ch in enumerate(chains):
        ch.seq = j                                           # uniforms are drawn per slot
    for _ in range(4):
        lockstep()
    for j, ch in enumerate(chains):
        assert int(eng.seq_len()[j].item()) == len(ch.tokens) - 1
    print(f"compaction ({kind}, keep {keep}): boundary cases {boundary}")
    assert boundary <= 2
    eng.close()


def test_compact_argument_and_state_errors():
    from paper_2604_26779_b200 import engine
    cfg = inputs.model_config("c1")
    sc = engine.make_spec_config(cfg, draft_kind="none", k_max=1, max_batch=3, kv_num_blocks=9, max_blocks_per_seq=3, seed=1)
    eng = engine.SpecStep(sc)
    eng.load_target_weights(inputs.make_target_weights(cfg, seed=1))
    eng.seq_init(np.array([3, 5, 17], np.int32), np.array([1, 2, 3], np.int32), np.arange(9, dtype=np.int32))
    for bad in ([2, 1], [0, 0], [3], [0, 1, 2, 2]):
        with pytest.raises(RuntimeError):
            eng.seq_compact(bad)
    assert eng.B == 3
    eng.verify(0)
    with pytest.raises(RuntimeError):                       # a verified step is waiting for its commit
        eng.seq_compact([0])
    eng.reject_sample(0)
    eng.kv_commit()
    eng.seq_compact([0, 1, 2])                              # the identity
    assert eng.B == 3 and eng.seq_len().cpu().tolist() == [4, 6, 18]
    eng.seq_compact([2])
    assert eng.B == 1 and eng.seq_len().cpu().tolist()[:1] == [18]
    top = int(eng.tensor("FREE_TOP", 0, torch.int32, (1,)).item())
    assert top == 9 - 2                                     # 18 cached positions: two blocks stay out
    eng.verify(0); eng.reject_sample(0); eng.kv_commit()
    assert eng.seq_len().cpu().tolist()[:1] == [19] and eng.status().device_status == 0
    eng.seq_compact([])                                     # everything retired
    assert eng.B == 0 and int(eng.tensor("FREE_TOP", 0, torch.int32, (1,)).item()) == 9
    eng.close()
