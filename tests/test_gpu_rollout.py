"""GPU parity of a multi-step rollout with continuous batching: seven sequences through three slots, prompts prefilled
through forced verify steps while other slots speculate, the draft length changing from step to step, finished slots
refilled and finally retired.  Every sequence's response must equal what the cache-free CPU oracle chain produces for
the same (seed, slot, first step, k sequence); the block pool must be whole again at the end."""
import numpy as np
import pytest

from oracle.chain import ChainOracle
from paper_2604_26779_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kind,compact,graphs", [("eagle3", 0.0, False), ("ngram", 0.0, False), ("eagle3", 0.7, False), ("ngram", 0.7, False),
                                                 ("eagle3", 0.7, True), ("ngram", 0.0, True)])
def test_rollout_with_refill_matches_oracle_chains(kind, compact, graphs):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26779_b200 import engine, rollout
    cfg = dict(inputs.model_config("c1"), ngram_n=2)
    seed, k_max, slots = 977, 4, 3
    W = inputs.make_target_weights(cfg, seed=inputs.sub_seed(3, 0))
    H = inputs.make_eagle3_weights(cfg, seed=inputs.sub_seed(3, 1)) if kind == "eagle3" else None
    p_lens = [5, 9, 2, 13, 4, 7, 6]
    wants = [9, 30, 5, 17, 12, 6, 21]
    rng = np.random.default_rng(11)
    prompts = [rng.integers(0, 64 if kind == "ngram" else cfg["vocab"], n).astype(np.int32) for n in p_lens]
    sc = engine.make_spec_config(cfg, draft_kind=kind, k_max=k_max, max_batch=slots, kv_num_blocks=16, max_blocks_per_seq=5,
                                 seed=seed)
    eng = engine.SpecStep(sc)
    eng.load_target_weights(W)
    if H is not None:
        eng.load_draft_weights(H)
    order = inputs.make_block_order(sc.kv_num_blocks, inputs.sub_seed(3, 3))
    ro = rollout.Rollout(eng, prompts, wants, order, k_policy=lambda step, n_active, alpha: 1 + step % k_max,
                         compact_fraction=compact, use_graphs=graphs)
    done = ro.run(max_steps=400)
    assert sorted(done) == list(range(7))
    assert max(ro.active_trace) == slots and min(ro.active_trace) >= 1
    boundary = 0
    for i in range(7):
        rec = done[i]
        assert len(rec.tokens) == wants[i]
        ch = ChainOracle(cfg, W, H, kind, seed, rec.slots[0], prompts[i], step0=rec.first_decode_step)
        # the sequence's decode steps are consecutive device steps, so the chain's step counter follows by itself; the slot
        # (and with it the Philox stream) changes when the batch is compacted
        got, ref = rec.tokens, []
        for k, slot in zip(rec.ks, rec.slots):
            ch.seq = slot
            r = ch.step_once(k)
            new = [int(t) for t in r["out_tokens"][: r["n_emitted"]]]
            n_have = len(ref)
            if got[n_have : n_have + len(new)] != new[: max(0, len(got) - n_have)]:
                mg = r["margins"]
                assert np.any(mg[:k] < 1e-4) or mg[k] < 1e-6, (i, k, new, got[n_have:], mg)
                boundary += 1
                break
            ref += new
    print(f"rollout {kind}: {ro.step} steps, k trace {ro.k_trace[:8]}..., boundary {boundary}")
    assert boundary <= 1
    if graphs:
        assert ro.graph_steps >= 1
    if compact:
        assert len(ro.compactions) >= 1 and ro.compactions[-1][2] < slots
    # everything is retired and every block is back
    assert eng.seq_len().cpu().tolist() == [-1] * eng.B
    assert int(eng.tensor("FREE_TOP", 0, torch.int32, (1,)).item()) == sc.kv_num_blocks
    free = eng.tensor("FREE_STACK", 0, torch.int32, (sc.kv_num_blocks,)).cpu().numpy()
    assert sorted(free.tolist()) == list(range(sc.kv_num_blocks))
    assert np.all(eng.block_table().cpu().numpy() == -1)
    eng.close()
