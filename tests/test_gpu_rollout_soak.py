"""A longer rollout at the production shape (8B-shaped target, EAGLE-3 head; bf16, and with 8-bit projections + 8-bit cache): 96 prompts through 48 slots with
long-tailed response lengths, prompts prefilled through forced verify steps, finished slots refilled, the batch compacted
as it thins.  No oracle here (the small lock-step tests carry parity): this checks the properties that must hold at any
size - every response has the requested length, every token is a valid id, the device never reports an error, the block
pool is whole again at the end - while the step runs through every size regime (tile GEMMs, thin-batch GEMMs, coarse and
fine attention chunks)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("variant", ["bf16", "8-bit projections and cache"])
def test_rollout_soak_production_shape(variant):
    from paper_2604_26779_b200 import rollout, workloads
    over = dict(w_fp8=True, kv_fp8=(0.0625, 0.0625)) if variant != "bf16" else None
    slots, n_prompts, k = 48, 96, 3
    rng = np.random.default_rng(2604)
    p_lens = rng.integers(8, 64, n_prompts)
    wants = np.clip(np.exp(rng.normal(np.log(48.0), 0.9, n_prompts)).astype(np.int64), 4, 400)     # long-tailed
    # room for prompt + response + k + 1 per sequence
    eng, info = workloads.build_dense_workload("c3", lens=np.full(slots, 640, np.int32), k=k, n_layers=8, steps_budget=4, cfg_over=over)
    vocab = info["cfg"]["vocab"]
    prompts = [rng.integers(0, vocab, n).astype(np.int32) for n in p_lens]
    ro = rollout.Rollout(eng, prompts, [int(w) for w in wants], info["block_order"],
                         k_policy=lambda step, n_active, alpha: 3 if n_active > 8 else 2, compact_fraction=0.5)
    done = ro.run(max_steps=5000)
    assert sorted(done) == list(range(n_prompts))
    for i in range(n_prompts):
        t = np.asarray(done[i].tokens)
        assert len(t) == wants[i] and t.min() >= 0 and t.max() < vocab
    assert eng.status().device_status == 0
    assert len(ro.compactions) >= 2 and ro.compactions[-1][2] <= slots // 4
    assert min(ro.active_trace) >= 1 and max(ro.active_trace) == slots
    top = int(eng.tensor("FREE_TOP", 0, torch.int32, (1,)).item())
    assert top == info["num_blocks"]
    free = eng.tensor("FREE_STACK", 0, torch.int32, (info["num_blocks"],)).cpu().numpy()
    assert np.array_equal(np.sort(free), np.arange(info["num_blocks"]))
    emitted = sum(len(done[i].tokens) for i in range(n_prompts))
    print(f"soak ({variant}): {ro.step} steps, {emitted} response tokens, compactions {ro.compactions}, "
          f"acceptance estimate {rollout.acceptance_rate(*ro._acc):.3f}")
    eng.close()
