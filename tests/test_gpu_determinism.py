"""Run-to-run determinism of the whole step.  Work is handed out through atomic counters (attention units, persistent
GEMM tiles) and split-K / split-KV partials are summed afterwards, so the ORDER of every sum must not depend on which CTA
got which unit: two runs from the same state have to agree bit for bit - logits, emitted tokens, log-probabilities and
the cache itself."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def run_once(name, cfg_over, draft, lens, k, steps, n_layers, vocab):
    from paper_2604_26779_b200 import workloads
    eng, info = workloads.build_dense_workload(name, lens=np.array(lens, np.int32), k=k, draft=draft, steps_budget=steps + 2,
                                               n_layers=n_layers, vocab=vocab, cfg_over=cfg_over)
    if draft != "none":
        workloads.bootstrap(eng)
    outs = []
    for _ in range(steps):
        if draft != "none":
            workloads.spec_step(eng, k)
        else:
            workloads.bootstrap(eng)
        outs.append((eng.logits(k if draft != "none" else 0).clone(), eng.out_tokens(k if draft != "none" else 0).clone(), eng.n_emitted().clone()))
    assert eng.status().device_status == 0
    pools = [eng.kv_pool("KV_K", 0).clone(), eng.kv_pool("KV_V", 0).clone()]
    seq = eng.seq_len().clone()
    eng.close()
    return outs, pools, seq


@pytest.mark.parametrize("name,cfg_over,draft,n_layers,vocab", [
    ("c3", None, "eagle3", 3, 4096),
    ("c3", dict(kv_fp8=(0.0625, 0.0625)), "eagle3", 3, 4096),
    ("c4", None, "mtp", 2, 4096),
    ("c5", dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=64, n_experts=16, experts_top_k=4, d_expert_ffn=128), "none", None, 1024),
])
def test_two_runs_agree_bit_for_bit(name, cfg_over, draft, n_layers, vocab):
    lens = [5000, 37, 4096, 900, 12000, 1, 260, 4097, 8191, 64, 3000, 15]      # several chunks per sequence, ragged tails
    a = run_once(name, cfg_over, draft, lens, 3, 3, n_layers, vocab)
    b = run_once(name, cfg_over, draft, lens, 3, 3, n_layers, vocab)
    for (la, ta, na), (lb, tb, nb) in zip(a[0], b[0]):
        assert torch.equal(na, nb) and torch.equal(ta, tb)
        assert torch.equal(la.view(torch.int32), lb.view(torch.int32))
    for pa, pb in zip(a[1], b[1]):
        assert torch.equal(pa.view(torch.uint8), pb.view(torch.uint8))
    assert torch.equal(a[2], b[2])
    assert int(a[2].sum()) > int(sum(lens))                                     # tokens were committed


def test_two_contexts_on_two_host_threads_match_the_single_threaded_run():
    """Different contexts may be driven from different host threads (each on its own stream): the calls hold no shared
    mutable state beyond per-device one-time set-up, so every context produces the bits it produces alone."""
    import threading
    from paper_2604_26779_b200 import workloads
    lens = [300, 37, 4096, 900, 1, 260, 64, 2000]
    kw = dict(k=3, draft="eagle3", steps_budget=6, n_layers=2, vocab=2048,      # as run_once builds it: the same pools, the same synthetic cache
              cfg_over=dict(d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=128, d_ffn=1024))
    alone = run_once("c3", kw["cfg_over"], "eagle3", lens, 3, 4, 2, 2048)
    engines = [workloads.build_dense_workload("c3", lens=np.array(lens, np.int32), **kw)[0] for _ in range(2)]
    torch.cuda.synchronize()                                     # the weights were filled on the default stream
    results, errors = [None, None], []

    def work(i):
        try:
            torch.cuda.set_device(0)
            with torch.cuda.stream(torch.cuda.Stream()):
                eng = engines[i]
                workloads.bootstrap(eng)
                outs = []
                for _ in range(4):
                    workloads.spec_step(eng, 3)
                    outs.append((eng.logits(3).clone(), eng.out_tokens(3).clone(), eng.n_emitted().clone()))
                torch.cuda.current_stream().synchronize()
                results[i] = outs
        except Exception as e:                                   # surfaced in the main thread below
            errors.append(e)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for outs in results:
        for (la, ta, na), (lb, tb, nb) in zip(alone[0], outs):
            assert torch.equal(na, nb) and torch.equal(ta, tb)
            assert torch.equal(la.view(torch.int32), lb.view(torch.int32))
    for eng in engines:
        assert eng.status().device_status == 0
        eng.close()
