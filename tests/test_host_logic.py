"""Host-side logic of the library that needs no device: configuration checks, arena sizing, tensor placement."""
import ctypes as C

import numpy as np
import pytest

from paper_2604_26779_b200 import binding as B, engine, inputs


def sizes_of(sc):
    s = B.spec_sizes()
    return B.lib().spec_query_sizes(C.byref(sc), C.byref(s)), s


def test_sizes_of_the_8b_configuration():
    cfg = inputs.model_config("c3")
    sc = engine.make_spec_config(cfg, draft_kind="eagle3", k_max=3, max_batch=256, kv_num_blocks=1000, max_blocks_per_seq=64,
                                 kv_layer_pools=16)
    code, s = sizes_of(sc)
    assert code == 0
    per_layer = 4096 * 6144 + 4096 * 4096 + 3 * 4096 * 14336
    params = 32 * per_layer + 2 * 128256 * 4096
    assert params * 2 <= s.weights_bytes <= params * 2 + (32 * 6 + 3) * 256 + 33 * 2 * 4096 * 4 + 4096
    assert abs(params - 128256 * 4096 - 7.505e9) < 0.01e9                       # 7.5 B parameters besides the embedding table
    assert s.kv_bytes == 16 * 2 * 1000 * 8 * 16 * 128 * 2                       # pools x (K,V) x blocks x heads x 16 x 128 x bf16
    assert s.draft_kv_bytes == 2 * 1000 * 8 * 16 * 128 * 2
    head = 3 * 4096 * 4096 + 6144 * 8192 + 4096 * 4096 + 3 * 4096 * 14336 + 128256 * 4096
    assert head * 2 <= s.draft_weights_bytes <= head * 2 + 64 * 1024
    assert s.workspace_bytes > 1024 * 128256 * 4 and s.state_bytes > 256 * 64 * 4


@pytest.mark.parametrize("change,code", [
    (dict(struct_size=8), -1), (dict(abi_version=99), -1), (dict(n_q_heads=30), -2), (dict(k_max=8), -2),
    (dict(kv_layer_pools=0), -2), (dict(kv_layer_pools=33), -2), (dict(temperature=0.0), -3), (dict(dtype=5), -3),
    (dict(d_ffn=1000), -2), (dict(vocab=128255), -2), (dict(vocab=1 << 20), -2), (dict(draft_kind=7), -3),
    (dict(n_experts=4, experts_top_k=8, d_expert_ffn=128), -2), (dict(n_experts=4, experts_top_k=2, d_expert_ffn=100), -3)])
def test_bad_configurations_are_refused(change, code):
    cfg = inputs.model_config("c3")
    sc = engine.make_spec_config(cfg, draft_kind="none", k_max=3, max_batch=8, kv_num_blocks=100, max_blocks_per_seq=16)
    for k, v in change.items():
        setattr(sc, k, v)
    got, _ = sizes_of(sc)
    assert got == code, (change, got)


def test_create_checks_pointers_and_tensors_do_not_overlap():
    cfg = inputs.model_config("c1")
    sc = engine.make_spec_config(cfg, draft_kind="eagle3", k_max=3, max_batch=4, kv_num_blocks=32, max_blocks_per_seq=8)
    code, s = sizes_of(sc)
    assert code == 0
    L = B.lib()
    bufs = B.spec_buffers()
    base = 1 << 30                                             # fake, aligned, never dereferenced by these calls
    offs = {}
    for i, name in enumerate(("weights", "draft_weights", "kv", "draft_kv", "workspace", "state")):
        offs[name] = base + i * (1 << 32)
        setattr(bufs, name, offs[name])
    h = C.c_void_p()
    bufs.kv = offs["kv"] + 8                                   # misaligned arena
    assert L.spec_create(C.byref(sc), C.byref(bufs), C.byref(h)) == -1
    bufs.kv = offs["kv"]
    assert L.spec_create(C.byref(sc), C.byref(bufs), C.byref(h)) == 0
    spans = []
    for name, tid in B.T.items():
        for layer in range(cfg["n_layers"] if 3 <= tid <= 8 else 1):
            p, n = C.c_void_p(), C.c_size_t()
            rc = L.spec_tensor(h, tid, layer, C.byref(p), C.byref(n))
            if rc != 0:
                continue                                         # tensors this configuration does not have
            assert p.value % 256 == 0 and n.value > 0
            arena = max((a for a in offs.values() if a <= p.value))
            aname = [k for k, v in offs.items() if v == arena][0]
            assert p.value + n.value <= arena + getattr(s, aname + "_bytes"), name
            if name not in ("HIDDEN",):
                spans.append((p.value, p.value + n.value, name))
    spans.sort()
    for (a0, a1, an), (b0, b1, bn) in zip(spans, spans[1:]):
        assert a1 <= b0, (an, bn)
    # calls that are out of order are refused with a reason
    assert L.spec_draft(h, 3, None) == -4 and b"no committed step" in L.spec_last_error(h)
    assert L.spec_kv_commit(h, None, None, None) == -4
    assert L.spec_reject_sample(h, 3, None, None) == -4
    assert L.spec_verify(h, 9, None, None) == -2 and b"k outside" in L.spec_last_error(h)
    assert L.spec_tensor(h, 9999, 0, C.byref(C.c_void_p()), C.byref(C.c_size_t())) == -1
    assert L.spec_destroy(h) == 0


def test_k_policy_arithmetic():
    """Expected tokens per step under independent acceptance is the geometric sum; the chosen k is the brute-force best."""
    from paper_2604_26779_b200 import rollout
    for a in (0.0, 0.3, 0.8, 1.0):
        for k in (0, 1, 3, 7):
            assert abs(rollout.expected_tokens_per_step(a, k) - sum(a ** i for i in range(k + 1))) < 1e-12
    # Monte Carlo check of the same quantity: the accepted prefix of k Bernoulli(a) trials plus one token
    rng = np.random.default_rng(0)
    acc = rng.random((200000, 5)) < 0.6
    n = np.where(acc.all(1), 5, np.argmin(acc, 1))
    assert abs((n + 1).mean() - rollout.expected_tokens_per_step(0.6, 5)) < 0.02
    assert rollout.acceptance_rate(30, 50) == 0.6 and rollout.acceptance_rate(0, 0) == 0.0
    # cost linear in rows: a thin batch prefers long drafts, a full one short drafts
    cost = lambda B, k: 10.0 + 0.05 * B * (k + 1)
    assert rollout.choose_k(0.7, 4, cost, range(1, 8)) == 7
    assert rollout.choose_k(0.7, 2048, cost, range(1, 8)) <= 2
    for a in (0.2, 0.5, 0.9):
        for B in (1, 64, 1024):
            ks = list(range(1, 8))
            rates = [rollout.expected_tokens_per_step(a, k) / cost(B, k) for k in ks]
            assert rollout.choose_k(a, B, cost, ks) == ks[int(np.argmax(rates))]


def test_sizes_and_refusals_with_8bit_projections():
    """SPEC_W_E4M3: one byte per projection weight + one fp32 scale per weight row (embedding, norms and the draft head stay
    16-bit); refused for the combinations the 8-bit path does not cover."""
    cfg = inputs.model_config("c3")
    kw = dict(draft_kind="eagle3", k_max=3, max_batch=256, kv_num_blocks=1000, max_blocks_per_seq=64, kv_layer_pools=16)
    code16, s16 = sizes_of(engine.make_spec_config(cfg, **kw))
    code8, s8 = sizes_of(engine.make_spec_config(cfg, w_fp8=True, **kw))
    assert code16 == 0 and code8 == 0
    per_layer = 4096 * 6144 + 4096 * 4096 + 3 * 4096 * 14336
    rows = 32 * (6144 + 4096 + 2 * 14336 + 4096) + 128256                        # one scale per weight row
    want = 32 * per_layer + 128256 * 4096 + rows * 4 + 128256 * 4096 * 2       # codes + scales + the 16-bit embedding
    assert want <= s8.weights_bytes <= want + (32 * 10 + 4) * 256 + 33 * 2 * 4096 * 4 + 4096
    assert s8.draft_weights_bytes == s16.draft_weights_bytes and s8.kv_bytes == s16.kv_bytes
    assert s8.workspace_bytes >= s16.workspace_bytes + 5 * 1024 * 14336          # five quantised-activation slots
    sc = engine.make_spec_config(cfg, w_fp8=True, **dict(kw, draft_kind="mtp", draft_d_ffn=14336))
    assert sizes_of(sc)[0] == 0                                                  # the MTP head scores with the 8-bit LM head
    moe = inputs.model_config("c5")
    c16, m16 = sizes_of(engine.make_spec_config(moe, draft_kind="none", k_max=3, max_batch=8, kv_num_blocks=100, max_blocks_per_seq=16))
    c8, m8 = sizes_of(engine.make_spec_config(moe, draft_kind="none", k_max=3, max_batch=8, kv_num_blocks=100, max_blocks_per_seq=16, w_fp8=True))
    assert c16 == 0 and c8 == 0
    experts = moe["n_experts"] * 3 * moe["d_expert_ffn"] * moe["d_model"]           # gate, up, down: one byte instead of two
    assert m16.weights_bytes - m8.weights_bytes > experts * 0.99
    for change in (dict(dtype=B.SPEC_DTYPE_F32), dict(weight_dtype=7)):
        sc = engine.make_spec_config(cfg, w_fp8=True, **kw)
        for k, v in change.items():
            setattr(sc, k, v)
        got, _ = sizes_of(sc)
        assert got == -3, (change, got)


def test_8bit_operator_argument_checks_need_no_device():
    """spec_quantize_rows / spec_gemm_e4m3 refuse bad arguments on the host, before anything is launched."""
    L = B.lib()
    fake = 4096                                                 # non-null, 16-byte aligned, never dereferenced on the host
    assert L.spec_quantize_rows(0, 64, None, None, None, None) == 0
    assert L.spec_quantize_rows(4, 0, fake, fake, fake, None) == -1
    assert L.spec_quantize_rows(4, 64, None, fake, fake, None) == -1
    assert L.spec_quantize_rows(4, 12, fake, fake, fake, None) == -2
    assert L.spec_gemm_e4m3(0, 64, 64, None, None, None, None, None, 1, 0, None) == 0
    assert L.spec_gemm_e4m3(4, 64, 64, fake, None, fake, fake, fake, 1, 0, None) == -1
    assert L.spec_gemm_e4m3(4, 60, 64, fake, fake, fake, fake, fake, 1, 0, None) == -2
    assert L.spec_gemm_e4m3(4, 64, 24, fake, fake, fake, fake, fake, 1, 0, None) == -2       # K % 16
    assert L.spec_gemm_e4m3(4, 64, 64, fake + 8, fake, fake, fake, fake, 1, 0, None) == -2   # operand alignment
