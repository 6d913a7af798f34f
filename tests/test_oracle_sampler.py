"""Pins for the CPU oracle's uniforms, softmax, inverse CDF, rejection sampler and KV bookkeeping.

None of these compares the oracle with itself: each pin is a published vector, a library routine, a closed
form, an invariant, or a brute-force probe of the code path.
"""
import os

import numpy as np
import pytest
import scipy.special
import scipy.stats

import oracle
from paper_2604_26779_b200 import inputs


# ---- uniforms ------------------------------------------------------------------------------------------------

def test_philox_known_answers(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) if not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_uniform_range_and_mapping():
    u = oracle.uniforms(seed=0x1234567890ABCDEF, step=3, stream=0, n_seq=2000, n_slots=8)
    assert u.dtype == np.float32 and u.min() >= 0.0 and u.max() < 1.0
    # 24-bit grid: u * 2^24 is an integer
    assert np.all(u * 16777216.0 == np.floor(u * 16777216.0))
    # first word of the generator, key = (lo, hi) of the seed, counter = (step, seq, slot, stream)
    w = oracle.philox4x32_10([3, 17, 5, 0], [0x90ABCDEF, 0x12345678])
    assert u[17, 5] == np.float32(int(w[0]) >> 8) / np.float32(16777216.0)
    # uniformity (Kolmogorov-Smirnov) and independence across streams
    assert scipy.stats.kstest(u.ravel().astype(np.float64), "uniform").pvalue > 1e-3
    u1 = oracle.uniforms(seed=0x1234567890ABCDEF, step=3, stream=1, n_seq=2000, n_slots=8)
    assert abs(np.corrcoef(u.ravel(), u1.ravel())[0, 1]) < 0.05


# ---- softmax -------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("T", [1.0, 0.7, 2.0])
def test_softmax_matches_scipy(T):
    rng = np.random.default_rng(5)
    lg = (rng.standard_normal((7, 1027)) * 3).astype(np.float32)
    got = oracle.softmax(lg, T)
    ref = scipy.special.softmax(lg.astype(np.float64) / T, axis=-1)
    assert np.max(np.abs(got - ref)) < 1e-7
    assert np.allclose(got.sum(-1), 1.0, atol=1e-5)
    m, z = oracle.softmax_stats(lg[0], T)
    assert m == lg[0].max() and np.isclose(np.log(z) + m / T, scipy.special.logsumexp(lg[0].astype(np.float64) / T))


def test_logprob_matches_scipy_log_softmax():
    rng = np.random.default_rng(9)
    lg = (rng.standard_normal(5000) * 4).astype(np.float32)
    for T in (1.0, 0.6):
        ref = scipy.special.log_softmax(lg.astype(np.float64) / T)
        for t in (0, 17, 4999, int(np.argmax(lg))):
            assert abs(oracle.logprob(lg, t, T) - ref[t]) < 1e-12


# ---- inverse CDF ---------------------------------------------------------------------------------------------

def test_invcdf_edges():
    w = np.array([0.0, 0.25, 0.0, 0.5, 0.25, 0.0], np.float32)
    assert oracle.invcdf(w, 0.0)[0] == 1            # u = 0 takes the first positive bin
    assert oracle.invcdf(w, 0.2499)[0] == 1
    assert oracle.invcdf(w, 0.25)[0] == 3           # strict comparison: the edge belongs to the next positive bin
    assert oracle.invcdf(w, 0.7499)[0] == 3
    assert oracle.invcdf(w, 0.75)[0] == 4
    assert oracle.invcdf(w, 0.99999994)[0] == 4     # never a zero-weight bin, never past the last positive one
    assert oracle.invcdf(np.zeros(4, np.float32), 0.5)[0] == -1
    # scale invariance: weights need not be normalised
    assert oracle.invcdf(w * 7.0, 0.6)[0] == oracle.invcdf(w, 0.6)[0]
    # margin = distance to the nearer bin edge in units of the total
    assert np.isclose(oracle.invcdf(w, 0.30)[1], 0.05)


def test_invcdf_frequencies():
    rng = np.random.default_rng(11)
    w = rng.random(8).astype(np.float32)
    us = (np.arange(1 << 16) + 0.5) / (1 << 16)
    cnt = np.bincount([oracle.invcdf(w, u)[0] for u in us], minlength=8)
    assert np.max(np.abs(cnt / len(us) - w / w.sum())) < 2e-5


# ---- rejection sampler: deterministic probe of the code path (vocab 8, k <= 3) --------------------------------

def _tables(rng, V, n):
    t = 0.6 * rng.dirichlet(np.ones(V), size=n) + 0.4 / V
    return (t / t.sum(-1, keepdims=True)).astype(np.float32)


def _threshold_by_bisection(p, q, draft, pos):
    """Largest u (on the 2^-24 grid) for which position `pos` is still accepted, found by probing the code."""
    k = q.shape[0]
    lo, hi = -1, 1 << 24                   # grid indices: accept(lo) true, accept(hi) false
    while hi - lo > 1:
        mid = (lo + hi) // 2
        u = np.zeros(k + 1, np.float32)    # u = 0 accepts every earlier position (all probabilities positive)
        u[pos] = mid / 16777216.0
        _, n, _, _ = oracle.reject_sample_seq(p, q, draft, u)
        if n > pos + 1:
            lo = mid
        else:
            hi = mid
    return hi / 16777216.0                 # P(accept) = measure of {u : accepted} = hi * 2^-24


@pytest.mark.parametrize("k", [1, 2, 3])
def test_first_token_distribution_is_target_by_enumeration(k):
    """Enumerates every first draft token, measures the code's accept threshold by bisection and its resample
    frequencies on a fine grid of the final uniform, and checks  q(x) a(x) + sum_d q(d)(1-a(d)) res_d(x) = p(x)."""
    V = 8
    rng = np.random.default_rng(100 + k)
    p = _tables(rng, V, k + 1)
    q = _tables(rng, V, k)
    grid = (np.arange(4096) + 0.5) / 4096
    total = np.zeros(V)
    for d in range(V):
        draft = np.array([d] + [0] * (k - 1), np.int32)
        a = _threshold_by_bisection(p, q, draft, 0)
        assert abs(a - min(1.0, float(p[0, d]) / float(q[0, d]))) < 1e-6
        total[d] += q[0, d] * a
        res = np.zeros(V)
        for u_last in grid:
            u = np.zeros(k + 1, np.float32)
            u[0] = 0.99999994              # reject position 1 whenever it can be rejected
            u[k] = u_last
            toks, n, _, _ = oracle.reject_sample_seq(p, q, draft, u)
            if n == 1:
                res[toks[0]] += 1
        if a < 1.0:
            assert res.sum() == len(grid)
            res /= res.sum()
            assert np.all(res[p[0] <= q[0]] == 0)          # a resampled token always has p > q
            total += q[0, d] * (1.0 - a) * res
    assert np.max(np.abs(total - p[0])) < 5e-4


def test_full_step_enumeration_k2_vocab4():
    """Exhaustive: every draft pair, every combination of accept/reject regions, resample grid -> the joint of
    the emitted prefix of length <= 2 marginalises to the target product on its first token and, where two tokens
    are produced by acceptance, to p_1(x1) p_2(x2|x1)."""
    V, k = 4, 2
    rng = np.random.default_rng(7)
    P1 = _tables(rng, V, 1)[0]
    P2 = _tables(rng, V, V)        # p_2(. | d_1)
    P3 = _tables(rng, V, V)        # p_3(. | d_2) (bonus row)
    Q1 = _tables(rng, V, 1)[0]
    Q2 = _tables(rng, V, V)
    G = 48
    grid = ((np.arange(G) + 0.5) / G).astype(np.float32)
    joint = np.zeros((V, V))       # distribution of the first two emitted tokens when at least two are emitted this step
    first = np.zeros(V)
    for d1 in range(V):
        for d2 in range(V):
            p = np.stack([P1, P2[d1], P3[d2]])
            q = np.stack([Q1, Q2[d1]])
            wd = float(Q1[d1]) * float(Q2[d1, d2])
            for u0 in grid:
                for u1 in grid:
                    for u2 in grid[::4]:
                        toks, n, _, _ = oracle.reject_sample_seq(p, q, [d1, d2], [u0, u1, u2])
                        w = wd / (G * G * (G // 4))
                        first[toks[0]] += w
                        if n >= 2:
                            joint[toks[0], toks[1]] += w
    assert np.max(np.abs(first - P1)) < 1.5e-2
    # whenever position 1 is accepted a second token is emitted in the same step, and it must follow p_2(.|x1)
    acc1 = joint.sum(1)
    cond = joint / acc1[:, None]
    assert np.max(np.abs(cond - P2)) < 3e-2
    assert np.allclose(acc1, np.minimum(P1, Q1), atol=1.5e-2)


# ---- rejection sampler: chi-square over 1e6 seeded trials (vocab 8, k = 3) -------------------------------------

def _run_chain_trials(P0, P, Q0, Q, k, n_trials, seed, swap=False):
    """Markov toy models: target p(x | prev) = P[prev], draft q(x | prev) = Q[prev]; first conditionals P0/Q0.
    Runs speculation steps until every trial has emitted k+1 tokens; returns the first k+1 tokens per trial."""
    V = P.shape[0]
    need = k + 1
    emitted = np.full((n_trials, need + k + 1), -1, np.int64)
    count = np.zeros(n_trials, np.int64)
    prev = np.full(n_trials, -1, np.int64)          # -1: start state
    step = 0
    Pfull = np.concatenate([P, P0[None]], 0)        # index -1 -> start row
    Qfull = np.concatenate([Q, Q0[None]], 0)
    while count.min() < need:
        p = np.zeros((n_trials, k + 1, V), np.float32)
        q = np.zeros((n_trials, k, V), np.float32)
        drafts = np.zeros((n_trials, k), np.int32)
        cur = prev.copy()
        ud = oracle.uniforms(seed, step, 1, n_trials, k)
        for i in range(k):
            q[:, i, :] = Qfull[cur]
            p[:, i, :] = Pfull[cur]
            d, _ = oracle.sample_rows(q[:, i, :], ud[:, i])
            drafts[:, i] = d
            cur = d.astype(np.int64)
        p[:, k, :] = Pfull[cur]
        if swap:
            toks, n, _, _ = oracle.reject_sample(np.concatenate([q, p[:, k:, :]], 1), p[:, :k, :], drafts, seed, step)
        else:
            toks, n, _, _ = oracle.reject_sample(p, q, drafts, seed, step)
        assert n.min() >= 1 and n.max() <= k + 1            # 1 <= tokens per step <= k+1
        for j in range(k + 1):
            live = (j < n) & (count + j < emitted.shape[1])
            emitted[np.nonzero(live)[0], (count + j)[live]] = toks[live, j]
        prev = toks[np.arange(n_trials), n - 1].astype(np.int64)
        count += n
        step += 1
    return emitted[:, :need]


def _chain_expected(P0, P, need):
    V = P.shape[0]
    e = P0.astype(np.float64).copy()
    for _ in range(need - 1):
        e = e[..., None] * P.astype(np.float64).reshape((1,) * (e.ndim - 1) + (V, V))
    return e


def test_emitted_distribution_chi_square_1e6():
    V, k, n = 8, 3, 1_000_000
    rng = np.random.default_rng(2604)
    P0, Q0 = _tables(rng, V, 1)[0], _tables(rng, V, 1)[0]
    P, Q = _tables(rng, V, V), _tables(rng, V, V)
    exp = _chain_expected(P0, P, k + 1).ravel()
    assert exp.min() * n > 5                                # chi-square valid without pooling
    toks = _run_chain_trials(P0, P, Q0, Q, k, n, seed=inputs.BASE_SEED)
    idx = np.ravel_multi_index(toks.T, (V,) * (k + 1))
    obs = np.bincount(idx, minlength=V ** (k + 1))
    chi = scipy.stats.chisquare(obs, exp / exp.sum() * n)
    assert chi.pvalue > 1e-4, chi
    # control: the same test must have the power to reject a wrong sampler (target and draft roles swapped)
    bad = _run_chain_trials(P0, P, Q0, Q, k, 100_000, seed=inputs.BASE_SEED, swap=True)
    obs_bad = np.bincount(np.ravel_multi_index(bad.T, (V,) * (k + 1)), minlength=V ** (k + 1))
    assert scipy.stats.chisquare(obs_bad, exp / exp.sum() * 100_000).pvalue < 1e-12


# ---- special cases and closed forms --------------------------------------------------------------------------

def test_draft_equals_target_accepts_everything():
    V, k, B = 1000, 5, 64
    rng = np.random.default_rng(3)
    p = oracle.softmax(rng.standard_normal((B, k + 1, V)).astype(np.float32))
    q = p[:, :k, :].copy()
    d = rng.integers(0, V, (B, k)).astype(np.int32)
    toks, n, fl, _ = oracle.reject_sample(p, q, d, seed=9, step=0)
    assert np.all(n == k + 1) and np.all(toks[:, :k] == d) and np.all(fl == 0)
    # the bonus token is the inverse CDF of p_{k+1} at the slot-k uniform
    u = oracle.uniforms(9, 0, 0, B, k + 1)
    for b in range(0, B, 7):
        assert toks[b, k] == oracle.invcdf(p[b, k], u[b, k])[0]


@pytest.mark.parametrize("a", [0.9601, 0.8026, 0.6171])
def test_iid_acceptance_mean_length(a):
    """Independent positions with acceptance probability a each: E[tokens per step] = (1 - a^(k+1)) / (1 - a)."""
    k, B = 3, 200_000
    q_row = np.array([0.5, 0.5, 0.0, 0.0], np.float32)
    p_row = np.array([0.5 * a, 0.5 * a, (1 - a) / 2, (1 - a) / 2], np.float32)
    p = np.broadcast_to(p_row, (B, k + 1, 4)).copy()
    q = np.broadcast_to(q_row, (B, k, 4)).copy()
    ud = oracle.uniforms(77, 0, 1, B, k)
    d = np.stack([oracle.sample_rows(q[:, i], ud[:, i])[0] for i in range(k)], 1)
    assert set(np.unique(d)) <= {0, 1}
    toks, n, _, _ = oracle.reject_sample(p, q, d, seed=77, step=0)
    expect = (1 - a ** (k + 1)) / (1 - a)
    sd = np.sqrt(np.var(n) / B)
    assert abs(n.mean() - expect) < 5 * sd + 1e-3
    # a rejected position resamples only where p > q
    rej = n <= k
    assert np.all(toks[rej, n[rej] - 1] >= 2)


def test_one_hot_draft_special_case():
    """q = one-hot(d): accept iff u < p(d); the residual is p with p(d) removed."""
    V = 8
    rng = np.random.default_rng(21)
    p = _tables(rng, V, 2)
    d = 3
    q = np.zeros((1, V), np.float32)
    q[0, d] = 1.0
    pd = float(p[0, d])
    below, above = np.float32(np.floor(pd * 2 ** 24 - 1) / 2 ** 24), np.float32(np.ceil(pd * 2 ** 24 + 1) / 2 ** 24)
    assert oracle.reject_sample_seq(p, q, [d], [below, 0.3])[1] == 2
    toks, n, _, _ = oracle.reject_sample_seq(p, q, [d], [above, 0.3])
    assert n == 1
    w = p[0].copy()
    w[d] = 0
    assert toks[0] == oracle.invcdf(w, 0.3)[0] and toks[0] != d


def test_zero_draft_probability_and_bad_rows():
    V = 4
    p = np.array([[0.5, 0.5, 0, 0], [0.25, 0.25, 0.25, 0.25]], np.float32)
    q = np.array([[0.0, 1.0, 0, 0]], np.float32)
    assert oracle.reject_sample_seq(p, q, [0], [0.999, 0.1])[1] == 2     # q(d)=0, p(d)>0: accepted
    assert oracle.reject_sample_seq(p, q, [2], [0.0, 0.1])[1] == 1       # q(d)=0, p(d)=0: rejected
    # residual without mass (p == q, yet rejected is impossible; force it with p<q everywhere but the sums garbage)
    p2 = np.array([[0.1, 0.1, 0.1, 0.1], [0.25] * 4], np.float32)
    q2 = np.array([[0.4, 0.4, 0.4, 0.4]], np.float32)
    toks, n, fl, _ = oracle.reject_sample_seq(p2, q2, [1], [0.9, 0.6])
    assert n == 1 and fl & 1 and toks[0] == 2                            # falls back to p_{n+1}, flagged


def test_residual_invariants():
    rng = np.random.default_rng(8)
    p = oracle.softmax(rng.standard_normal((50, 300)).astype(np.float32) * 2)
    q = oracle.softmax(rng.standard_normal((50, 300)).astype(np.float32) * 2)
    res = np.maximum(0.0, p.astype(np.float64) - q.astype(np.float64)).sum(-1)
    assert np.allclose(res, 1.0 - np.minimum(p, q).astype(np.float64).sum(-1), atol=1e-6)


def test_c2_input_recipe_acceptance_closed_form():
    """Draft logits = target + N(0, tau^2): the acceptance probability sum_v min(p, q) tends to 2*Phi(-tau/2)."""
    V = 151936
    for tau, tol in [(0.1, 0.003), (0.5, 0.003), (1.0, 0.003)]:
        t, d = inputs.make_sampler_logits(B=4, k=1, V=V, sigma=1.0, tau=tau, seed=inputs.sub_seed(2, int(tau * 10)))
        p, q = oracle.softmax(t[:, 0]), oracle.softmax(d[:, 0])
        a = np.minimum(p, q).astype(np.float64).sum(-1)
        ref = 2 * scipy.stats.norm.cdf(-tau / 2)
        assert abs(a.mean() - ref) < tol and np.all(np.abs(a - ref) < 3 * tol), (tau, a)


def test_sampler_acceptance_rate_on_c2_recipe():
    B, k, V, tau = 96, 3, 4096, 0.5
    t, d = inputs.make_sampler_logits(B, k, V, sigma=1.0, tau=tau, seed=5)
    p, q = oracle.softmax(t), oracle.softmax(d)
    rates = []
    for step in range(20):
        ud = oracle.uniforms(5, step, 1, B, k)
        drafts = np.stack([oracle.sample_rows(q[:, i], ud[:, i])[0] for i in range(k)], 1)
        _, n, _, _ = oracle.reject_sample(p, q, drafts, seed=5, step=step)
        rates.append(np.mean(n >= 2))
    a = 2 * scipy.stats.norm.cdf(-tau / 2)
    assert abs(np.mean(rates) - a) < 0.03


# ---- KV bookkeeping ------------------------------------------------------------------------------------------

def test_kv_reserve_commit_conserves_blocks():
    B, bt, maxb, nblk, k = 7, 16, 12, 84, 3
    rng = np.random.default_rng(4)
    seq_len = rng.integers(1, 100, B).astype(np.int32)
    table = np.full((B, maxb), -1, np.int32)
    free = inputs.make_block_order(nblk, 1)
    top = np.array([nblk], np.int32)
    start_free = set(free.tolist())
    for it in range(30):
        assert oracle.kv_reserve(k, bt, seq_len, table, free, top) == 0
        owned = table[table >= 0]
        assert len(set(owned.tolist())) == owned.size                       # no block owned twice
        assert set(owned.tolist()) | set(free[: top[0]].tolist()) == start_free
        assert owned.size + top[0] == nblk                                   # owned + free = total
        for b in range(B):
            need = -(-(seq_len[b] + k + 1) // bt)
            assert np.all(table[b, :need] >= 0) and np.all(table[b, need:] == -1)
        n_emit = rng.integers(1, k + 2, B).astype(np.int32)
        before = seq_len.copy()
        oracle.kv_commit(bt, n_emit, seq_len, table, free, top)
        assert np.all(seq_len == before + n_emit)
        for b in range(B):
            keep = -(-seq_len[b] // bt)
            assert np.all(table[b, :keep] >= 0) and np.all(table[b, keep:] == -1)
        if seq_len.max() + k + 1 > maxb * bt:
            break
    # exhaustion is reported and leaves the state untouched
    top2 = np.array([0], np.int32)
    t2 = np.full((B, maxb), -1, np.int32)
    assert oracle.kv_reserve(k, bt, seq_len, t2, free, top2) == -1 and np.all(t2 == -1)


def test_kv_replace_returns_and_reissues_blocks():
    """Worked by hand: stack [5,4,3,2,1,0] (top last); A holds [0,1], B holds [2]; replacing A by a 40-token sequence
    pushes 0 then 1 (stack [5,4,3,0,1]) and pops 1, 0, 3 in that order."""
    bt, maxb = 16, 4
    seq_len = np.array([20, 7], np.int32)
    table = np.array([[0, 1, -1, -1], [2, -1, -1, -1]], np.int32)
    free = np.array([5, 4, 3, 9, 9, 9], np.int32)
    top = np.array([3], np.int32)
    assert oracle.kv_replace([0], [40], bt, seq_len, table, free, top) == 0
    assert table.tolist() == [[1, 0, 3, -1], [2, -1, -1, -1]] and seq_len.tolist() == [40, 7] and top[0] == 2
    assert free[:2].tolist() == [5, 4]
    # an empty replacement only returns blocks; asking for more than exist changes nothing
    assert oracle.kv_replace([1], [0], bt, seq_len, table, free, top) == 0
    assert table[1].tolist() == [-1] * 4 and top[0] == 3 and free[:3].tolist() == [5, 4, 2] and seq_len[1] == 0
    before = (seq_len.copy(), table.copy(), free.copy(), top.copy())
    assert oracle.kv_replace([1], [64], bt, seq_len, table, free, top) == -1
    assert all(np.array_equal(a, b) for a, b in zip(before, (seq_len, table, free, top)))


# ---- the paper's reporting formula (Section 2.2) against its own tables ---------------------------------------

def test_amdahl_bound_against_paper_tables(golden_dir):
    g = {l.split()[0]: float(l.split()[1]) for l in open(os.path.join(golden_dir, "paper_tables.txt"))
         if l.strip() and not l.startswith("#")}
    from paper_2604_26779_b200.report import step_speedup_bound
    for tag in ("rl_zero", "rl_think"):
        r_gen = g[f"{tag}_gen_ar"] / g[f"{tag}_step_ar"]
        s_gen = g[f"{tag}_gen_ar"] / g[f"{tag}_gen_spec"]
        assert abs(step_speedup_bound(r_gen, s_gen) - g[f"{tag}_step_speedup"]) < 0.015
    # the three simulator pairs (rollout, end-to-end) imply the same generation share
    shares = []
    for s in "abc":
        ro, e2e = g[f"sim_rollout_{s}"], g[f"sim_e2e_{s}"]
        shares.append((1 - 1 / e2e) / (1 - 1 / ro))
    assert max(shares) - min(shares) < 0.005 and abs(np.mean(shares) - 0.65) < 0.005


def test_kv_bookkeeping_random_walk_with_replacement():
    """Random sequences of reserve / commit / replace / retire: blocks are conserved, no block is owned twice, every live
    sequence owns exactly the blocks its length needs after a commit, retired slots own nothing and are passed over."""
    rng = np.random.default_rng(12)
    B, bt, maxb, nblk, k = 6, 16, 10, 40, 3
    seq_len = np.zeros(B, np.int32)
    table = np.full((B, maxb), -1, np.int32)
    free = inputs.make_block_order(nblk, 9)
    top = np.array([nblk], np.int32)
    everything = set(free.tolist())
    for it in range(400):
        live = seq_len >= 0
        if oracle.kv_reserve(k, bt, seq_len, table, free, top) == 0:
            n = rng.integers(1, k + 2, B).astype(np.int32)
            before = seq_len.copy()
            oracle.kv_commit(bt, n, seq_len, table, free, top)
            assert np.all(seq_len[live] == before[live] + n[live]) and np.all(seq_len[~live] == -1)
        owned = table[table >= 0]
        assert len(set(owned.tolist())) == owned.size and owned.size + top[0] == nblk
        assert set(owned.tolist()) | set(free[: top[0]].tolist()) == everything
        for b in range(B):
            keep = 0 if seq_len[b] < 0 else -(-int(seq_len[b]) // bt)
            assert np.all(table[b, :keep] >= 0) and np.all(table[b, keep:] == -1)
        # finished or overlong sequences leave; their slot gets a new prompt, or retires
        leave = [b for b in range(B) if seq_len[b] >= 0 and (seq_len[b] + k + 1 > (maxb - 1) * bt or rng.random() < 0.05)]
        back = [b for b in range(B) if seq_len[b] < 0 and rng.random() < 0.3]
        if leave or back:
            slots = leave + back
            new_len = [int(rng.choice([-1, 0, 5, 33])) for _ in leave] + [int(rng.choice([0, 17])) for _ in back]
            r = oracle.kv_replace(slots, new_len, bt, seq_len, table, free, top)
            assert r in (0, -1)
            if r == 0:
                for s_, nl in zip(slots, new_len):
                    assert seq_len[s_] == (nl if nl >= 0 else -1)


# ---- 8-bit KV cache codes ------------------------------------------------------------------------------------

def test_e4m3_codes_match_the_library_cast():
    """The oracle's e4m3 rounding (nearest even, saturating at 448) against torch's float8_e4m3fn cast on every code's
    value, on the midpoints between neighbouring codes, and on random values; the read-back is exact."""
    import torch
    codes = np.arange(256, dtype=np.uint8)
    vals = oracle.e4m3_dequantize(codes)
    ref_vals = torch.from_numpy(codes).view(torch.float8_e4m3fn).float().numpy()
    finite = np.isfinite(ref_vals)
    assert np.array_equal(vals[finite], ref_vals[finite]) and np.all(np.isnan(vals[~finite]))
    assert vals[0x7e] == 448.0 and vals[0x01] == 2.0 ** -9 and vals[0x08] == 2.0 ** -6
    pos = np.sort(vals[finite & (vals >= 0)])
    mids = ((pos[:-1].astype(np.float64) + pos[1:].astype(np.float64)) / 2).astype(np.float32)     # exact in fp32
    rng = np.random.default_rng(5)
    xs = np.concatenate([pos, -pos, mids, -mids, rng.normal(0, 1, 20000).astype(np.float32),
                         rng.normal(0, 100, 20000).astype(np.float32), (rng.normal(0, 1e-3, 5000)).astype(np.float32),
                         np.array([447.9, 448.0, 463.9], np.float32)])
    xs = xs[np.abs(xs) < 464.0]                                   # beyond the last rounding boundary torch returns NaN, we saturate
    got = oracle.e4m3_quantize(xs)
    ref = torch.from_numpy(xs).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(got, ref)
    assert oracle.e4m3_quantize(np.array([1e9, -1e9], np.float32)).tolist() == [0x7e, 0xfe]      # saturation, not NaN
    # a scale divides before rounding and multiplies after
    x = rng.normal(0, 3, 1000).astype(np.float32)
    assert np.array_equal(oracle.e4m3_roundtrip(x, 0.25), oracle.e4m3_dequantize(oracle.e4m3_quantize(x / np.float32(0.25))) * np.float32(0.25))
    assert np.max(np.abs(oracle.e4m3_roundtrip(x) - x) / np.maximum(np.abs(x), 2.0 ** -6)) <= 2.0 ** -4 + 1e-7


def test_kv_compact_hand_worked():
    # 4 slots, 16-token blocks, 10 blocks.  Slot 0 holds 20 tokens (blocks 9, 8), slot 1 holds 5 (block 7), slot 2 is retired,
    # slot 3 holds 33 (blocks 6, 5, 4); free stack below the top: [0, 1, 2, 3].
    bt = 16
    seq_len = np.array([20, 5, -1, 33], np.int32)
    table = np.full((4, 4), -1, np.int32)
    table[0, :2] = [9, 8]; table[1, :1] = [7]; table[3, :3] = [6, 5, 4]
    free = np.array([0, 1, 2, 3, -1, -1, -1, -1, -1, -1], np.int32)
    top = np.array([4], np.int32)
    new_len, new_table = oracle.kv_compact([1, 3], bt, seq_len, table, free, top)
    # worked by hand: slot 0 is dropped (its blocks 9 then 8 are pushed), slot 2 owns nothing; slots 1 and 3 move to 0 and 1
    assert top[0] == 6 and free[:6].tolist() == [0, 1, 2, 3, 9, 8]
    assert new_len.tolist() == [5, 33]
    assert new_table.tolist() == [[7, -1, -1, -1], [6, 5, 4, -1]]
    # blocks are conserved: free ones plus owned ones are all ten, none twice
    owned = [b for row in new_table for b in row if b >= 0]
    assert sorted(free[: top[0]].tolist() + owned) == list(range(10))
    # keeping everything is the identity
    l2, t2 = oracle.kv_compact([0, 1], bt, new_len.copy(), new_table.copy(), free, top)
    assert l2.tolist() == [5, 33] and t2.tolist() == new_table.tolist() and top[0] == 6
