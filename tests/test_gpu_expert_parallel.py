"""GPU parity of the expert-parallel mixture-of-experts block (route -> pull rows from peers -> grouped expert GEMMs ->
pull outputs back and combine), ranks emulated inside one process on one GPU (stream order is the barrier).

Bars: the receive layout (offsets, row order, received rows) is index / byte work and must match the oracle's layout
exactly; the top-k choice is taken on the device's own fp32 router logits; outputs within 2e-2 of the row maximum (bf16
operands, as for the single-GPU block); and a token's output must be BIT-identical for every ep_size (the arithmetic per
row does not depend on where the row is computed).
"""
import numpy as np
import pytest

from oracle import model
from paper_2604_26779_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def make_case(E, top_k, d, Fe, rows_per_rank, seed, on_device=False):
    if on_device:                                            # large shapes: seeded normal draws on the device
        g = torch.Generator(device="cuda").manual_seed(seed)
        rn = lambda shape, scale: (torch.randn(shape, generator=g, device="cuda", dtype=torch.float32) * scale).to(torch.bfloat16)
        lw = dict(router=rn((E, d), 4 / np.sqrt(d)), experts_gate=rn((E, Fe, d), 1 / np.sqrt(d)),
                  experts_up=rn((E, Fe, d), 1 / np.sqrt(d)), experts_down=rn((E, d, Fe), 1 / np.sqrt(Fe)))
        hs = [rn((n, d), 1.0) for n in rows_per_rank]
        xs = [torch.randn((n, d), generator=g, device="cuda", dtype=torch.float32).cpu() for n in rows_per_rank]
        return lw, hs, xs
    rng = np.random.default_rng(seed)
    bf = lambda a: torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16)
    lw = dict(router=bf(rng.standard_normal((E, d)) / np.sqrt(d) * 4),
              experts_gate=bf(rng.standard_normal((E, Fe, d)) / np.sqrt(d)),
              experts_up=bf(rng.standard_normal((E, Fe, d)) / np.sqrt(d)),
              experts_down=bf(rng.standard_normal((E, d, Fe)) / np.sqrt(Fe)))
    hs = [bf(rng.standard_normal((n, d))) for n in rows_per_rank]
    xs = [torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32)) for n in rows_per_rank]
    return lw, hs, xs


def run_ep(lw, hs, xs, ep_size, top_k, cap_rows=None):
    from paper_2604_26779_b200 import expert_parallel as ep
    from paper_2604_26779_b200.engine import stack_gate_up
    E, Fe, d = lw["experts_gate"].shape
    per = E // ep_size
    max_rows = max(max(h.shape[0] for h in hs), 1)
    ranks = [ep.EpRank(ep_size, r, E, top_k, d, Fe, max_rows, cap_rows) for r in range(ep_size)]
    router = lw["router"].cuda()
    gus = [stack_gate_up(lw["experts_gate"][r * per : (r + 1) * per], lw["experts_up"][r * per : (r + 1) * per]).contiguous().cuda()
           for r in range(ep_size)]
    dns = [lw["experts_down"][r * per : (r + 1) * per].contiguous().cuda() for r in range(ep_size)]
    xd = [x.clone().cuda() for x in xs]
    ep.run_block_single_process(ranks, [h.cuda() for h in hs], router, gus, dns, xd)
    torch.cuda.synchronize()
    return ranks, xd


def f64(t):
    return t.to(torch.float32).cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("ep_size,rows", [(1, [37]), (2, [37, 150]), (4, [37, 150, 0, 260]), (8, [5, 16, 0, 33, 129, 7, 64, 1])])
def test_ep_block_layout_and_outputs(ep_size, rows):
    E, top_k, d, Fe = 16, 4, 512, 128
    lw, hs, xs = make_case(E, top_k, d, Fe, rows, seed=100 + ep_size)
    ranks, xd = run_ep(lw, hs, xs, ep_size, top_k)
    for r in ranks:
        r.check_status()
    per = E // ep_size
    # routing decisions on the device's own logits are covered by the single-GPU block's test; here: take the device's ids
    ids = [r.tensor("IDS")[: n].cpu().numpy() for r, n in zip(ranks, rows)]
    wts = [r.tensor("WTS")[: n].cpu().numpy() for r, n in zip(ranks, rows)]
    for s in range(ep_size):
        if rows[s]:
            lg = f64(hs[s]) @ f64(lw["router"]).T
            o_ids, o_w = model.moe_route(lg, top_k)
            # fp32 tensor-core logits vs fp64: a swap can only happen between near-equal logits
            diff = o_ids != ids[s]
            if diff.any():
                srt = np.sort(lg, -1)[:, ::-1]
                gaps = np.abs(srt[:, : top_k] - srt[:, 1 : top_k + 1]).min(-1)
                assert (gaps[diff.any(-1)] < 1e-3).all()
            assert np.allclose(wts[s].sum(-1), 1.0, atol=1e-5)
    rows_o, off_o = model.ep_receive_layout(ids, E, ep_size)
    for dr, r in enumerate(ranks):
        assert int(r.tensor("RECV_TOTAL")[0]) == len(rows_o[dr])
        assert np.array_equal(r.tensor("RECV_OFF").cpu().numpy(), off_o[dr])
        got = r.tensor("RECV_ROWS")[: len(rows_o[dr])].cpu()
        for t, (e, s, m, j) in enumerate(rows_o[dr]):
            assert torch.equal(got[t], hs[s][m]), (dr, t)
        counts = r.tensor("COUNTS").cpu().numpy()
        assert np.array_equal(counts, np.bincount(ids[dr].reshape(-1), minlength=E))
    # outputs against the oracle's expert-parallel flow, routed with the device's decisions
    lw64 = {k: f64(v) for k, v in lw.items()}
    worst = 0.0
    for s in range(ep_size):
        if not rows[s]:
            continue
        m = f64(hs[s])
        ref = np.zeros_like(m)
        for t in range(m.shape[0]):
            for j in range(top_k):
                e = ids[s][t, j]
                ref[t] += float(wts[s][t, j]) * ((model.silu(lw64["experts_gate"][e] @ m[t]) * (lw64["experts_up"][e] @ m[t])) @ lw64["experts_down"][e].T)
        got = xd[s].cpu().numpy().astype(np.float64) - xs[s].numpy().astype(np.float64)
        worst = max(worst, float((np.abs(got - ref).max(-1) / np.abs(ref).max(-1)).max()))
    print(f"ep_size {ep_size}: worst relative error of the block output {worst:.2e}")
    assert worst < 2e-2


def test_ep_output_is_bit_identical_across_ep_sizes():
    E, top_k, d, Fe = 16, 4, 512, 128
    rows = [70, 3, 129, 40]
    lw, hs, xs = make_case(E, top_k, d, Fe, rows, seed=7)
    _, x4 = run_ep(lw, hs, xs, 4, top_k)
    _, x2 = run_ep(lw, [torch.cat(hs[:2]), torch.cat(hs[2:])], [torch.cat(xs[:2]), torch.cat(xs[2:])], 2, top_k)
    _, x1 = run_ep(lw, [torch.cat(hs)], [torch.cat(xs)], 1, top_k)
    a = torch.cat([x.cpu() for x in x4])
    assert torch.equal(a, torch.cat([x.cpu() for x in x2]))
    assert torch.equal(a, x1[0].cpu())
    assert not torch.equal(a, torch.cat(xs))


def test_ep_capacity_overflow_is_reported_not_fatal():
    from paper_2604_26779_b200 import binding as api
    E, top_k, d, Fe = 16, 4, 512, 128
    rows = [64, 64]
    lw, hs, xs = make_case(E, top_k, d, Fe, rows, seed=9)
    ranks, xd = run_ep(lw, hs, xs, 2, top_k, cap_rows=128)       # 512 entries for 2 ranks: about 256 each, capacity 128
    status = [r.status.cpu().tolist() for r in ranks]
    totals = [int(r.tensor("RECV_TOTAL")[0]) for r in ranks]
    assert sum(totals) == 512
    for st, tot in zip(status, totals):
        if tot > 128:
            assert st[0] == -20 and st[1] == tot                 # SPEC_ERR_EP_CAPACITY, detail = rows routed here
            assert api.STATUS_NAMES[st[0]] == "SPEC_ERR_EP_CAPACITY"
    assert any(t > 128 for t in totals)
    assert all(torch.isfinite(x).all() for x in xd)


def test_ep_host_errors():
    from paper_2604_26779_b200 import binding as api
    ok = api.spec_ep_config(2, 0, 16, 4, 512, 128, 64, 256)
    api.spec_ep_query_sizes(ok)
    for bad, code in [(api.spec_ep_config(3, 0, 16, 4, 512, 128, 64, 256), -2),      # experts not divisible by ranks
                      (api.spec_ep_config(2, 2, 16, 4, 512, 128, 64, 256), -1),      # rank out of range
                      (api.spec_ep_config(32, 0, 64, 4, 512, 128, 64, 256), -3),     # more ranks than supported
                      (api.spec_ep_config(2, 0, 16, 4, 500, 128, 64, 256), -2),
                      (api.spec_ep_config(2, 0, 16, 40, 512, 128, 64, 256), -2)]:
        with pytest.raises(api.SpecError) as e:
            api.spec_ep_query_sizes(bad)
        assert e.value.code == code
    # the 8-bit form wants both scale arrays
    sizes = api.spec_ep_query_sizes(ok)
    win = torch.zeros(sizes.window_bytes, dtype=torch.uint8, device="cuda")
    scr = torch.zeros(sizes.scratch_bytes, dtype=torch.uint8, device="cuda")
    w = torch.zeros(16, dtype=torch.uint8, device="cuda")
    sc = torch.ones(16, dtype=torch.float32, device="cuda")
    for gs, ds in ((None, sc), (sc, None)):
        with pytest.raises(api.SpecError) as e:
            api.spec_ep_experts_e4m3(ok, [win.data_ptr(), win.data_ptr()], scr, w, gs, w, ds)
        assert e.value.code == -1


def test_ep_block_235b_shape_sampled():
    # 128 experts, top-8, d 4096, expert FFN 1536: four ranks of 256 rows; sampled rows against the oracle
    E, top_k, d, Fe = 128, 8, 4096, 1536
    rows = [256, 256, 256, 256]
    lw, hs, xs = make_case(E, top_k, d, Fe, rows, seed=3, on_device=True)
    ranks, xd = run_ep(lw, hs, xs, 4, top_k)
    for r in ranks:
        r.check_status()
    lw64 = None
    worst = 0.0
    for s, t in [(0, 0), (1, 17), (3, 255)]:
        ids = ranks[s].tensor("IDS")[t].cpu().numpy()
        wts = ranks[s].tensor("WTS")[t].cpu().numpy()
        m = f64(hs[s][t])
        ref = np.zeros(d)
        for j in range(top_k):
            e = int(ids[j])
            g, u, dn = f64(lw["experts_gate"][e]), f64(lw["experts_up"][e]), f64(lw["experts_down"][e])
            ref += float(wts[j]) * ((model.silu(g @ m) * (u @ m)) @ dn.T)
        got = xd[s][t].cpu().numpy().astype(np.float64) - xs[s][t].numpy().astype(np.float64)
        worst = max(worst, float(np.abs(got - ref).max() / np.abs(ref).max()))
    print(f"235B-shape expert-parallel block, 4 ranks: worst sampled relative error {worst:.2e}")
    assert worst < 2e-2


def run_ep_8bit(lw, hs, xs, ep_size, top_k):
    """The block with 8-bit expert weights: every rank's local experts quantised row by row on the device."""
    from paper_2604_26779_b200 import binding as api, expert_parallel as ep
    from paper_2604_26779_b200.engine import stack_gate_up
    E, Fe, d = lw["experts_gate"].shape
    per = E // ep_size
    max_rows = max(max(h.shape[0] for h in hs), 1)
    ranks = [ep.EpRank(ep_size, r, E, top_k, d, Fe, max_rows) for r in range(ep_size)]
    gus, dns, scales = [], [], []
    for r in range(ep_size):
        gu = stack_gate_up(lw["experts_gate"][r * per : (r + 1) * per], lw["experts_up"][r * per : (r + 1) * per]).contiguous().cuda()
        dn = lw["experts_down"][r * per : (r + 1) * per].contiguous().cuda()
        gu8, dn8 = torch.empty(gu.shape, dtype=torch.uint8, device="cuda"), torch.empty(dn.shape, dtype=torch.uint8, device="cuda")
        gs = torch.empty(per * 2 * Fe, dtype=torch.float32, device="cuda")
        ds = torch.empty(per * d, dtype=torch.float32, device="cuda")
        api.spec_quantize_rows(gu.view(-1, d), gu8.view(-1, d), gs)
        api.spec_quantize_rows(dn.view(-1, Fe), dn8.view(-1, Fe), ds)
        gus.append(gu8); dns.append(dn8); scales.append((gs, ds))
    xd = [x.clone().cuda() for x in xs]
    ep.run_block_single_process(ranks, [h.cuda() for h in hs], lw["router"].cuda(), gus, dns, xd, scales=scales)
    torch.cuda.synchronize()
    for r in ranks:
        r.check_status()
    return ranks, xd


def test_ep_block_with_8bit_experts():
    """8-bit expert weights (Section 5.1 names FP8 as the precision of the paper's large-scale projection): bit-identical for
    every ep_size, and against the oracle's 8-bit block routed with the device's decisions.  The block's input rows are
    given, so both sides quantise the same rows; what is left is the rare SwiGLU output that rounds to the neighbouring
    bf16 value on one side (a code step in one element, or - for a row maximum - a 2^-8 shift of that row's scale):
    bar 1e-2 of the row maximum."""
    E, top_k, d, Fe = 16, 4, 512, 128
    rows = [70, 3, 129, 40]
    lw, hs, xs = make_case(E, top_k, d, Fe, rows, seed=21)
    r4, x4 = run_ep_8bit(lw, hs, xs, 4, top_k)
    _, x2 = run_ep_8bit(lw, [torch.cat(hs[:2]), torch.cat(hs[2:])], [torch.cat(xs[:2]), torch.cat(xs[2:])], 2, top_k)
    _, x1 = run_ep_8bit(lw, [torch.cat(hs)], [torch.cat(xs)], 1, top_k)
    a = torch.cat([x.cpu() for x in x4])
    assert torch.equal(a, torch.cat([x.cpu() for x in x2])) and torch.equal(a, x1[0].cpu())
    _, x16 = run_ep(lw, hs, xs, 4, top_k)
    assert not torch.equal(a, torch.cat([x.cpu() for x in x16]))                   # the 8-bit path really ran
    lw64 = {k: f64(v) for k, v in lw.items()}
    lwo = dict(router=lw64["router"], experts_gate=list(lw64["experts_gate"]), experts_up=list(lw64["experts_up"]),
               experts_down=list(lw64["experts_down"]))
    worst = 0.0
    for s in range(4):
        n = rows[s]
        ids = r4[s].tensor("IDS")[:n].cpu().numpy()
        wts = r4[s].tensor("WTS")[:n].cpu().numpy()
        # hand the oracle the device's decisions: logits that reproduce ids in order and the device's weights
        fake = np.full((n, E), -1e9)
        for t in range(n):
            fake[t, ids[t]] = np.log(wts[t].astype(np.float64))
        ref = model.moe_mlp(lwo, f64(hs[s]), top_k, router_logits=fake, cfg={"w_fp8": True})
        got = x4[s].cpu().numpy().astype(np.float64) - xs[s].numpy().astype(np.float64)
        worst = max(worst, float((np.abs(got - ref).max(-1) / np.abs(ref).max(-1)).max()))
    print(f"expert-parallel block, 8-bit experts: worst relative error {worst:.2e}")
    assert worst < 1e-2


def test_8bit_experts_after_a_16bit_route_is_reported():
    """spec_ep_experts_e4m3 pulls the codes spec_ep_route_e4m3 publishes; a source that routed with the 16-bit call is
    reported in the status word (SPEC_ERR_STATE, detail = the source's rank), nothing faults."""
    from paper_2604_26779_b200 import binding as api, expert_parallel as ep
    E, top_k, d, Fe = 16, 4, 512, 128
    lw, hs, xs = make_case(E, top_k, d, Fe, [20, 20], seed=5)
    ranks = [ep.EpRank(2, r, E, top_k, d, Fe, 20) for r in range(2)]
    addrs = [r.window.data_ptr() for r in ranks]
    for r in ranks:
        r.set_peers(addrs)
    ranks[0].route(hs[0].cuda(), lw["router"].cuda(), rows8=True)
    ranks[1].route(hs[1].cuda(), lw["router"].cuda(), rows8=False)              # this rank did not publish codes
    w8 = torch.zeros((8, 2 * Fe, d), dtype=torch.uint8, device="cuda")
    d8 = torch.zeros((8, d, Fe), dtype=torch.uint8, device="cuda")
    sc = (torch.ones(8 * 2 * Fe, dtype=torch.float32, device="cuda"), torch.ones(8 * d, dtype=torch.float32, device="cuda"))
    ranks[0].experts(w8, d8, scales=sc)
    torch.cuda.synchronize()
    st = ranks[0].status.cpu().tolist()
    assert st[0] == -4 and st[1] == 1 and api.STATUS_NAMES[-4] == "SPEC_ERR_STATE"
