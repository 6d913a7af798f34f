"""GPU parity of the two heavy operators through their stateless C entry points: paged grouped-query attention and
the GEMM, against the CPU oracle / fp64 products on the same seeded bytes.

Bars: bf16 results within 2e-2 of the row's largest magnitude (the same inf-norm-relative bar as for logits), fp32
results within 1e-4.
"""
import numpy as np
import pytest

from oracle import model
from paper_2604_26779_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26779_b200 import binding
    binding.lib()
    return binding


def paged_case(lens, R, Hq, Hkv, dh, dtype, seed):
    """Random cache contents in a permuted block pool; returns device tensors and the logical K/V per sequence."""
    B, bt = len(lens), 16
    rng = np.random.default_rng(seed)
    max_blocks = -(-(max(lens) + R) // bt) + 1
    nblk = sum(-(-(l + R) // bt) for l in lens) + 5
    order = inputs.make_block_order(nblk, seed)
    table = np.full((B, max_blocks), -1, np.int32)
    nxt = 0
    for b, l in enumerate(lens):
        for j in range(-(-(l + R) // bt)):
            table[b, j] = order[nxt]
            nxt += 1
    kind = "bf16" if dtype == torch.bfloat16 else "f32"
    kpool = inputs.make_kv_values((nblk, Hkv, bt, dh), seed + 1, kind)
    vpool = inputs.make_kv_values((nblk, Hkv, bt, dh), seed + 2, kind)
    q = inputs.make_kv_values((B, R, Hq, dh), seed + 3, kind)
    logical = []
    for b, l in enumerate(lens):
        n = l + R
        blocks = table[b, : -(-n // bt)]
        k = kpool[blocks].transpose(0, 2, 1, 3).reshape(-1, Hkv, dh)[:n]
        v = vpool[blocks].transpose(0, 2, 1, 3).reshape(-1, Hkv, dh)[:n]
        logical.append((k, v))
    return q, kpool, vpool, table, logical


@pytest.mark.parametrize("lens,R,Hq,Hkv,dh,dtype", [
    ([0, 1, 15, 16, 17, 700, 2047, 2048, 2049, 5003], 4, 32, 8, 128, torch.bfloat16),   # 8B shape: 16 rows per KV head
    ([3, 100, 4100], 1, 32, 8, 128, torch.bfloat16),                                   # plain decode rows
    ([64, 777, 2500], 5, 16, 4, 128, torch.bfloat16),                                  # k = 4: 20 rows -> two row tiles
    ([10, 300, 2100], 8, 8, 2, 128, torch.bfloat16),                                   # k = 7: 32 rows
    ([50, 1234], 4, 32, 2, 128, torch.bfloat16),                                       # group 16: 64 rows (MoE layer shape)
    ([0, 7, 127, 128, 129, 4093, 4100, 9001], 4, 32, 2, 128, torch.bfloat16),          # 64 rows, tile edges, several chunks
    ([33, 640, 5000], 8, 32, 2, 128, torch.bfloat16),                                  # k = 7 on a 16-head group: 128 rows
    ([100, 3000], 17, 2, 2, 128, torch.bfloat16),                                      # 17 rows: just past the 16-row kernel
    ([5, 130, 2300], 4, 8, 4, 64, torch.bfloat16),                                     # head_dim 64
    ([0, 9, 40, 333], 4, 4, 4, 64, torch.float32),                                     # fp32 reference path
])
def test_paged_attention_matches_oracle(api, lens, R, Hq, Hkv, dh, dtype):
    q, kpool, vpool, table, logical = paged_case(lens, R, Hq, Hkv, dh, dtype, seed=len(lens) * 7 + R)
    B = len(lens)
    dq = torch.from_numpy(q).cuda().to(dtype)
    dk, dv = torch.from_numpy(kpool).cuda().to(dtype), torch.from_numpy(vpool).cuda().to(dtype)
    out = torch.full((B, R, Hq, dh), 7.0, dtype=dtype, device="cuda")
    nbytes = api.spec_attention_scratch_bytes(B, R, Hq, Hkv, dh, table.shape[1] * 16)
    scratch = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    api.spec_attention(dq, dk, dv, torch.from_numpy(table).cuda(), torch.tensor(lens, dtype=torch.int32, device="cuda"),
                       out, scratch)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy()
    tol = 2e-2 if dtype == torch.bfloat16 else 1e-4
    worst = 0.0
    for b, l in enumerate(lens):
        k, v = logical[b]
        ref = model.attention(q[b].astype(np.float64), k.astype(np.float64), v.astype(np.float64), n_past=l)
        err = np.abs(got[b] - ref).max(-1) / np.abs(ref).max(-1)
        worst = max(worst, float(err.max()))
    print(f"attention R={R} Hq={Hq}/{Hkv} dh={dh} {dtype}: worst row error {worst:.2e}")
    assert worst < tol


@pytest.mark.parametrize("M,N,K,din,dout,acc", [
    (16, 768, 256, torch.float32, torch.float32, False),
    (5, 1024, 1024, torch.float32, torch.float32, True),
    (128, 256, 64, torch.bfloat16, torch.float32, False),          # one tile, one k-step
    (128, 256, 512, torch.bfloat16, torch.bfloat16, False),
    (1024, 6144, 4096, torch.bfloat16, torch.bfloat16, False),     # 8B QKV projection
    (1024, 4096, 14336, torch.bfloat16, torch.float32, True),      # 8B down projection into the fp32 residual
    (256, 4096, 4096, torch.bfloat16, torch.float32, True),        # decode-sized M: two m-tiles per CTA
    (200, 1000, 2048, torch.bfloat16, torch.bfloat16, False),      # the same variant with ragged M and N
    (129, 512, 320, torch.bfloat16, torch.float32, False),
    (1000, 520, 192, torch.bfloat16, torch.bfloat16, False),       # ragged M and N tails
    (77, 1000, 4096, torch.bfloat16, torch.float32, False),
    (1024, 16384, 1024, torch.bfloat16, torch.float32, False),     # LM-head-like slice: fp32 logits
    # very few rows (thin-batch kernel: weights as the MMA's M operand): every token-tile width, ragged M and N, both outputs
    (1, 4096, 4096, torch.bfloat16, torch.float32, False),
    (7, 96, 256, torch.bfloat16, torch.bfloat16, False),
    (8, 6144, 4096, torch.bfloat16, torch.bfloat16, False),
    (9, 1000, 512, torch.bfloat16, torch.float32, True),
    (16, 4096, 14336, torch.bfloat16, torch.float32, True),
    (17, 28672, 4096, torch.bfloat16, torch.bfloat16, False),
    (31, 50, 768, torch.bfloat16, torch.bfloat16, True),
    (32, 16384, 4096, torch.bfloat16, torch.float32, False),
    (32, 4096, 4096, torch.bfloat16, torch.float32, True),         # 17..64 rows: the tensor-core kernel with swapped operands (weights as the M operand)
    (20, 6144, 4096, torch.bfloat16, torch.bfloat16, False),
    (25, 4000, 14336, torch.bfloat16, torch.float32, True),
    (32, 4096, 320, torch.bfloat16, torch.float32, False),
    (33, 1000, 512, torch.bfloat16, torch.float32, False),         # 64-wide token tile, ragged features
    (48, 6144, 4096, torch.bfloat16, torch.bfloat16, True),
    (64, 4096, 4096, torch.bfloat16, torch.float32, True),
])
def test_gemm_matches_fp64(api, M, N, K, din, dout, acc):
    kind = "bf16" if din == torch.bfloat16 else "f32"
    A = inputs.make_kv_values((M, K), 1, kind)
    W = inputs.make_kv_values((N, K), 2, kind) * np.float32(0.05)
    W = inputs.round_to_bf16(W) if kind == "bf16" else W
    C0 = inputs.make_kv_values((M, N), 3, "bf16" if dout == torch.bfloat16 else "f32")
    dA, dW = torch.from_numpy(A).cuda().to(din), torch.from_numpy(W).cuda().to(din)
    dC = torch.from_numpy(C0).cuda().to(dout)
    api.spec_gemm(dA, dW, dC, accumulate=acc)
    torch.cuda.synchronize()
    # fp64 reference on sampled rows (all rows when small)
    rows = np.arange(M) if M * N * K < 2e9 or M <= 128 else np.unique(np.concatenate([np.arange(0, M, 37), [M - 1, M - 2, 127, 128]]))
    ref = A[rows].astype(np.float64) @ W.astype(np.float64).T + (C0[rows].astype(np.float64) if acc else 0.0)
    got = dC.float().cpu().numpy()[rows]
    err = np.abs(got - ref).max(-1) / np.abs(ref).max(-1)
    print(f"gemm {M}x{N}x{K} {din}->{dout} acc={acc}: worst row error {err.max():.2e}")
    assert err.max() < (2e-2 if dout == torch.bfloat16 else (1e-3 if din == torch.bfloat16 else 1e-5))


def test_bounded_wait_times_out_cleanly(api):
    """A wait that nothing satisfies gives up after its limit, reports SPEC_ERR_TIMEOUT, and leaves the device usable."""
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    el = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert api.lib().spec_selftest_bounded_wait(st.data_ptr(), el.data_ptr(), torch.cuda.current_stream().cuda_stream) == 0
    torch.cuda.synchronize()
    assert st[0].item() == -19 and 1500 < el.item() < 200000
    # the context is intact: a GEMM right after still gives the right answer
    A = torch.randn((128, 64), device="cuda", dtype=torch.bfloat16)
    W = torch.randn((256, 64), device="cuda", dtype=torch.bfloat16)
    Cc = torch.zeros((128, 256), device="cuda", dtype=torch.float32)
    api.spec_gemm(A, W, Cc)
    torch.cuda.synchronize()
    assert torch.allclose(Cc, A.float() @ W.float().t(), atol=1e-2, rtol=1e-3)


@pytest.mark.parametrize("M,N,K,dout,acc", [
    (128, 256, 128, torch.float32, False),             # one tile, one k-block
    (1024, 4096, 4096, torch.bfloat16, False),
    (300, 1000, 14336, torch.float32, True),           # ragged M and N, long K
    (64, 512, 272, torch.float32, False),              # K not a multiple of the 128-element k-block
])
def test_gemm_e4m3_matches_oracle(api, M, N, K, dout, acc):
    """8-bit projection: the row quantiser's codes and scales equal the oracle's bit for bit (same bf16 inputs), and the
    product of the codes - exact integer-like arithmetic in fp32 accumulation - matches the oracle's fp64 product of the
    dequantised operands to fp32 rounding."""
    import oracle
    A = inputs.round_to_bf16(inputs.make_kv_values((M, K), 11, "bf16"))
    W = inputs.round_to_bf16(inputs.make_kv_values((N, K), 12, "bf16") * np.float32(0.05))
    C0 = inputs.make_kv_values((M, N), 13, "bf16" if dout == torch.bfloat16 else "f32")
    dA, dW = torch.from_numpy(A).cuda().to(torch.bfloat16), torch.from_numpy(W).cuda().to(torch.bfloat16)
    a8, w8 = torch.empty((M, K), dtype=torch.uint8, device="cuda"), torch.empty((N, K), dtype=torch.uint8, device="cuda")
    sa, sw = torch.empty(M, dtype=torch.float32, device="cuda"), torch.empty(N, dtype=torch.float32, device="cuda")
    api.spec_quantize_rows(dA, a8, sa)
    api.spec_quantize_rows(dW, w8, sw)
    oa, osa = oracle.e4m3_quantize_rows(A)
    ow, osw = oracle.e4m3_quantize_rows(W)
    assert np.array_equal(a8.cpu().numpy(), oa) and np.array_equal(sa.cpu().numpy(), osa)
    assert np.array_equal(w8.cpu().numpy(), ow) and np.array_equal(sw.cpu().numpy(), osw)
    dC = torch.from_numpy(C0).cuda().to(dout)
    api.spec_gemm_e4m3(a8, sa, w8, sw, dC, accumulate=acc)
    torch.cuda.synchronize()
    rows = np.arange(M) if M <= 300 else np.unique(np.concatenate([np.arange(0, M, 37), [M - 1, 127, 128]]))
    ref = model.proj({"w_fp8": True}, A[rows], W) + (C0[rows].astype(np.float64) if acc else 0.0)
    got = dC.float().cpu().numpy()[rows]
    err = np.abs(got - ref).max(-1) / np.abs(ref).max(-1)
    print(f"e4m3 gemm {M}x{N}x{K} ->{dout} acc={acc}: worst row error {err.max():.2e}")
    assert err.max() < (1e-2 if dout == torch.bfloat16 else 1e-5)
