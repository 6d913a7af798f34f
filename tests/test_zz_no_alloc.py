"""spec_attention_noalloc: the attention entry point for callers that cannot allocate device memory (its scratch is a
32 MiB array inside the library).  Checked against spec_attention, which takes the scratch from the caller, on two calls
in a row with different inputs, so that anything the first call leaves in the shared array would show in the second.
This file sorts last on purpose: a run that stops at the first failure has by then run every other test.
"""
import numpy as np
import pytest

from tests.test_gpu_ops import paged_case

torch = pytest.importorskip("torch")


def test_oversize_request_is_refused_on_the_host():
    """More scratch than the built-in 32 MiB -> SPEC_ERR_SHAPE before anything touches a device (runs without a GPU)."""
    from paper_2604_26779_b200 import binding
    L = binding.lib()
    fake = 4096                                     # non-null, never dereferenced on the host
    need = L.spec_attention_scratch_bytes(256, 4, 32, 8, 128, 16640)
    assert need > 32 << 20
    assert L.spec_attention_noalloc(256, 4, 32, 8, 128, 16, 1040, fake, fake, fake, fake, fake, fake, 0, None) == -2
    assert L.spec_attention_noalloc(4, 4, 32, 8, 128, 16, 64, None, fake, fake, fake, fake, fake, 0, None) == -1
    assert L.spec_attention_noalloc(0, 4, 32, 8, 128, 16, 64, None, None, None, None, None, None, 0, None) == 0


@pytest.mark.gpu
def test_noalloc_attention_matches_spec_attention_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_26779_b200 import binding as api
    api.lib()
    cases = [([0, 17, 700, 2049, 5003, 33], 4, 32, 8, 128, 11), ([2600, 5, 1500], 4, 32, 8, 128, 12)]
    for lens, R, Hq, Hkv, dh, seed in cases:
        q, kpool, vpool, table, _ = paged_case(lens, R, Hq, Hkv, dh, torch.bfloat16, seed=seed)
        B = len(lens)
        dq = torch.from_numpy(q).cuda().to(torch.bfloat16)
        dk, dv = torch.from_numpy(kpool).cuda().to(torch.bfloat16), torch.from_numpy(vpool).cuda().to(torch.bfloat16)
        dt, dl = torch.from_numpy(table).cuda(), torch.tensor(lens, dtype=torch.int32, device="cuda")
        ref = torch.zeros((B, R, Hq, dh), dtype=torch.bfloat16, device="cuda")
        scratch = torch.zeros(api.spec_attention_scratch_bytes(B, R, Hq, Hkv, dh, table.shape[1] * 16), dtype=torch.uint8, device="cuda")
        api.spec_attention(dq, dk, dv, dt, dl, ref, scratch)
        got = torch.full_like(ref, 3.0)
        api.spec_attention_noalloc(dq, dk, dv, dt, dl, got)
        torch.cuda.synchronize()
        a, b = got.float().cpu().numpy(), ref.float().cpu().numpy()
        err = np.abs(a - b).max(-1) / np.maximum(np.abs(b).max(-1), 1e-6)
        assert err.max() < 2e-2, err.max()              # the bar of the attention tests; the two paths run the same kernels
        assert np.isfinite(a).all()
