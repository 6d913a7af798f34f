"""The smoke entry point as a test: one speculation step of a 2-layer, full-width (d=4096) bf16 model on 8 ragged
sequences, checked against the oracle.  At M=32 rows the O and down projections have few tiles, so this also covers the
split-K path of the tensor-core GEMM."""
import pytest

torch = pytest.importorskip("torch")


@pytest.mark.gpu
def test_smoke_entry_point():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as g
    g.smoke()
