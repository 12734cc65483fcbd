"""Parity of the weight-streaming skinny GEMM (csd_linear) with the oracle's contraction."""
import numpy as np
import pytest
import torch

from gpu_util import rel_l2, require_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=[1, 2, 3], ids=["cuda-core", "tensor-core", "tensor-core-row-ranges"])
def b(request):
    """Every test here runs once per GEMM kernel: 128-bit loads + fp32 FMA, TMA + tcgen05 with equal
    shares of (tile, K block) units, and TMA + tcgen05 with whole output columns per CTA."""
    require_gpu()
    from paper_2312_11462_b200 import binding
    binding.csd_set_gemm_path(request.param)
    yield binding
    binding.csd_set_gemm_path(0)


def case(b, orc, m, N, K, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    W = (0.05 * torch.randn(N, K, generator=g, device="cuda")).to(torch.bfloat16)
    X = torch.randn(m, K, generator=g, device="cuda")
    Y = b.csd_linear(W, X)
    Y2 = b.csd_linear(W, X)                      # split-K partials are summed in a fixed order
    assert torch.equal(Y, Y2)
    ref = orc.linear(orc.blob_to_u16(W).reshape(N, K), X.cpu().numpy())
    got = Y.cpu().numpy()
    # fp32 accumulation of K products of magnitude |w||x|: error ~ sqrt(K) * 2^-24 * |y|
    # (the tensor cores add partial products with a little less care than an fp32 FMA chain)
    assert rel_l2(got, ref) < 5e-6, (m, N, K)
    assert np.abs(got - ref).max() < 1e-4 * max(1.0, np.abs(ref).max())


@pytest.mark.parametrize("m", [1, 2, 5, 8, 9, 16, 17])
def test_layer_shapes(b, orc, m):
    # the matrix shapes of the small models plus ragged ones (N not a tile multiple, K one
    # partial step, K with a tail slice)
    for N, K in ((768, 768), (2304, 768), (4096, 256), (256, 1024), (64, 64), (1000, 136), (37, 2056), (4099, 520)):
        case(b, orc, m, N, K, seed=N + K + m)


def test_every_block_size(b, orc):
    # all seventeen row counts (every operand padding of the tensor-core kernels: 16, 32, 48, 64 rows of
    # terms) on a shape with several tiles per CTA share and on one with a single short tile
    for m in range(1, 18):
        case(b, orc, m, 3072, 4096, seed=100 + m)
        case(b, orc, m, 200, 1160, seed=200 + m)


@pytest.mark.parametrize("N,K", [(4096, 4096), (12288, 4096), (4096, 11008)])
def test_7b_layer_shapes(b, orc, N, K):
    for m in (5, 17):
        case(b, orc, m, N, K, seed=m)


def test_head_shape_and_uneven_ranges(b, orc):
    # the vocabulary projection (two row ranges per CTA in the row-range kernel) and row counts
    # that leave ranges of unequal length, a K tail and fewer K blocks than a stage holds
    for m, N, K in ((5, 32000, 4096), (3, 20011, 1032), (8, 2371, 4104), (2, 2368, 72)):
        case(b, orc, m, N, K, seed=N + m)


def test_wide_blocks(orc):
    # 18 to 128 rows: the wide-block tensor-core kernel of the prefill.  Each fp32 value enters as two
    # bf16 terms (16 mantissa bits), so the bound is 2^-17-sized, not the 5e-6 of the review kernels.
    require_gpu()
    from paper_2312_11462_b200 import binding as b
    for m, N, K in ((18, 4096, 4096), (64, 12288, 4096), (128, 4096, 11008), (127, 32000, 4096), (33, 4099, 520),
                    (100, 20011, 1032), (128, 2371, 4104)):
        g = torch.Generator(device="cuda")
        g.manual_seed(m + N)
        W = (0.05 * torch.randn(N, K, generator=g, device="cuda")).to(torch.bfloat16)
        X = torch.randn(m, K, generator=g, device="cuda")
        Y = b.csd_linear(W, X)
        assert torch.equal(Y, b.csd_linear(W, X))
        rows = [0, 1, m // 2, m - 2, m - 1]                 # the oracle on a few rows bounds its cost
        ref = orc.linear(orc.blob_to_u16(W).reshape(N, K), X[rows].cpu().numpy())
        got = Y[rows].cpu().numpy()
        assert rel_l2(got, ref) < 3e-5, (m, N, K, rel_l2(got, ref))
        # every row against a float64 product on the GPU side of the harness (torch matmul as the library step)
        full = (X.double() @ W.double().T)
        assert float((Y.double() - full).norm() / full.norm()) < 3e-5
    assert b.csd_device_status() == 0
