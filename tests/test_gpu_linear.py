"""GPU parity: the tcgen05 GEMM (every projection of the forward pass) against the oracle's definition
C = A B^T evaluated in float64 on the bf16 inputs."""
import numpy as np
import pytest
import torch

from paper_2506_10848_b200 import binding as sfs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run(M, N, K, out_dtype, scale=1.0, seed=0, lda=None, ldb=None, ldc=None):
    g = torch.Generator().manual_seed(seed)
    lda, ldb, ldc = lda or K, ldb or K, ldc or N
    A = (torch.randn((M, lda), generator=g) * 0.5).to(torch.bfloat16)
    Bm = (torch.randn((N, ldb), generator=g) * 0.5).to(torch.bfloat16)
    C = torch.full((M, ldc), 7.0, dtype=torch.float32 if out_dtype else torch.bfloat16, device=DEV)
    sfs.sfs_linear(A.to(DEV), lda, Bm.to(DEV), ldb, C, ldc, M, N, K, out_dtype, scale)
    sfs.sfs_check_device_status()
    ref = scale * (A[:, :K].double().numpy() @ Bm[:, :K].double().numpy().T)
    got = C.cpu().double().numpy()
    return got, ref


@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (128, 256, 128), (96, 768, 256), (100, 200, 688), (257, 300, 72),
                                   (512, 1024, 4096), (1, 8, 8), (130, 4096, 1024)])
def test_linear_fp32_out(M, N, K):
    got, ref = run(M, N, K, 1, ldc=(N + 7) // 8 * 8)
    err = np.abs(got[:, :N] - ref).max()
    assert err <= 1e-3 * max(1.0, np.abs(ref).max()), err       # fp32 accumulation of exact bf16 products


def test_linear_bf16_out_scale_and_strides():
    got, ref = run(200, 264, 320, 0, scale=8.0, lda=328, ldb=336, ldc=272)
    assert np.all(got[:, 264:] == 7.0)                          # padding columns untouched
    rel = np.abs(got[:, :264] - ref) / np.maximum(np.abs(ref), 1.0)
    assert rel.max() <= 2.0 ** -8                               # one bf16 rounding of the fp32 result


def test_linear_wide_tile_config():
    # enough tiles that the 128 x 256 configuration is chosen
    got, ref = run(1024, 8192, 512, 1, seed=3)
    assert np.abs(got - ref).max() <= 1e-3 * np.abs(ref).max()


@pytest.mark.parametrize("M,N,K,out_dtype", [(512, 12288, 4096, 1), (512, 12288, 4096, 0), (384, 6144, 2048, 1), (512, 3000, 1024, 0)])
def test_linear_few_wide_tiles(M, N, K, out_dtype):
    """Shapes with fewer wide tiles than SM pairs (the planner narrows the tiles), large K, ragged N; bf16 and fp32 out."""
    for rep in range(2):
        got, ref = run(M, N, K, out_dtype, seed=5 + rep)
        if out_dtype:
            assert np.abs(got - ref).max() <= 1e-3 * np.abs(ref).max()
        else:
            # one bf16 rounding (half an ulp: up to 2^-8 relative) of an fp32 sum of K products whose own error grows with K
            rel = np.abs(got - ref) / np.maximum(np.abs(ref), 1.0)
            assert rel.max() <= 2.0 ** -8 + 1e-7 * K


@pytest.mark.parametrize("M,N,K,out_dtype", [(128, 12288, 4096, 0), (128, 4096, 12288, 1), (77, 4096, 4096, 1), (128, 126464, 512, 0), (5, 3000, 1024, 0)])
def test_linear_few_rows(M, N, K, out_dtype):
    """At most 128 rows: the single-CTA tiles (weights streamed through every SM), at the widths of the cached partial steps."""
    got, ref = run(M, N, K, out_dtype, seed=11)
    if out_dtype:
        assert np.abs(got - ref).max() <= 1e-3 * np.abs(ref).max()
    else:
        rel = np.abs(got - ref) / np.maximum(np.abs(ref), 1.0)
        assert rel.max() <= 2.0 ** -8 + 1e-7 * K
