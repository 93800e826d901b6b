"""The tensor-core GEMM building block (tcgen05 / TMEM / TMA) against an exact float64 product of the same
bf16 operands, for both operand majors, full tiles, ragged edges and a K tail."""
import numpy as np
import pytest
import torch

from paper_2003_03477_b200 import binding as ss
from parity import assert_close

pytestmark = pytest.mark.gpu


def _operand(rng, rows, k, mn_major, ld_pad):
    """A logical [rows, k] bf16 matrix stored k-contiguous ([rows, ld]) or rows-contiguous ([k, ld])."""
    vals = torch.from_numpy(rng.normal(size=(rows, k)).astype(np.float32)).to(torch.bfloat16)
    if mn_major:
        ld = rows + ld_pad
        buf = torch.zeros(k, ld, dtype=torch.bfloat16)
        buf[:, :rows] = vals.T
    else:
        ld = k + ld_pad
        buf = torch.zeros(rows, ld, dtype=torch.bfloat16)
        buf[:, :k] = vals
    return vals.double().numpy(), buf.cuda(), ld


SHAPES = [(128, 128, 64), (256, 256, 320), (200, 72, 104), (328, 512, 1728), (512, 1728, 2048), (64, 64, 16),
          (1000, 8, 24),
          (2400, 4000, 520),     # enough tiles for the 128 x 256 variant: ragged last tile in M, N and K
          (19 * 128, 2048, 1024)]  # enough 128 x 128 tiles for the deep (6-stage) ring


@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 0), (1, 1)])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_tensor_core_gemm_matches_exact_product(M, N, K, a_mn, b_mn):
    rng = np.random.default_rng(M * 7 + N * 3 + K + a_mn * 2 + b_mn)
    # MN-major operands need M (or N) to be a multiple of 8 for a 16-byte row pitch: pad the pitch instead
    a, da, lda = _operand(rng, M, K, a_mn, 8 if a_mn == 0 else (8 - M % 8) % 8 + 8)
    b, db, ldb = _operand(rng, N, K, b_mn, 16 if b_mn == 0 else (8 - N % 8) % 8)
    c = torch.full((M, N + 4), -3.0, device="cuda")
    ss.ss_gemm_bf16(da, a_mn, lda, db, b_mn, ldb, c, N + 4, M, N, K)
    torch.cuda.synchronize()
    assert ss.ss_device_error() == 0
    want = a @ b.T
    got = c.cpu().numpy()
    assert_close(got[:, :N], want, 2e-5, f"gemm {M}x{N}x{K} majors {a_mn}{b_mn}")
    assert (got[:, N:] == -3.0).all()          # nothing written outside the N columns
    # the SIMT kernel computes the same product
    c2 = torch.zeros(M, N + 4, device="cuda")
    ss.ss_gemm_bf16(da, a_mn, lda, db, b_mn, ldb, c2, N + 4, M, N, K, force_simt=1)
    torch.cuda.synchronize()
    assert_close(c2.cpu().numpy()[:, :N], want, 2e-5, "simt gemm")


def test_gemm_rejects_unaligned_operands():
    a = torch.zeros(64, 70, dtype=torch.bfloat16, device="cuda")
    b = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    c = torch.zeros(64, 64, device="cuda")
    with pytest.raises(ss.SsError) as e:
        ss.ss_gemm_bf16(a, 0, 70, b, 0, 64, c, 64, 64, 64, 64)     # pitch of A not a multiple of 8
    assert e.value.status == -3
