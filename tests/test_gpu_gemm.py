"""The tensor-core contraction primitive against a float64 product of the decoded operands, for
every combination of operand storage (K-major / MN-major), FP8 and bf16, ragged sizes."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import fp8
from paper_2609_39813_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39813_b200 import binding
    binding.lib()
    return binding


def _operand(rng, rows, K, elem, fmt, mn):
    """Returns (values float64 [rows, K], device tensor in the requested storage, pitch)."""
    from paper_2609_39813_b200.harness import up
    if elem == 1:
        codes = rng.integers(0, 0x78 if fmt == fp8.E4M3 else 0x78, size=(rows, K), dtype=np.uint8)
        codes |= (rng.integers(0, 2, size=(rows, K), dtype=np.uint8) << 7)
        vals = fp8.decode(codes, fmt)
        host = codes
    else:
        vals32 = workloads.to_bf16_grid(rng.standard_normal((rows, K)).astype(np.float32))
        vals = vals32.astype(np.float64)
        host = vals32
    mat = host.T if mn else host                      # stored [K][rows] when MN-major
    r, c = mat.shape
    pitch = (c * elem + 15) // 16 * 16 // elem        # pad the pitch to 16 bytes
    buf = np.zeros((r, pitch), dtype=host.dtype)
    buf[:, :c] = mat
    dev = torch.from_numpy(buf).cuda() if elem == 1 else up(buf, "bf16")
    return vals, dev, pitch


@pytest.mark.parametrize("elem", [1, 2])
@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (1, 0), (0, 1), (1, 1)])
# the last shape has ten tile columns: the tile walk takes them as a band of eight and a band of two
@pytest.mark.parametrize("M,N,K", [(128, 256, 128), (200, 144, 328), (64, 520, 1000), (260, 1160, 96)])
def test_gemm_operand_majors(b, elem, a_mn, b_mn, M, N, K):
    rng = np.random.default_rng(M + 7 * N + 13 * K + elem)
    a_fmt, b_fmt = fp8.E5M2, fp8.E4M3
    A, dA, lda = _operand(rng, M, K, elem, a_fmt, a_mn)
    B, dB, ldb = _operand(rng, N, K, elem, b_fmt, b_mn)
    ldc = (N + 3) // 4 * 4
    C = torch.full((M, ldc), float("nan"), device="cuda")
    diag = b.new_diag()
    b.bsp_gemm(M, N, K, elem, dA, lda, a_mn, a_fmt, dB, ldb, b_mn, b_fmt, 1.0, C, ldc, diag)
    assert b.read_diag(diag)["status"] == 0
    got = C.cpu().numpy()[:, :N].astype(np.float64)
    want = A @ B.T
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert rel <= 2e-3, rel
    assert rel <= 1e-5      # products of FP8 / bf16 values are exact in FP32: only the summation order differs
