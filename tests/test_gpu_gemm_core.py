"""tcgen05 GEMM core against an fp64 matmul of the same bf16 bits, all four operand-major combinations."""
import numpy as np
import pytest
import torch

from paper_2603_06626_b200 import synth
from tests.gpu_util import bits_to_bf16

pytestmark = pytest.mark.gpu

SHAPES = [(128, 256, 64), (128, 256, 256), (256, 512, 320), (200, 264, 136), (1024, 2304, 512), (8, 8, 8)]


@pytest.mark.parametrize("a_mn", [False, True])
@pytest.mark.parametrize("b_mn", [False, True])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_dense_gemm(M, N, K, a_mn, b_mn):
    from paper_2603_06626_b200 import binding
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    A = synth.f32_to_bf16_bits(rng.standard_normal((M, K), dtype=np.float32))
    B = synth.f32_to_bf16_bits(rng.standard_normal((N, K), dtype=np.float32))
    ref = synth.bf16_bits_to_f64(A) @ synth.bf16_bits_to_f64(B).T
    A_dev = bits_to_bf16(A.T.copy() if a_mn else A)
    B_dev = bits_to_bf16(B.T.copy() if b_mn else B)
    C = binding.dense_gemm(A_dev, a_mn, B_dev, b_mn, M, N, K).cpu().numpy().astype(np.float64)
    err = np.linalg.norm(C - ref) / np.linalg.norm(ref)
    assert err < 2e-6, f"rel Frobenius {err}"
    assert np.abs(C - ref).max() < 1e-3 * max(1.0, np.abs(ref).max())
