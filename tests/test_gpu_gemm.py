"""The tensor-core dense product on its own (`mixlora_gemm_bf16`) against the plain definition
C = A B^T evaluated in float64 on the same bf16-rounded operands."""
import numpy as np
import pytest

from paper_2404_15159_b200 import synth

pytestmark = pytest.mark.gpu


def run_gemm(M, N, K, b_is_kn, seed=0):
    import torch
    from paper_2404_15159_b200 import binding as B

    rng = np.random.Generator(np.random.Philox(key=synth.BASE_SEED + 500 + seed))
    A = synth.round_to_bf16(rng.standard_normal((M, K), dtype=np.float32))
    Bm = synth.round_to_bf16(rng.standard_normal((K, N) if b_is_kn else (N, K), dtype=np.float32))
    dA = torch.from_numpy(A).cuda().to(torch.bfloat16)
    dB = torch.from_numpy(Bm).cuda().to(torch.bfloat16)
    dC = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.mixlora_gemm_bf16(dA, dB, dC, M, N, K, b_is_kn, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "a bounded wait inside the kernel ran out"
    return A, Bm, dC.float().cpu().numpy()


def check(M, N, K, b_is_kn, seed=0, sample=None):
    A, Bm, C = run_gemm(M, N, K, b_is_kn, seed)
    A64, B64 = A.astype(np.float64), Bm.astype(np.float64)
    if sample is None:
        ref = A64 @ (B64 if b_is_kn else B64.T)
        got = C
    else:
        rng = np.random.default_rng(1)
        rows = np.unique(np.concatenate([rng.integers(0, M, sample), [0, M - 1]]))
        ref = A64[rows] @ (B64 if b_is_kn else B64.T)
        got = C[rows]
    assert np.isfinite(got).all()
    err = np.abs(got - ref).max() / np.abs(ref).max()
    assert err < 6e-3, f"M={M} N={N} K={K} kn={b_is_kn}: relative error {err:.3e}"   # bf16 output rounding is 2^-9


@pytest.mark.parametrize("b_is_kn", [False, True])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (128, 256, 512), (256, 512, 128), (300, 264, 200), (1000, 1376, 520),
                                   (77, 128, 4096), (129, 24, 64), (128, 64, 8), (640, 8, 72)])
def test_gemm_matches_the_float64_product(M, N, K, b_is_kn):
    check(M, N, K, b_is_kn)


@pytest.mark.parametrize("b_is_kn", [False, True])
def test_gemm_large_on_sampled_rows(b_is_kn):
    check(4096, 11008, 4096, b_is_kn, seed=3, sample=64)
