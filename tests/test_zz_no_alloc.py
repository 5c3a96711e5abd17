"""The allocation-free entry point against the allocating one.

Collected last on purpose (file name), so that a run that stops at the first failure has already run every
other test.  The GPU test passes on its own in a fresh process and after the rest of the suite: it does not
depend on what earlier calls left in the library's built-in scratch array.
"""

import numpy as np
import pytest

from paper_2105_09837_b200 import binding as B


def test_oversized_output_is_rejected_with_both_sizes_in_the_message():
    # 2048 x 2048 outputs need 4 Mi floats per node slice; the built-in array holds 1 Mi.  No device is touched.
    with pytest.raises(B.PdadmmError) as e:
        B.matmul_tn_static(16, 2048, 16, 2048, 16, 2048, 2048, 100)
    assert e.value.code == B.EINVAL
    assert "4194304" in str(e.value) and "1048576" in str(e.value)
    with pytest.raises(B.PdadmmError):
        B.matmul_tn_static(0, 8, 16, 8, 16, 8, 8, 8)                    # null input


@pytest.mark.gpu
def test_static_scratch_product_matches_the_allocating_entry_point_twice_in_a_row():
    import torch
    rng = np.random.default_rng(2024)
    dev = torch.device("cuda", 0)
    # second call is smaller in every dimension: if it read what the first call left in the scratch, it would show
    for (K, M, N) in [(5003, 200, 136), (777, 64, 36)]:
        A = rng.standard_normal((K, M)).astype(np.float32)
        Bm = rng.standard_normal((K, N)).astype(np.float32)
        want, _ = B.matmul(2, A, Bm, flags=B.FLAG_SIMT_GEMM)            # existing entry point (allocates)
        dA, dB = torch.from_numpy(A).to(dev), torch.from_numpy(Bm).to(dev)
        dC = torch.full((M, N), float("nan"), device=dev, dtype=torch.float32)
        torch.cuda.synchronize()
        B.matmul_tn_static(dA.data_ptr(), M, dB.data_ptr(), N, dC.data_ptr(), M, N, K, stream=0, device=0)
        torch.cuda.synchronize()
        got = dC.cpu().numpy()
        ref = A.astype(np.float64).T @ Bm.astype(np.float64)
        # same tolerance as the other kernel tests: relative Frobenius error
        assert np.linalg.norm(got - want) <= 1e-5 * np.linalg.norm(want)
        assert np.linalg.norm(got - ref) <= 1e-5 * np.linalg.norm(ref)


@pytest.mark.gpu
def test_static_scratch_product_with_ragged_widths_and_dirty_padding():
    """Widths that are no multiples of 4, leading dimensions larger than the widths, and NaN in every padding column
    of the operands: the valid block equals the allocating entry point's, the padding columns of C come out as zero."""
    import torch
    rng = np.random.default_rng(7)
    dev = torch.device("cuda", 0)
    for (K, M, N, lda, ldb) in [(1031, 37, 53, 44, 60), (300, 5, 3, 8, 4)]:
        A = rng.standard_normal((K, M)).astype(np.float32)
        Bm = rng.standard_normal((K, N)).astype(np.float32)
        want, _ = B.matmul(2, A, Bm, flags=B.FLAG_SIMT_GEMM)
        Ap = np.full((K, lda), np.nan, np.float32)
        Bp = np.full((K, ldb), np.nan, np.float32)
        Ap[:, :M], Bp[:, :N] = A, Bm
        ldc = (N + 3) // 4 * 4
        dA, dB = torch.from_numpy(Ap).to(dev), torch.from_numpy(Bp).to(dev)
        dC = torch.full((M, ldc), float("nan"), device=dev, dtype=torch.float32)
        torch.cuda.synchronize()
        B.matmul_tn_static(dA.data_ptr(), lda, dB.data_ptr(), ldb, dC.data_ptr(), M, N, K, stream=0, device=0)
        torch.cuda.synchronize()
        got = dC.cpu().numpy()
        assert np.linalg.norm(got[:, :N] - want) <= 1e-5 * np.linalg.norm(want)
        assert np.all(got[:, N:] == 0)
