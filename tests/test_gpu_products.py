"""The three-product TF32 tensor-core kernel of the subspace solve (Sec. 3.3.1: the SVD behind Eq. 3-5
and 3-6 is taken through products with the Gram matrix) against float64, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2503_10501_b200 import binding as tcb

pytestmark = pytest.mark.gpu


def _check(batch, M, NN, K, seed, scale_rows=False):
    rng = np.random.default_rng(seed)
    A = rng.standard_normal((batch, M, K)).astype(np.float32)
    B = rng.standard_normal((batch, NN, K)).astype(np.float32)
    if scale_rows:
        # columns of very different size, as the panels of the solve have before they are
        # orthonormalised: the error must stay relative to |a| |b|, not to the largest entry
        A *= np.geomspace(1.0, 1e-6, K).astype(np.float32)[None, None, :]
        B *= np.geomspace(1.0, 1e-3, NN).astype(np.float32)[None, :, None]
    C, CT, st = tcb.tc_matmul_f32x3(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(),
                                    transposed=True)
    torch.cuda.synchronize()
    assert int(st.abs().sum()) == 0
    C, CT = C.cpu().numpy(), CT.cpu().numpy()
    A64, B64 = A.astype(np.float64), B.astype(np.float64)
    ref = np.einsum("bmk,bnk->bmn", A64, B64)
    mag = np.einsum("bmk,bnk->bmn", np.abs(A64), np.abs(B64))   # sum_k |a_k| |b_k|
    err = np.abs(C - ref) / np.maximum(mag, 1e-300)
    # 3 x 2^-22 from the split plus the float32 additions of the K / 32 slab sums
    assert err.max() < 1.5e-6, err.max()
    assert np.array_equal(CT, np.swapaxes(C, 1, 2))
    return err.max()


@pytest.mark.parametrize("NN", [128, 144, 160, 192])
def test_product_square_k(NN):
    # the shapes of Y R^{-1} and of the back-transformation: M = N tokens (ragged last tile), K = k
    _check(3, 576, NN, NN, seed=NN)


@pytest.mark.parametrize("M,NN,K", [(576, 144, 576), (144, 144, 576), (200, 160, 580), (64, 128, 36),
                                    (2880, 192, 2880)])
def test_product_shapes(M, NN, K):
    # G Q (M = K = N), Y^T Y (M = NN = k, second row tile nearly empty), ragged M and K tails
    _check(2 if M < 2000 else 1, M, NN, K, seed=M + K)


def test_product_graded_columns():
    _check(2, 576, 144, 576, seed=7, scale_rows=True)


def test_product_rejects_other_widths():
    A = torch.zeros(1, 64, 32, device="cuda")
    B = torch.zeros(1, 136, 32, device="cuda")
    with pytest.raises(tcb.TokenCarveError) as e:
        tcb.tc_matmul_f32x3(A, B)
    assert e.value.status == 2
