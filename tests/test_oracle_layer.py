"""Pins of the checker's layer functions against what the mathematics fixes (CPU only).

The layer is W = A B (Eq. 3) applied as y = x W^T.  With L = <y, dY> the loss is
linear in each of x, A, B separately, so central differences are exact up to rounding;
that pins every gradient element by element.  A dense restatement through W pins the
forward and the gradients again by a different route, and a full-rank factor pair must
reproduce the dense layer.
"""
import numpy as np
import pytest

from oracle import ab_oracle as orc


def _case(seed, N, m, n, r):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((N, n)), rng.standard_normal((N, m)),
            rng.standard_normal((m, r)), rng.standard_normal((r, n)))


def _loss(x, dY, A, B):
    # independent of oracle.forward: three explicit loops would be slow, einsum is a different routine
    return float(np.einsum("in,rn,mr,im->", x, B, A, dY))


@pytest.mark.parametrize("N,m,n,r", [(3, 4, 5, 2), (5, 3, 7, 3), (1, 1, 1, 1), (6, 8, 4, 4)])
def test_finite_differences(N, m, n, r):
    x, dY, A, B = _case(N * 100 + m, N, m, n, r)
    dX, dA, dB, _ = orc.backward(x, dY, A, B)
    h = 1e-3
    for name, arr, grad in (("x", x, dX), ("A", A, dA), ("B", B, dB)):
        num = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            old = arr[idx]
            arr[idx] = old + h
            lp = _loss(x, dY, A, B)
            arr[idx] = old - h
            lm = _loss(x, dY, A, B)
            arr[idx] = old
            num[idx] = (lp - lm) / (2 * h)
        assert np.allclose(num, grad, rtol=1e-9, atol=1e-9), name


def test_forward_elementwise_brute_force():
    x, _, A, B = _case(7, 4, 5, 6, 3)
    T, y = orc.forward(x, A, B)
    for i in range(4):
        for j in range(5):
            acc = 0.0
            for k in range(3):
                t = sum(x[i, q] * B[k, q] for q in range(6))
                assert abs(T[i, k] - t) < 1e-12
                acc += t * A[j, k]
            assert abs(y[i, j] - acc) < 1e-12


def test_dense_restatement():
    x, dY, A, B = _case(11, 33, 20, 28, 6)
    W = A @ B
    _, y = orc.forward(x, A, B)
    assert np.allclose(y, x @ W.T, rtol=1e-12, atol=1e-12)
    dX, dA, dB, dT = orc.backward(x, dY, A, B)
    dW = dY.T @ x                       # gradient of the dense layer
    assert np.allclose(dX, dY @ W, rtol=1e-12, atol=1e-11)
    assert np.allclose(dA, dW @ B.T, rtol=1e-12, atol=1e-11)
    assert np.allclose(dB, A.T @ dW, rtol=1e-12, atol=1e-11)
    assert dT.shape == (33, 6)


def test_swapped_factor_would_fail():
    # a transposed operand must not slip through: shapes that make A^T B^T also valid
    x, dY, A, B = _case(5, 4, 3, 3, 3)
    _, y = orc.forward(x, A, B)
    wrong = (x @ B) @ A
    assert not np.allclose(y, wrong)


def test_full_rank_factors_reproduce_dense_layer():
    rng = np.random.default_rng(3)
    W = rng.standard_normal((12, 9))
    U, s, Vt = np.linalg.svd(W, full_matrices=False)
    A = U * np.sqrt(s)
    B = np.sqrt(s)[:, None] * Vt
    x = rng.standard_normal((7, 9))
    _, y = orc.forward(x, A, B)
    assert np.allclose(y, x @ W.T, atol=1e-12)


def test_dense_layer_loops_finite_differences_and_factorised_form():
    """The dense layer of the full-rank phases: element-wise loops, central differences of L = <y, dY> (exact
    up to rounding: L is linear in x and in W), and agreement with the factorised layer when W = A B."""
    rng = np.random.default_rng(21)
    N, m, n, r = 5, 4, 6, 3
    x, dY, W = rng.standard_normal((N, n)), rng.standard_normal((N, m)), rng.standard_normal((m, n))
    y = orc.dense_forward(x, W)
    for i in range(N):
        for j in range(m):
            assert np.isclose(y[i, j], sum(x[i, k] * W[j, k] for k in range(n)), rtol=1e-13)
    dX, dW = orc.dense_backward(x, dY, W)
    h = 1e-3

    def loss(xx, ww):
        return float(np.sum(orc.dense_forward(xx, ww) * dY))
    for i in range(N):
        for k in range(n):
            e = np.zeros_like(x); e[i, k] = h
            assert np.isclose((loss(x + e, W) - loss(x - e, W)) / (2 * h), dX[i, k], rtol=1e-9, atol=1e-11)
    for j in range(m):
        for k in range(n):
            e = np.zeros_like(W); e[j, k] = h
            assert np.isclose((loss(x, W + e) - loss(x, W - e)) / (2 * h), dW[j, k], rtol=1e-9, atol=1e-11)
    A, B = rng.standard_normal((m, r)), rng.standard_normal((r, n))
    assert np.allclose(orc.dense_forward(x, A @ B), orc.forward(x, A, B)[1], atol=1e-12)
    dXf, dAf, dBf, _ = orc.backward(x, dY, A, B)
    dXd, dWd = orc.dense_backward(x, dY, A @ B)
    assert np.allclose(dXd, dXf, atol=1e-12)
    assert np.allclose(dWd @ B.T, dAf, atol=1e-12) and np.allclose(A.T @ dWd, dBf, atol=1e-12)


def test_conv3x3_rows_against_direct_convolution_and_adjoint():
    """im2col rows times a flattened weight equal the convolution written as loops; col2im is the exact
    transpose of im2col (<im2col(x), R> = <x, col2im(R)>); the factorised convolution's dX matches central
    differences."""
    rng = np.random.default_rng(31)
    B, H, W, C, m, r = 2, 3, 4, 3, 4, 2
    x = rng.standard_normal((B, H, W, C))
    Wt = rng.standard_normal((m, 3, 3, C))
    y = orc.im2col_3x3(x) @ Wt.reshape(m, 9 * C).T
    for b in range(B):
        for oy in range(H):
            for ox in range(W):
                for o in range(m):
                    acc = 0.0
                    for ky in range(3):
                        for kx in range(3):
                            iy, ix = oy + ky - 1, ox + kx - 1
                            if 0 <= iy < H and 0 <= ix < W:
                                acc += float(np.dot(x[b, iy, ix], Wt[o, ky, kx]))
                    assert np.isclose(y[(b * H + oy) * W + ox, o], acc, rtol=1e-12, atol=1e-13)
    R = rng.standard_normal((B * H * W, 9 * C))
    assert np.isclose(np.sum(orc.im2col_3x3(x) * R), np.sum(x * orc.col2im_3x3(R, B, H, W, C)), rtol=1e-12)
    A, Bf = rng.standard_normal((m, r)), rng.standard_normal((r, 9 * C))
    dY = rng.standard_normal((B * H * W, m))
    dX, dA, dB, _ = orc.conv3x3_backward(x, dY, A, Bf)
    h = 1e-3
    for idx in [(0, 0, 0, 0), (1, 2, 3, 2), (0, 1, 2, 1), (1, 0, 3, 0)]:
        e = np.zeros_like(x); e[idx] = h
        num = (np.sum(orc.conv3x3_forward(x + e, A, Bf)[1] * dY) - np.sum(orc.conv3x3_forward(x - e, A, Bf)[1] * dY)) / (2 * h)
        assert np.isclose(num, dX[idx], rtol=1e-8, atol=1e-10)
