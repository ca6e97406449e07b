"""Pins for the oracle's losses and gradients (Eq. 1, Eq. 2)."""
import numpy as np
import pytest
import torch

from oracle import models


def _fd_grad(f, w, eps=1e-6):
    g = np.zeros_like(w)
    for i in range(w.shape[0]):
        wp, wm = w.copy(), w.copy()
        wp[i] += eps
        wm[i] -= eps
        g[i] = (f(wp) - f(wm)) / (2 * eps)
    return g


def _mean_sample_loss(kind, dims, w, X, y):
    return float(np.mean([models.sample_loss(kind, dims, w, X[b], y[b]) for b in range(len(y))]))


@pytest.mark.parametrize("kind,dims", [
    (models.LSQ, [7, 1]),
    (models.SOFTMAX, [6, 4]),
    (models.MLP, [5, 7, 3]),
    (models.MLP, [4, 6, 5, 3]),
])
def test_gradient_matches_finite_differences(kind, dims):
    rng = np.random.default_rng(11)
    B = 9
    X = rng.standard_normal((B, dims[0]))
    if kind == models.LSQ:
        y = rng.standard_normal(B)
    else:
        y = rng.integers(0, dims[-1], size=B)
    w = rng.standard_normal(models.n_params(kind, dims)) * 0.7
    loss, grad = models.loss_grad(kind, dims, w, X, y)
    # the batched loss is the mean of the unbatched per-sample losses (Eq. 1)
    assert abs(loss - _mean_sample_loss(kind, dims, w, X, y)) < 1e-12 * max(1, abs(loss))
    fd = _fd_grad(lambda v: _mean_sample_loss(kind, dims, v, X, y), w)
    assert np.linalg.norm(grad - fd) <= 1e-6 * max(1.0, np.linalg.norm(fd))


def test_lsq_closed_form():
    rng = np.random.default_rng(2)
    X, y, w = rng.standard_normal((16, 5)), rng.standard_normal(16), rng.standard_normal(5)
    loss, grad = models.lsq_loss_grad(w, X, y)
    assert np.allclose(grad, X.T @ (X @ w - y) / 16, rtol=1e-13, atol=1e-13)
    assert np.isclose(loss, 0.5 * np.sum((X @ w - y) ** 2) / 16, rtol=1e-13)


def test_softmax_gradient_against_autograd():
    """Independent route: torch autograd on cross_entropy (library routine)."""
    rng = np.random.default_rng(4)
    dims = [6, 8, 5]
    B = 10
    X, y = rng.standard_normal((B, 6)), rng.integers(0, 5, size=B)
    w = rng.standard_normal(models.n_params(models.MLP, dims)) * 0.5
    loss, grad = models.net_loss_grad(dims, w, X, y)
    tw = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    W1, b1 = tw[:48].reshape(6, 8), tw[48:56]
    W2, b2 = tw[56:96].reshape(8, 5), tw[96:101]
    h = torch.relu(torch.tensor(X) @ W1 + b1)
    tl = torch.nn.functional.cross_entropy(h @ W2 + b2, torch.tensor(y))
    tl.backward()
    assert abs(float(tl.detach()) - loss) < 1e-12
    assert np.allclose(tw.grad.numpy(), grad, rtol=1e-10, atol=1e-12)


def test_bias_gradient_rows_sum_to_zero():
    # soft-max outputs sum to one, so the last layer's bias gradient sums to zero
    rng = np.random.default_rng(8)
    dims = [5, 4]
    X, y = rng.standard_normal((12, 5)), rng.integers(0, 4, size=12)
    w = rng.standard_normal(models.n_params(models.SOFTMAX, dims))
    _, grad = models.net_loss_grad(dims, w, X, y)
    assert abs(grad[-4:].sum()) < 1e-14


def test_large_logits_do_not_overflow():
    dims = [2, 3]
    w = np.array([800.0, -800.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0])
    X, y = np.array([[1.0, 0.0]]), np.array([1])
    loss, grad = models.net_loss_grad(dims, w, X, y)
    assert np.isfinite(loss) and np.all(np.isfinite(grad))
    assert abs(loss - 1600.0) < 1e-9


def test_round_bf16_matches_library_conversion():
    rng = np.random.default_rng(0)
    a = np.concatenate([rng.standard_normal(5000) * 10.0 ** rng.integers(-20, 20, size=5000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38, 1e-40]])
    ours = models.round_bf16(a)
    ref = torch.tensor(a, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64)
    assert np.array_equal(ours, ref.numpy())
    # ties go to the even neighbour
    assert models.round_bf16(np.array([1.00390625]))[0] == 1.0
    assert models.round_bf16(np.array([1.01171875]))[0] == 1.015625


def test_quantisation_points_by_hand():
    """dims [1,1,2], one sample, every number worked by hand.

    x = 1, W1 = 1 + 2^-8 (a tie, rounds to 1.0 as a stored activation),
    W2 = [0, ln 2-ish chosen representable], labels y = 0.
    """
    w2b = 0.6875                       # bf16-representable
    w = np.array([1.00390625, 0.0, 0.0, w2b, 0.0, 0.0])
    X, y = np.array([[1.0]]), np.array([0])
    dims = [1, 1, 2]
    # exact arithmetic
    _, g_exact = models.net_loss_grad(dims, w, X, y, quant=False)
    p1 = np.exp(w2b * 1.00390625) / (1.0 + np.exp(w2b * 1.00390625))
    assert np.isclose(g_exact[5], p1, rtol=1e-14)                # d/db2[1] = p1
    assert np.isclose(g_exact[3], 1.00390625 * p1, rtol=1e-14)   # dW2[1] = h * p1
    # bf16 storage points
    _, g = models.net_loss_grad(dims, w, X, y, quant=True)
    h = 1.0                                                      # stored activation
    p1q = np.exp(w2b * h) / (1.0 + np.exp(w2b * h))
    d1 = float(models.round_bf16(np.array([p1q]))[0])            # stored delta of class 1
    d0 = -d1                                                     # p0 - 1 = -p1 with two classes
    assert g[4] == d0 and g[5] == d1                             # bias grads are the stored deltas
    assert g[2] == h * d0 and g[3] == h * d1                     # W2 grads use the stored activation
    back = float(models.round_bf16(np.array([d0 * 0.0 + d1 * w2b]))[0])
    assert g[0] == back and g[1] == back                         # hidden delta is stored rounded
    # the values really are different from the exact ones (the test has teeth)
    assert g[3] != g_exact[3] and g[0] != g_exact[0]
    # 2/3 rounds to 171/256
    assert models.round_bf16(np.array([2.0 / 3.0]))[0] == 0.66796875


# ---------------------------------------------------------------- CNN (Sec. V-A: two convolutional + three fully connected layers)
def _cnn_case(seed=0, B=3):
    rng = np.random.default_rng(seed)
    conv = (14, 14, 2, 3, 3, 4)                      # 14x14x2 -> conv3 12x12x3 -> pool 6x6 -> conv3 4x4x4 -> pool 2x2x4
    dims = [16, 7, 6, 5]                             # three fully connected layers
    w = rng.standard_normal(models.cnn_n_params(conv, dims)) * 0.3
    X = rng.standard_normal((B, 14 * 14 * 2))
    y = rng.integers(0, 5, size=B)
    return conv, dims, w, X, y


def test_cnn_gradient_matches_finite_differences_of_the_loop_form():
    """The batched loss/gradient against central differences of the sample loss written with
    plain loops over output pixels (an independent statement of the same network)."""
    conv, dims, w, X, y = _cnn_case()
    loss, g = models.cnn_loss_grad(conv, dims, w, X, y)
    f = lambda v: np.mean([models.cnn_sample_loss(conv, dims, v, X[i], y[i]) for i in range(len(y))])
    assert np.isclose(loss, f(w), rtol=1e-12)
    rng = np.random.default_rng(1)
    eps = 1e-6
    for i in rng.choice(w.shape[0], 60, replace=False):
        wp, wm = w.copy(), w.copy()
        wp[i] += eps
        wm[i] -= eps
        fd = (f(wp) - f(wm)) / (2 * eps)
        assert abs(fd - g[i]) <= 1e-6 * max(1.0, abs(fd)), (i, fd, g[i])


def test_cnn_against_library_convolution_and_autograd():
    """Same network through torch's conv2d / max_pool2d / autograd (library routines, float64):
    parameter layouts [k][k][C_in][C_out] and [H][W][C] images, pooling, flatten order."""
    torch = pytest.importorskip("torch")
    import torch.nn.functional as F
    conv, dims, w, X, y = _cnn_case(seed=3, B=4)
    H, W, Cin, k, C1, C2 = conv
    loss, g = models.cnn_loss_grad(conv, dims, w, X, y)
    wt = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    n1, n2 = k * k * Cin * C1, k * k * C1 * C2
    W1 = wt[:n1].reshape(k, k, Cin, C1).permute(3, 2, 0, 1)          # torch wants [out][in][kh][kw]
    b1 = wt[n1:n1 + C1]
    o2 = n1 + C1
    W2 = wt[o2:o2 + n2].reshape(k, k, C1, C2).permute(3, 2, 0, 1)
    b2 = wt[o2 + n2:o2 + n2 + C2]
    x = torch.tensor(X, dtype=torch.float64).reshape(-1, H, W, Cin).permute(0, 3, 1, 2)
    h = F.max_pool2d(F.relu(F.conv2d(x, W1, b1)), 2)
    h = F.max_pool2d(F.relu(F.conv2d(h, W2, b2)), 2)
    h = h.permute(0, 2, 3, 1).reshape(x.shape[0], -1)                # (row, column, channel) order
    off = o2 + n2 + C2
    for l in range(len(dims) - 1):
        i, o = dims[l], dims[l + 1]
        h = h @ wt[off:off + i * o].reshape(i, o) + wt[off + i * o:off + i * o + o]
        off += i * o + o
        if l < len(dims) - 2:
            h = F.relu(h)
    ref = F.cross_entropy(h, torch.tensor(y, dtype=torch.long))
    ref.backward()
    assert np.isclose(loss, float(ref.detach()), rtol=1e-12)
    assert np.allclose(g, wt.grad.numpy(), rtol=1e-9, atol=1e-12)


def test_cnn_pool_ties_go_to_the_first_maximum():
    """A window whose maximum occurs twice passes the gradient to the first one in (row, column)
    order: one 4x4 single-channel image, k = 1 identity convolutions, worked by hand."""
    a = np.array([[[[1.0], [1.0]], [[0.5], [1.0]]]])                  # one 2x2 window, maximum 1.0 three times
    pooled, arg = models._pool_forward(a)
    assert pooled[0, 0, 0, 0] == 1.0 and arg[0, 0, 0, 0] == 0
    back = models._pool_backward(np.array([[[[7.0]]]]), arg, 2, 2)
    assert back.reshape(-1).tolist() == [7.0, 0.0, 0.0, 0.0]
    a = np.array([[[[0.25], [2.0]], [[2.0], [-1.0]]]])
    pooled, arg = models._pool_forward(a)
    assert pooled[0, 0, 0, 0] == 2.0 and arg[0, 0, 0, 0] == 1        # (row 0, column 1) comes before (1, 0)


def test_cnn_one_by_one_kernels_reduce_to_an_mlp_on_pooled_pixels():
    """k = 1 with identity 1x1 kernels and zero bias makes each block relu + pool of its input, so
    the network is the MLP applied to the twice max-pooled (non-negative part of the) image."""
    rng = np.random.default_rng(5)
    conv = (8, 8, 2, 1, 2, 2)
    dims = [2 * 2 * 2, 6, 5, 3]
    w_fc = rng.standard_normal(models.n_params(models.MLP, dims)) * 0.4
    eye = np.eye(2).reshape(-1)
    w = np.concatenate([eye, np.zeros(2), eye, np.zeros(2), w_fc])
    X = rng.standard_normal((5, 8 * 8 * 2))
    y = rng.integers(0, 3, size=5)
    loss, g = models.cnn_loss_grad(conv, dims, w, X, y)
    img = np.maximum(X.reshape(5, 8, 8, 2), 0.0)
    pooled = img.reshape(5, 2, 4, 2, 4, 2).max(axis=(2, 4))          # 4x4 max-pool = two 2x2 pools
    loss_ref, g_ref = models.net_loss_grad(dims, w_fc, pooled.reshape(5, -1), y)
    assert np.isclose(loss, loss_ref, rtol=1e-13)
    assert np.allclose(g[-w_fc.shape[0]:], g_ref, rtol=1e-12, atol=1e-15)


def test_cnn_quantisation_points():
    """bf16 mode: the stored ReLU outputs of both convolutions are bfloat16 values, and the run
    differs from the exact one."""
    conv, dims, w, X, y = _cnn_case(seed=7)
    Xq = models.round_bf16(X)
    wq = models.round_bf16(w)
    _, g_exact = models.cnn_loss_grad(conv, dims, wq, Xq, y)
    _, g = models.cnn_loss_grad(conv, dims, wq, Xq, y, quant=True)
    assert not np.array_equal(g, g_exact)
    assert np.linalg.norm(g - g_exact) < 0.05 * np.linalg.norm(g_exact)
