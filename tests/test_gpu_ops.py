"""Parity of the stand-alone least-squares gradient operation with the oracle's
minibatch loss/gradient (Eq. 2, U = 1) averaged over the workers (Eq. 3)."""
import numpy as np
import pytest

from oracle import models
from paper_2301_08895_b200 import abs as gpu

pytestmark = pytest.mark.gpu


def _case(n, B, d, M, bf16, seed):
    import torch
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((M, d)).astype(np.float32)
    w = rng.standard_normal(d).astype(np.float32)
    y = rng.standard_normal(M).astype(np.float32)
    idx = rng.integers(0, M, size=(n, B)).astype(np.int32)
    Xd, wd = torch.from_numpy(X).cuda(), torch.from_numpy(w).cuda()
    if bf16:
        Xd, wd = Xd.to(torch.bfloat16), wd.to(torch.bfloat16)
        X, w = Xd.float().cpu().numpy(), wd.float().cpu().numpy()
    return X, y, w, idx, Xd, torch.from_numpy(y).cuda(), wd, torch.from_numpy(idx).cuda()


def oracle_mean_gradient(X, y, w, idx):
    losses, g = [], np.zeros(X.shape[1])
    for i in range(idx.shape[0]):
        loss, grad = models.lsq_loss_grad(w.astype(np.float64), X[idx[i]].astype(np.float64),
                                          y[idx[i]].astype(np.float64))
        losses.append(loss)
        g += grad
    return np.array(losses), g / idx.shape[0]


@pytest.mark.parametrize("n,B,d,bf16", [(1, 1, 1, False), (7, 19, 77, False), (64, 32, 4096, True),
                                        (300, 5, 130, True), (1024, 2, 24, False)])
def test_lsq_gradient_matches_oracle(n, B, d, bf16):
    import torch
    X, y, w, idx, Xd, yd, wd, idxd = _case(n, B, d, 5000, bf16, n + d)
    g = torch.empty(d, device="cuda")
    loss = torch.empty(n, device="cuda")
    scratch = torch.empty(n * d + 3, device="cuda")
    gpu.lsq_gradient(Xd, yd, wd, idxd, g, loss, scratch)
    torch.cuda.synchronize()
    ol, og = oracle_mean_gradient(X, y, w, idx)
    assert np.allclose(loss.cpu().numpy(), ol, rtol=2e-5, atol=1e-6)
    assert np.linalg.norm(g.cpu().numpy() - og) <= 1e-5 * max(np.linalg.norm(og), 1e-30)


def test_lsq_gradient_rejects_bad_arguments():
    import torch
    X, y, w, idx, Xd, yd, wd, idxd = _case(4, 8, 16, 100, False, 1)
    g, loss = torch.empty(16, device="cuda"), torch.empty(4, device="cuda")
    with pytest.raises(gpu.AbsError) as e:
        gpu.lsq_gradient(Xd, yd, wd, idxd, g, loss, torch.empty(63, device="cuda"))
    assert e.value.code == gpu.ENOSPACE
    l = gpu.lib()
    assert l.abs_lsq_gradient(None, yd.data_ptr(), wd.data_ptr(), idxd.data_ptr(), 4, 8, 16, 0,
                              g.data_ptr(), 64, g.data_ptr(), loss.data_ptr(), None) == gpu.EINVAL
    assert l.abs_lsq_gradient(Xd.data_ptr(), yd.data_ptr(), wd.data_ptr(), idxd.data_ptr(), 0, 8, 16, 0,
                              g.data_ptr(), 64, g.data_ptr(), loss.data_ptr(), None) == gpu.EINVAL
