"""The no-allocation variant of the least-squares gradient operation.

Some users of this library run it where device allocation is not an option:
the memory of the GPU is planned ahead and handed out by someone else, or the
call sits on a path that must not hit the implicit synchronisation of an
allocation.  `abs_lsq_gradient_noalloc` keeps its per-worker partial sums in an
array compiled into the library instead of caller scratch.  This file checks,
through the C ABI, that it returns what `abs_lsq_gradient` returns -- twice in
a row, with different shapes, because the built-in array is shared by all calls
and still holds the first call's partial sums when the second one starts.

Collected last on purpose (file name): a failure here cannot hide other tests
from a run that stops at the first failure.
"""
import numpy as np
import pytest

from oracle import models
from paper_2301_08895_b200 import abs as gpu

pytestmark = pytest.mark.gpu


def _inputs(n, B, d, bf16, seed):
    import torch
    g = torch.Generator(device="cpu").manual_seed(seed)
    M = 4096
    X = torch.randn(M, d, generator=g)
    w = torch.randn(d, generator=g)
    y = torch.randn(M, generator=g)
    idx = torch.randint(0, M, (n, B), generator=g, dtype=torch.int32)
    dt = torch.bfloat16 if bf16 else torch.float32
    return X.to(dt).cuda(), y.cuda(), w.to(dt).cuda(), idx.cuda()


def _oracle(X, y, w, idx):
    """Eq. 2 (U = 1) per worker and the mean of the uploads (the sum of Eq. 3 over n), by the oracle."""
    Xh, yh = X.float().cpu().numpy().astype(np.float64), y.cpu().numpy().astype(np.float64)
    wh, ih = w.float().cpu().numpy().astype(np.float64), idx.cpu().numpy()
    losses, g = [], np.zeros(Xh.shape[1])
    for i in range(ih.shape[0]):
        loss, grad = models.lsq_loss_grad(wh, Xh[ih[i]], yh[ih[i]])
        losses.append(loss)
        g += grad
    return g / ih.shape[0], np.array(losses)


def _both(n, B, d, bf16, seed):
    import torch
    X, y, w, idx = _inputs(n, B, d, bf16, seed)
    g_ref, l_ref = torch.empty(d, device="cuda"), torch.empty(n, device="cuda")
    g_new, l_new = torch.full((d,), 7.0, device="cuda"), torch.full((n,), 7.0, device="cuda")
    gpu.lsq_gradient(X, y, w, idx, g_ref, l_ref, torch.empty(n * d, device="cuda"))
    gpu.lsq_gradient_noalloc(X, y, w, idx, g_new, l_new)
    torch.cuda.synchronize()
    g_o, l_o = _oracle(X, y, w, idx)
    return g_ref.cpu().numpy(), l_ref.cpu().numpy(), g_new.cpu().numpy(), l_new.cpu().numpy(), g_o, l_o


def test_noalloc_matches_scratch_variant_on_two_calls_in_a_row():
    # second call is smaller and of another type: stale partial sums of the first call sit right
    # behind (and under) the region it uses
    for n, B, d, bf16, seed in ((200, 32, 4096, True, 1), (37, 19, 301, False, 2)):
        g_ref, l_ref, g_new, l_new, g_o, l_o = _both(n, B, d, bf16, seed)
        assert np.linalg.norm(g_new - g_ref) <= 1e-5 * np.linalg.norm(g_ref)
        assert np.allclose(l_new, l_ref, rtol=1e-5, atol=0.0)
        # and against the oracle itself, not only through the other entry point
        assert np.linalg.norm(g_new - g_o) <= 1e-5 * np.linalg.norm(g_o)
        assert np.allclose(l_new, l_o, rtol=2e-5, atol=1e-6)
        assert np.all(np.isfinite(g_new)) and not np.any(l_new == 7.0)


def test_noalloc_rejects_sizes_beyond_the_built_in_array():
    import torch
    X, y, w, idx = _inputs(1024, 2, 2048, False, 3)          # n*d = 2^21 > 2^20
    g, loss = torch.zeros(2048, device="cuda"), torch.zeros(1024, device="cuda")
    with pytest.raises(gpu.AbsError) as e:
        gpu.lsq_gradient_noalloc(X, y, w, idx, g, loss)
    assert e.value.code == gpu.ENOSPACE and "1048576" in str(e.value)
    torch.cuda.synchronize()
    assert float(g.abs().sum()) == 0.0 and float(loss.abs().sum()) == 0.0   # nothing ran
    # exactly at the limit is accepted
    X, y, w, idx = _inputs(512, 2, 2048, False, 4)
    g_ref, l_ref = torch.empty(2048, device="cuda"), torch.empty(512, device="cuda")
    gpu.lsq_gradient(X, y, w, idx, g_ref, l_ref, torch.empty(512 * 2048, device="cuda"))
    g, loss = torch.empty(2048, device="cuda"), torch.empty(512, device="cuda")
    gpu.lsq_gradient_noalloc(X, y, w, idx, g, loss)
    torch.cuda.synchronize()
    assert torch.allclose(g, g_ref, rtol=1e-5, atol=1e-7) and torch.allclose(loss, l_ref, rtol=1e-5)
