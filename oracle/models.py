"""Sample losses f(w; xi) and minibatch gradients for the three model kinds.

Test infrastructure (see the package header).  The paper keeps f generic
(Eq. 1); a worker's upload is the mean minibatch gradient of Eq. 2 with U = 1
and its mean local loss (Algorithm 1, last worker line).  The concrete f are
the standard ones:

  LSQ      f = 1/2 (x.w - y)^2                    parameters: w[d]
  SOFTMAX  one affine layer + cross-entropy        parameters: W[in][C], b[C]
  MLP      affine layers with ReLU between them,
           cross-entropy on the soft-max of the last one

Parameter vector layout for SOFTMAX/MLP: for each layer in order, W stored
row-major as [in][out], followed by b[out].

All arithmetic is binary64.  With `quant=True` the values are additionally
rounded to bfloat16 (round to nearest even) at the points where the bf16
configurations store 16-bit values: the model copy a worker downloads, every
hidden activation, and every back-propagated delta of an MLP/SOFTMAX model.
The least-squares residual is never rounded.  The caller supplies inputs X
that are already bf16-representable in that mode.
"""
import numpy as np

LSQ, SOFTMAX, MLP = 0, 1, 2


def round_bf16(a):
    """Round binary64/32 values to the nearest bfloat16 (ties to even),
    returned as binary64.  Goes through binary32 first."""
    f = np.ascontiguousarray(np.asarray(a, dtype=np.float64).astype(np.float32))
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    rounded = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    out = rounded.astype(np.uint32).view(np.float32)
    nan = np.isnan(f)
    if np.any(nan):
        out = np.where(nan, f, out)
    return out.astype(np.float64)


def n_params(kind, dims):
    if kind == LSQ:
        return dims[0]
    return sum(dims[l] * dims[l + 1] + dims[l + 1] for l in range(len(dims) - 1))


def split_params(kind, dims, w):
    """Views (W_l, b_l) per layer into the flat parameter vector."""
    layers, off = [], 0
    for l in range(len(dims) - 1):
        i, o = dims[l], dims[l + 1]
        W = w[off:off + i * o].reshape(i, o)
        off += i * o
        b = w[off:off + o]
        off += o
        layers.append((W, b))
    assert off == w.shape[0]
    return layers


def lsq_loss_grad(w, Xb, yb):
    """Mean loss and mean gradient of f = 1/2 (x.w - y)^2 over a minibatch."""
    r = Xb @ w - yb
    loss = 0.5 * np.mean(r * r)
    grad = (Xb.T @ r) / Xb.shape[0]
    return loss, grad


def net_loss_grad(dims, w, Xb, yb, quant=False):
    """Mean cross-entropy loss and mean gradient of an affine/ReLU network.

    dims = [in, h1, ..., C]; one layer means soft-max regression.
    yb holds integer class labels.
    """
    q = round_bf16 if quant else (lambda a: a)
    layers = split_params(MLP, dims, w)
    nl = len(layers)
    B = Xb.shape[0]
    acts = [Xb]
    for l, (W, b) in enumerate(layers):
        z = acts[-1] @ W + b
        if l < nl - 1:
            acts.append(q(np.maximum(z, 0.0)))
    zmax = z.max(axis=1, keepdims=True)
    ez = np.exp(z - zmax)
    sez = ez.sum(axis=1, keepdims=True)
    p = ez / sez
    logp_true = (z - zmax)[np.arange(B), yb] - np.log(sez[:, 0])
    loss = -np.mean(logp_true)
    delta = p.copy()
    delta[np.arange(B), yb] -= 1.0
    delta = q(delta)
    grad = np.empty_like(w)
    off_end = w.shape[0]
    for l in range(nl - 1, -1, -1):
        W, b = layers[l]
        i, o = dims[l], dims[l + 1]
        gb = delta.sum(axis=0) / B
        gW = (acts[l].T @ delta) / B
        grad[off_end - o:off_end] = gb
        grad[off_end - o - i * o:off_end - o] = gW.reshape(-1)
        off_end -= o + i * o
        if l > 0:
            delta = q((delta @ W.T) * (acts[l] > 0.0))
    return loss, grad


def loss_grad(kind, dims, w, Xb, yb, quant=False):
    if kind == LSQ:
        return lsq_loss_grad(w, Xb, yb)
    return net_loss_grad(dims, w, Xb, yb, quant=quant)


def sample_loss(kind, dims, w, x, y):
    """f(w; xi) for one sample, written without any batching (used by pins)."""
    if kind == LSQ:
        return 0.5 * (float(x @ w) - float(y)) ** 2
    h = x
    layers = split_params(MLP, dims, w)
    for l, (W, b) in enumerate(layers):
        z = h @ W + b
        h = np.maximum(z, 0.0) if l < len(layers) - 1 else z
    z = h - h.max()
    return float(np.log(np.exp(z).sum()) - z[int(y)])
