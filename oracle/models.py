"""Sample losses f(w; xi) and minibatch gradients for the three model kinds.

Test infrastructure (see the package header).  The paper keeps f generic
(Eq. 1); a worker's upload is the mean minibatch gradient of Eq. 2 with U = 1
and its mean local loss (Algorithm 1, last worker line).  The concrete f are
the standard ones:

  LSQ      f = 1/2 (x.w - y)^2                    parameters: w[d]
  SOFTMAX  one affine layer + cross-entropy        parameters: W[in][C], b[C]
  MLP      affine layers with ReLU between them,
           cross-entropy on the soft-max of the last one
  CNN      two convolution + ReLU + max-pool blocks in front of an MLP
           (Sec. V-A; see the CNN section below)

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

LSQ, SOFTMAX, MLP, CNN = 0, 1, 2, 3


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


def net_loss_grad(dims, w, Xb, yb, quant=False, input_delta=False):
    """Mean cross-entropy loss and mean gradient of an affine/ReLU network.

    dims = [in, h1, ..., C]; one layer means soft-max regression.
    yb holds integer class labels.  With input_delta the per-sample gradient with respect to the
    input rows (delta of the first layer times its weights, unrounded, not divided by B) is
    returned as a third value, for models that feed the network from earlier layers.
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
        elif input_delta:
            return loss, grad, delta @ W.T
    return loss, grad


# ---------------------------------------------------------------------------------------------
# CNN: the paper's own model class (Sec. V-A: two convolutional layers and three fully connected
# layers on 32 x 32 x 3 images).  The paper gives no further detail; the reading used here is the
# common small image classifier: each convolution is k x k, stride 1, no padding, followed by ReLU
# and a 2 x 2 max-pool of stride 2; the pooled maps of the second block, flattened in (row,
# column, channel) order, feed affine layers with ReLU between them and soft-max cross-entropy.
#
#   conv = (H, W, C_in, k, C1, C2)       image size, kernel size, channels of the two blocks
#   dims = [F, h1, ..., classes]         the fully connected part; F = C2 * H2 * W2
#   parameters: conv1 W[k][k][C_in][C1], b[C1]; conv2 W[k][k][C1][C2], b[C2]; then the affine
#   layers in the layout of MLP.  Images are stored row-major as [H][W][C_in].
#
# A max-pool window that holds its maximum more than once passes the gradient to the first of
# them in (row, column) order.  With quant=True the stored quantities are rounded to bfloat16:
# the ReLU output of each convolution (the pooled maps are then exact), every delta that is
# stored between two layers, and the points net_loss_grad rounds.

def conv_shapes(conv):
    """(H1, W1, P1h, P1w, H2, W2, P2h, P2w): sizes after conv1, pool1, conv2, pool2."""
    H, W, _, k, _, _ = conv
    H1, W1 = H - k + 1, W - k + 1
    if H1 < 2 or W1 < 2 or H1 % 2 or W1 % 2:
        raise ValueError("first convolution output must be even-sized for the 2 x 2 pool")
    P1h, P1w = H1 // 2, W1 // 2
    H2, W2 = P1h - k + 1, P1w - k + 1
    if H2 < 2 or W2 < 2 or H2 % 2 or W2 % 2:
        raise ValueError("second convolution output must be even-sized for the 2 x 2 pool")
    return H1, W1, P1h, P1w, H2, W2, H2 // 2, W2 // 2


def cnn_n_params(conv, dims):
    _, _, Cin, k, C1, C2 = conv
    return k * k * Cin * C1 + C1 + k * k * C1 * C2 + C2 + n_params(MLP, dims)


def _patches(x, k):
    """x [B, H, W, C] -> [B, H-k+1, W-k+1, k, k, C]: the k x k windows of every output pixel."""
    v = np.lib.stride_tricks.sliding_window_view(x, (k, k), axis=(1, 2))      # [B, Ho, Wo, C, k, k]
    return np.ascontiguousarray(np.transpose(v, (0, 1, 2, 4, 5, 3)))


def _pool_forward(a):
    """2 x 2 max-pool, stride 2.  Returns the pooled maps and, per pooled element, the position
    (0..3 = (dy, dx) row-major) of the first maximum of its window."""
    B, H, W, C = a.shape
    win = a.reshape(B, H // 2, 2, W // 2, 2, C).transpose(0, 1, 3, 5, 2, 4).reshape(B, H // 2, W // 2, C, 4)
    arg = np.argmax(win, axis=-1)                 # first occurrence of the maximum
    return np.take_along_axis(win, arg[..., None], axis=-1)[..., 0], arg


def _pool_backward(dp, arg, H, W):
    """Gradient of the pooled maps routed to the window position that supplied the maximum."""
    B, Ph, Pw, C = dp.shape
    win = np.zeros((B, Ph, Pw, C, 4))
    np.put_along_axis(win, arg[..., None], dp[..., None], axis=-1)
    return win.reshape(B, Ph, Pw, C, 2, 2).transpose(0, 1, 4, 2, 5, 3).reshape(B, H, W, C)


def cnn_loss_grad(conv, dims, w, Xb, yb, quant=False):
    """Mean cross-entropy loss and mean gradient of the CNN over a minibatch.
    Xb [B, H*W*C_in] (rows are images in [H][W][C] order), yb integer labels."""
    q = round_bf16 if quant else (lambda a: a)
    H, W, Cin, k, C1, C2 = conv
    H1, W1, P1h, P1w, H2, W2, P2h, P2w = conv_shapes(conv)
    B = Xb.shape[0]
    n1, n2 = k * k * Cin * C1, k * k * C1 * C2
    Wc1, bc1 = w[:n1].reshape(k, k, Cin, C1), w[n1:n1 + C1]
    o2 = n1 + C1
    Wc2, bc2 = w[o2:o2 + n2].reshape(k, k, C1, C2), w[o2 + n2:o2 + n2 + C2]
    w_fc = w[o2 + n2 + C2:]
    assert dims[0] == P2h * P2w * C2
    x0 = Xb.reshape(B, H, W, Cin)
    # block 1: convolution, ReLU (stored), pool
    pat1 = _patches(x0, k)                                            # [B, H1, W1, k, k, Cin]
    a1 = q(np.maximum(np.tensordot(pat1, Wc1, axes=([3, 4, 5], [0, 1, 2])) + bc1, 0.0))
    p1, arg1 = _pool_forward(a1)
    # block 2
    pat2 = _patches(p1, k)                                            # [B, H2, W2, k, k, C1]
    a2 = q(np.maximum(np.tensordot(pat2, Wc2, axes=([3, 4, 5], [0, 1, 2])) + bc2, 0.0))
    p2, arg2 = _pool_forward(a2)
    feats = p2.reshape(B, -1)                                         # (row, column, channel) order
    # fully connected part; its first layer also back-propagates into the features
    loss, g_fc, d_feat = net_loss_grad(dims, w_fc, feats, yb, quant=quant, input_delta=True)
    # back through block 2: pool routing, ReLU, convolution
    dz2 = _pool_backward(q(d_feat).reshape(B, P2h, P2w, C2), arg2, H2, W2) * (a2 > 0.0)
    gW2 = np.tensordot(pat2, dz2, axes=([0, 1, 2], [0, 1, 2])) / B    # [k, k, C1, C2]
    gb2 = dz2.sum(axis=(0, 1, 2)) / B
    dp1 = np.zeros_like(p1)
    for dy in range(k):                                               # full correlation with the flipped kernel,
        for dx in range(k):                                           # written as a scatter of every tap
            dp1[:, dy:dy + H2, dx:dx + W2, :] += np.tensordot(dz2, Wc2[dy, dx], axes=([3], [1]))
    dz1 = _pool_backward(q(dp1), arg1, H1, W1) * (a1 > 0.0)
    gW1 = np.tensordot(pat1, dz1, axes=([0, 1, 2], [0, 1, 2])) / B
    gb1 = dz1.sum(axis=(0, 1, 2)) / B
    grad = np.concatenate([gW1.reshape(-1), gb1, gW2.reshape(-1), gb2, g_fc])
    return loss, grad


def cnn_sample_loss(conv, dims, w, x, y):
    """f(w; xi) for one image, with plain loops over the output pixels (used by pins)."""
    H, W, Cin, k, C1, C2 = conv
    n1, n2 = k * k * Cin * C1, k * k * C1 * C2
    Wc1, bc1 = w[:n1].reshape(k, k, Cin, C1), w[n1:n1 + C1]
    o2 = n1 + C1
    Wc2, bc2 = w[o2:o2 + n2].reshape(k, k, C1, C2), w[o2 + n2:o2 + n2 + C2]

    def block(img, Wk, bk):
        Hi, Wi, _ = img.shape
        Ho, Wo = Hi - k + 1, Wi - k + 1
        out = np.empty((Ho, Wo, Wk.shape[3]))
        for i in range(Ho):
            for j in range(Wo):
                out[i, j] = np.maximum(np.einsum("abc,abcd->d", img[i:i + k, j:j + k], Wk) + bk, 0.0)
        pooled = np.empty((Ho // 2, Wo // 2, Wk.shape[3]))
        for i in range(Ho // 2):
            for j in range(Wo // 2):
                pooled[i, j] = out[2 * i:2 * i + 2, 2 * j:2 * j + 2].max(axis=(0, 1))
        return pooled

    feats = block(block(x.reshape(H, W, Cin), Wc1, bc1), Wc2, bc2).reshape(-1)
    return sample_loss(MLP, dims, w[o2 + n2 + C2:], feats, y)


def loss_grad(kind, dims, w, Xb, yb, quant=False, conv=None):
    if kind == LSQ:
        return lsq_loss_grad(w, Xb, yb)
    if kind == CNN:
        return cnn_loss_grad(conv, dims, w, Xb, yb, quant=quant)
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
