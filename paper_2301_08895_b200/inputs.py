"""Seeded synthetic inputs and the five benchmark configurations.

This module only *generates data and names hyper-parameters*; it contains no
step of the ABS method.  The same arrays are handed to the GPU library and to
whatever checks it.  Shapes follow the paper's experimental setting (Sec. V-A:
image-sized inputs, ten classes, tens of thousands of samples, B = 32..128,
N = 8..1024 workers); the data themselves are random draws, not dataset items.

Generators use numpy `Generator(PCG64(seed))`; large matrices are produced in
row chunks with one child stream per chunk so the result does not depend on
the number of threads used.
"""
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace

import numpy as np

LSQ, SOFTMAX, MLP, CNN = 0, 1, 2, 3
FP32, BF16 = 0, 1
T_CONST, T_EXP, T_SHIFTED_EXP, T_PARETO2, T_GAMMA = 0, 1, 2, 3, 4


@dataclass
class TimeSpec:
    kind: int
    shift: float = 0.0
    rate: float = 1.0
    scale: float = 1.0
    slow_mod: int = 0
    slow_rem: int = 0
    slow_factor: float = 1.0
    shape: int = 1            # T_GAMMA: integer shape


@dataclass
class Config:
    name: str
    kind: int
    dims: tuple
    dtype: int
    W: int
    batch: int
    K0: int
    S: int
    rounds: int
    lr: float
    n_samples: int
    time: TimeSpec
    data: str                 # "lsq" | "mixture"
    sigma: float = 1.0        # mixture spread
    clip: bool = False        # clip mixture features to [0, 1]
    noise: float = 0.1        # lsq label noise
    w0: str = "zeros"         # "zeros" | "he"
    data_seed: int = 0
    run_seed: int = 0
    w0_seed: int = 0
    conv: tuple = None        # CNN: (H, W, C_in, k, C1, C2); dims then describes the fully connected part

    @property
    def x_len(self):
        """Elements of one dataset row."""
        return self.conv[0] * self.conv[1] * self.conv[2] if self.kind == CNN else self.dims[0]

    def scaled(self, **kw):
        return replace(self, **kw)


def config(i, W=None):
    """Configuration i = 1..5 of the benchmark (5 takes W in {256, 512, 1024}); 6 is the paper's own
    model class on image-shaped synthetic data (Sec. V-A: 32 x 32 x 3 inputs, two convolution
    blocks and three fully connected layers, B = 32, N = 20, K^0 = 5, gamma-distributed execution
    times; the step size is 0.003 instead of the paper's 0.1 because the synthetic features are
    not normalised)."""
    if i == 1:
        c = Config("lsq64_w8", LSQ, (64, 1), FP32, 8, 32, 2, 4, 200, 0.05, 8192,
                   TimeSpec(T_SHIFTED_EXP, shift=1.0, rate=1.0), "lsq")
    elif i == 2:
        c = Config("softmax784_w16", SOFTMAX, (784, 10), FP32, 16, 64, 4, 8, 1000, 0.1, 60000,
                   TimeSpec(T_EXP, rate=1.0), "mixture", sigma=2.0, clip=True)
    elif i == 3:
        c = Config("mlp784_256_w64", MLP, (784, 256, 10), BF16, 64, 128, 8, 8, 2000, 0.1, 60000,
                   TimeSpec(T_SHIFTED_EXP, shift=1.0, rate=1.0, slow_mod=10, slow_rem=9,
                            slow_factor=5.0),
                   "mixture", sigma=2.0, clip=True, w0="he")
    elif i == 4:
        c = Config("mlp3072_1024_512_w128", MLP, (3072, 1024, 512, 10), BF16, 128, 64, 16, 16,
                   2000, 0.01, 50000, TimeSpec(T_PARETO2, scale=1.0), "mixture", sigma=1.0,
                   w0="he")
    elif i == 5:
        W = 256 if W is None else W
        c = Config("lsq4096_w%d" % W, LSQ, (4096, 1), BF16, W, 32, W // 8, 32, 500, 0.01,
                   1_000_000, TimeSpec(T_EXP, rate=1.0), "lsq")
    elif i == 6:
        c = Config("cnn32_w20", CNN, (400, 120, 84, 10), BF16, 20, 32, 5, 8, 500, 0.003, 50000,
                   TimeSpec(T_GAMMA, shift=0.0, rate=3.0, shape=3), "mixture", sigma=1.0, w0="he",
                   conv=(32, 32, 3, 5, 6, 16))
    else:
        raise ValueError("config index 1..6")
    c.data_seed, c.run_seed, c.w0_seed = 1000 + i, 2000 + i, 3000 + i
    return c


def n_params(kind, dims, conv=None):
    if kind == LSQ:
        return dims[0]
    n = sum(dims[l] * dims[l + 1] + dims[l + 1] for l in range(len(dims) - 1))
    if kind == CNN:
        _, _, c_in, k, c1, c2 = conv
        n += k * k * c_in * c1 + c1 + k * k * c1 * c2 + c2
    return n


def to_bf16_bits(a32):
    """float32 array -> uint16 bfloat16 patterns (round to nearest even; finite inputs)."""
    bits = np.ascontiguousarray(a32, dtype=np.float32).view(np.uint32)
    return ((bits + np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits):
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


_CHUNK_ROWS = 8192


def _chunked(n_rows, seed, fill, out, threads=8):
    """Fill out[r0:r1] for each row chunk from its own child stream."""
    n_chunks = (n_rows + _CHUNK_ROWS - 1) // _CHUNK_ROWS
    children = np.random.SeedSequence(seed).spawn(n_chunks)

    def work(ci):
        r0, r1 = ci * _CHUNK_ROWS, min(n_rows, (ci + 1) * _CHUNK_ROWS)
        fill(np.random.Generator(np.random.PCG64(children[ci])), r0, r1, out)

    if n_chunks == 1:
        work(0)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(n_chunks)))
    return out


def make_data(cfg):
    """Dataset of a configuration.

    Returns (X, y, extra).  X is float32 [n, in] for FP32 configurations and
    uint16 bfloat16 patterns for BF16 ones; y is float32 (least squares) or
    int32 labels; extra carries the generating parameters (w_star or means).
    """
    n, d_in = cfg.n_samples, cfg.x_len
    rng = np.random.Generator(np.random.PCG64(cfg.data_seed))
    bf16 = cfg.dtype == BF16
    X = np.empty((n, d_in), dtype=np.uint16 if bf16 else np.float32)
    if cfg.data == "lsq":
        w_star = rng.standard_normal(d_in).astype(np.float32)
        y = np.empty(n, dtype=np.float32)

        def fill(g, r0, r1, out):
            x = g.standard_normal((r1 - r0, d_in), dtype=np.float32)
            if bf16:
                bits = to_bf16_bits(x)
                out[r0:r1] = bits
                x = bf16_bits_to_f32(bits)
            else:
                out[r0:r1] = x
            eps = g.standard_normal(r1 - r0).astype(np.float32) * np.float32(cfg.noise)
            y[r0:r1] = (x.astype(np.float64) @ w_star.astype(np.float64)).astype(np.float32) + eps

        _chunked(n, cfg.data_seed + 1, fill, X)
        return X, y, {"w_star": w_star}
    n_cls = cfg.dims[-1]
    means = rng.standard_normal((n_cls, d_in)).astype(np.float32)
    y = np.empty(n, dtype=np.int32)

    def fill(g, r0, r1, out):
        lab = g.integers(0, n_cls, size=r1 - r0, dtype=np.int32)
        x = means[lab] + np.float32(cfg.sigma) * g.standard_normal((r1 - r0, d_in), dtype=np.float32)
        if cfg.clip:
            np.clip(x, 0.0, 1.0, out=x)
        out[r0:r1] = to_bf16_bits(x) if bf16 else x
        y[r0:r1] = lab

    _chunked(n, cfg.data_seed + 1, fill, X)
    return X, y, {"means": means}


def make_w0(cfg):
    """Initial parameters, float32, layout: per layer W[in][out] then b[out]
    (least squares: w[d]; CNN: the two convolution blocks first)."""
    d = n_params(cfg.kind, cfg.dims, cfg.conv)
    w0 = np.zeros(d, dtype=np.float32)
    if cfg.w0 == "he":
        rng = np.random.Generator(np.random.PCG64(cfg.w0_seed))
        off = 0
        if cfg.kind == CNN:            # convolution blocks: W[k][k][C_in][C_out] with fan-in k k C_in, then b = 0
            _, _, c_in, k, c1, c2 = cfg.conv
            for ci, co in ((c_in, c1), (c1, c2)):
                n_w = k * k * ci * co
                w0[off:off + n_w] = rng.standard_normal(n_w).astype(np.float32) * np.float32(
                    np.sqrt(2.0 / (k * k * ci)))
                off += n_w + co
        for l in range(len(cfg.dims) - 1):
            i, o = cfg.dims[l], cfg.dims[l + 1]
            w0[off:off + i * o] = rng.standard_normal(i * o).astype(np.float32) * np.float32(
                np.sqrt(2.0 / i))
            off += i * o + o
    return w0
