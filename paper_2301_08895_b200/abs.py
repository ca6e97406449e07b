"""ctypes binding of the C-ABI library `libabs_b200.so` (see include/abs_b200.h).

Argument marshalling only: every step of the round loop runs in the library's
CUDA kernels.  PyTorch supplies device memory (workspace, dataset) and the
stream.  There is no CPU fallback: if the library has not been built, or no
CUDA device is present, the calls raise.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libabs_b200.so")

OK, EINVAL, ENOSPACE, EUNSUPPORTED, ESTATE, ECUDA, ETIMEOUT, EDIVERGED, ERANGE, ESTALE = \
    0, -1, -2, -3, -4, -5, -6, -7, -8, -9
LSQ, SOFTMAX, MLP, CNN = 0, 1, 2, 3
FP32, BF16_FP32MASTER = 0, 1
K_ADAPTIVE, K_FIXED = 0, 1
BOUND_ADAPTIVE, BOUND_FIXED, BOUND_OFFSET = 0, 1, 2
RESTART_ALGORITHM1, RESTART_EQ6, RESTART_NONE = 0, 1, 2
T_CONST, T_EXP, T_SHIFTED_EXP, T_PARETO2, T_GAMMA = 0, 1, 2, 3, 4
MAX_LAYERS = 7
FLAG_NO_TENSOR_CORES = 1
FLAG_NO_OVERLAP = 2
FLAG_NO_PERSISTENT = 8
FLAG_NO_BULK_PIPELINE = 32
FLAG_NO_FUSED_BACKWARD = 64
KC_NAMES = ("ctl", "gather", "fwd", "dgrad", "wgrad", "output", "lsq", "update", "rounds", "conv")


class ModelDesc(C.Structure):
    _fields_ = [("kind", C.c_int), ("n_layers", C.c_int), ("dims", C.c_int * (MAX_LAYERS + 1)),
                ("conv", C.c_int * 6), ("batch", C.c_int), ("lr", C.c_float), ("dtype", C.c_int),
                ("local_steps", C.c_int), ("k_mode", C.c_int), ("bound_mode", C.c_int),
                ("bound_offset", C.c_int), ("restart_rule", C.c_int), ("sa_penalty", C.c_int), ("max_rounds", C.c_int), ("flags", C.c_int), ("data_on_host", C.c_int),
                ("X", C.c_void_p), ("y", C.c_void_p), ("n_samples", C.c_longlong),
                ("w0", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("stream", C.c_void_p)]


class TimeDist(C.Structure):
    _fields_ = [("kind", C.c_int), ("shift", C.c_double), ("rate", C.c_double),
                ("scale", C.c_double), ("slow_mod", C.c_int), ("slow_rem", C.c_int),
                ("slow_factor", C.c_double), ("shape", C.c_int)]


class Trace(C.Structure):
    _fields_ = [("K", C.c_void_p), ("n_restart", C.c_void_p), ("theta", C.c_void_p),
                ("T_end", C.c_void_p), ("loss_mean", C.c_void_p), ("comm", C.c_void_p),
                ("sel_off", C.c_void_p), ("rst_off", C.c_void_p), ("sel_id", C.c_void_p),
                ("sel_tau", C.c_void_p), ("sel_loss", C.c_void_p), ("rst_id", C.c_void_p),
                ("cap_sel", C.c_size_t), ("cap_rst", C.c_size_t)]


class AbsError(RuntimeError):
    def __init__(self, code, text):
        super().__init__("abs_b200 error %d: %s" % (code, text))
        self.code = code


_lib = None


def lib():
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("%s is missing: run `python -m paper_2301_08895_b200.build` "
                               "(there is no CPU fallback)" % LIB_PATH)
        l = C.CDLL(LIB_PATH)
        l.abs_last_error.restype = C.c_char_p
        l.abs_workspace_bytes.argtypes = [C.POINTER(ModelDesc), C.c_int, C.c_int,
                                          C.POINTER(C.c_size_t)]
        l.abs_init.argtypes = [C.POINTER(C.c_void_p), C.POINTER(ModelDesc), C.c_int, C.c_int,
                               C.c_int, C.POINTER(TimeDist), C.c_ulonglong]
        l.abs_run_rounds.argtypes = [C.c_void_p, C.c_int]
        l.abs_enqueue_rounds.argtypes = [C.c_void_p, C.c_int]
        l.abs_rounds_done.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
        l.abs_get_params.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]
        l.abs_get_trace.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(Trace)]
        l.abs_state_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
        l.abs_save_state.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]
        l.abs_restore_state.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
        l.abs_launch_count.argtypes = [C.c_void_p, C.POINTER(C.c_longlong)]
        l.abs_lsq_gradient.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                       C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_size_t,
                                       C.c_void_p, C.c_void_p, C.c_void_p]
        l.abs_lsq_gradient_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                               C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p,
                                               C.c_void_p, C.c_void_p]
        l.abs_get_plan.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int),
                                   C.POINTER(C.c_int), C.POINTER(C.c_int)]
        l.abs_profile_start.argtypes = [C.c_void_p, C.c_int]
        l.abs_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_longlong), C.POINTER(C.c_double)]
        l.abs_profile_timeline.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.POINTER(C.c_int)]
        l.abs_selftest_wait_timeout.argtypes = [C.c_void_p, C.c_int]
        l.abs_destroy.argtypes = [C.c_void_p]
        _lib = l
    return _lib


def last_error():
    return lib().abs_last_error().decode()


def _check(rc):
    if rc != OK:
        raise AbsError(rc, last_error())


def n_params(kind, dims, conv=None):
    if kind == LSQ:
        return dims[0]
    n = sum(dims[l] * dims[l + 1] + dims[l + 1] for l in range(len(dims) - 1))
    if kind == CNN:
        _, _, c_in, k, c1, c2 = conv
        n += k * k * c_in * c1 + c1 + k * k * c1 * c2 + c2
    return n


def _desc(kind, dims, batch, lr, dtype, max_rounds, n_samples, k_mode, bound_mode,
          local_steps=1, data_on_host=0, flags=0, bound_offset=0, restart_rule=0, sa_penalty=0, conv=None):
    m = ModelDesc()
    m.kind, m.n_layers = kind, len(dims) - 1
    for i, v in enumerate(dims):
        m.dims[i] = int(v)
    m.batch, m.lr, m.dtype = int(batch), float(lr), dtype
    m.local_steps, m.k_mode, m.bound_mode = local_steps, k_mode, bound_mode
    m.max_rounds, m.data_on_host, m.n_samples = int(max_rounds), data_on_host, int(n_samples)
    m.flags = int(flags)
    m.bound_offset = int(bound_offset)
    m.restart_rule = int(restart_rule)
    m.sa_penalty = int(sa_penalty)
    for i, v in enumerate(conv or ()):
        m.conv[i] = int(v)
    return m


def workspace_bytes(kind, dims, batch, dtype, W, S, max_rounds, n_samples, data_on_host=0,
                    flags=0, local_steps=1):
    m = _desc(kind, dims, batch, 0.0, dtype, max_rounds, n_samples, 0, 0, local_steps, data_on_host, flags)
    out = C.c_size_t(0)
    _check(lib().abs_workspace_bytes(C.byref(m), W, S, C.byref(out)))
    return out.value


class Context:
    """One ABS run (abs_init .. abs_destroy).

    X, y: torch CUDA tensors (X float32 or bfloat16 [n, in]; y float32 or int32),
    or, with `data_on_host=True`, numpy arrays (bf16 as uint16 patterns) that the
    library copies to the device itself.  w0: numpy float32.
    """

    def __init__(self, kind, dims, X, y, w0, batch, lr, W, K0, S, time, seed, max_rounds,
                 dtype=FP32, k_mode=K_ADAPTIVE, bound_mode=BOUND_ADAPTIVE, local_steps=1,
                 data_on_host=False, stream=None, device="cuda:0", flags=0, bound_offset=0,
                 restart_rule=0, sa_penalty=0, conv=None):
        import torch
        self._torch = torch
        self.kind, self.dims, self.W, self.S = kind, list(dims), W, S
        self.conv = None if conv is None else tuple(conv)
        self.max_rounds = max_rounds
        n_samples = X.shape[0]
        m = _desc(kind, dims, batch, lr, dtype, max_rounds, n_samples, k_mode, bound_mode,
                  local_steps, 1 if data_on_host else 0, flags, bound_offset, restart_rule, sa_penalty, conv)
        need = C.c_size_t(0)
        _check(lib().abs_workspace_bytes(C.byref(m), W, S, C.byref(need)))
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.workspace = torch.empty(need.value, dtype=torch.uint8, device=self.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._keep = (X, y)
        if data_on_host:
            X = np.ascontiguousarray(X)
            y = np.ascontiguousarray(y)
            m.X, m.y = X.ctypes.data, y.ctypes.data
            self._keep = (X, y)
        else:
            assert X.is_cuda and y.is_cuda and X.is_contiguous() and y.is_contiguous()
            m.X, m.y = X.data_ptr(), y.data_ptr()
        w0 = np.ascontiguousarray(w0, dtype=np.float32)
        assert w0.shape[0] == n_params(kind, dims, conv)
        m.w0 = w0.ctypes.data
        m.workspace, m.workspace_bytes = self.workspace.data_ptr(), need.value
        m.stream = self.stream.cuda_stream
        td = TimeDist(time.kind, time.shift, time.rate, time.scale, time.slow_mod, time.slow_rem,
                      time.slow_factor, getattr(time, "shape", 1))
        self._ctx = C.c_void_p(None)
        self._desc = m
        _check(lib().abs_init(C.byref(self._ctx), C.byref(m), W, K0, S, C.byref(td),
                              C.c_ulonglong(seed)))

    def run_rounds(self, n):
        _check(lib().abs_run_rounds(self._ctx, n))

    def enqueue_rounds(self, n):
        _check(lib().abs_enqueue_rounds(self._ctx, n))

    def rounds_done(self):
        """(completed rounds, status code) without raising on a device status."""
        r = C.c_int(0)
        rc = lib().abs_rounds_done(self._ctx, C.byref(r))
        return r.value, rc

    def get_params(self):
        d = n_params(self.kind, self.dims, self.conv)
        out = np.empty(d, dtype=np.float32)
        got = C.c_size_t(0)
        _check(lib().abs_get_params(self._ctx, out.ctypes.data, d, C.byref(got)))
        assert got.value == d
        return out

    def save_state(self):
        """Checkpoint of the run between rounds as a uint8 array (abs_save_state)."""
        n = C.c_size_t(0)
        _check(lib().abs_state_bytes(self._ctx, C.byref(n)))
        out = np.empty(n.value, dtype=np.uint8)
        got = C.c_size_t(0)
        _check(lib().abs_save_state(self._ctx, out.ctypes.data, n.value, C.byref(got)))
        assert got.value == n.value
        return out

    def restore_state(self, image):
        """Continue from a checkpoint taken by a context with the same arguments (abs_restore_state)."""
        image = np.ascontiguousarray(image, dtype=np.uint8)
        _check(lib().abs_restore_state(self._ctx, image.ctypes.data, image.size))

    def get_trace(self, first=0, n=None):
        if n is None:
            n = self.rounds_done()[0] - first
        W = self.W
        a = dict(K=np.zeros(n, np.int32), n_restart=np.zeros(n, np.int32),
                 theta=np.zeros(n, np.int32), T_end=np.zeros(n, np.uint64),
                 loss_mean=np.zeros(n, np.float32), comm=np.zeros(n, np.uint64),
                 sel_off=np.zeros(n + 1, np.int64), rst_off=np.zeros(n + 1, np.int64),
                 sel_id=np.zeros(n * W, np.int32), sel_tau=np.zeros(n * W, np.int32),
                 sel_loss=np.zeros(n * W, np.float32), rst_id=np.zeros(n * W, np.int32))
        t = Trace()
        for k, v in a.items():
            setattr(t, k, v.ctypes.data)
        t.cap_sel = t.cap_rst = n * W
        _check(lib().abs_get_trace(self._ctx, first, n, C.byref(t)))
        ns, nr = int(a["sel_off"][n]), int(a["rst_off"][n])
        for k in ("sel_id", "sel_tau", "sel_loss"):
            a[k] = a[k][:ns]
        a["rst_id"] = a["rst_id"][:nr]
        return a

    def launch_count(self):
        v = C.c_longlong(0)
        _check(lib().abs_launch_count(self._ctx, C.byref(v)))
        return v.value

    def plan(self):
        """dict(partials, row_block, rows_cap, path) describing how the context runs."""
        P, rb, rc = C.c_int(0), C.c_int(0), C.c_int(0)
        path = (C.c_int * MAX_LAYERS)()
        _check(lib().abs_get_plan(self._ctx, C.byref(P), C.byref(rb), C.byref(rc), path))
        return dict(partials=P.value, row_block=rb.value, rows_cap=rc.value,
                    path=[path[i] for i in range(len(self.dims) - 1)])

    def profile_start(self, max_launches):
        _check(lib().abs_profile_start(self._ctx, int(max_launches)))

    def profile_read(self):
        """{class name: (launches, total ms)} of the launches recorded since profile_start."""
        n = (C.c_longlong * len(KC_NAMES))()
        ms = (C.c_double * len(KC_NAMES))()
        _check(lib().abs_profile_read(self._ctx, n, ms))
        return {KC_NAMES[i]: (int(n[i]), float(ms[i])) for i in range(len(KC_NAMES))}

    def profile_timeline(self, cap=4096):
        """[(class name, start ms, end ms)] of the launches recorded since profile_start (call
        before profile_read)."""
        cls = np.zeros(cap, np.int32)
        t0 = np.zeros(cap, np.float32)
        t1 = np.zeros(cap, np.float32)
        n = C.c_int(0)
        _check(lib().abs_profile_timeline(self._ctx, cap, cls.ctypes.data, t0.ctypes.data,
                                          t1.ctypes.data, C.byref(n)))
        return [(KC_NAMES[cls[i]], float(t0[i]), float(t1[i])) for i in range(n.value)]

    def selftest_wait_timeout(self, limit_us=1000):
        """abs_selftest_wait_timeout: lets a bounded device wait run out; raises AbsError(ETIMEOUT)."""
        _check(lib().abs_selftest_wait_timeout(self._ctx, int(limit_us)))

    def close(self):
        if self._ctx:
            lib().abs_destroy(self._ctx)
            self._ctx = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def lsq_gradient(X, y, w, idx, g_out, loss_out, scratch, stream=None):
    """abs_lsq_gradient on torch CUDA tensors: X [M, d] and w [d] float32 or bfloat16, y float32,
    idx int32 [n, B], g_out float32 [d], loss_out float32 [n], scratch float32 (>= n*d)."""
    import torch
    n, B = idx.shape
    d = X.shape[1]
    dtype = BF16_FP32MASTER if X.dtype == torch.bfloat16 else FP32
    s = stream if stream is not None else torch.cuda.current_stream(X.device)
    _check(lib().abs_lsq_gradient(X.data_ptr(), y.data_ptr(), w.data_ptr(), idx.data_ptr(), n, B, d,
                                  dtype, scratch.data_ptr(), scratch.numel(), g_out.data_ptr(),
                                  loss_out.data_ptr(), s.cuda_stream))


def lsq_gradient_noalloc(X, y, w, idx, g_out, loss_out, stream=None):
    """abs_lsq_gradient_noalloc: same operation as `lsq_gradient`, for callers that may not
    allocate device memory; partial sums use the library's built-in 4 MiB array, so n*d must be
    at most 1048576.  Calls sharing a device must not overlap on the GPU."""
    import torch
    n, B = idx.shape
    d = X.shape[1]
    dtype = BF16_FP32MASTER if X.dtype == torch.bfloat16 else FP32
    s = stream if stream is not None else torch.cuda.current_stream(X.device)
    _check(lib().abs_lsq_gradient_noalloc(X.data_ptr(), y.data_ptr(), w.data_ptr(), idx.data_ptr(),
                                          n, B, d, dtype, g_out.data_ptr(), loss_out.data_ptr(),
                                          s.cuda_stream))


def trace_rows(tr):
    """Trace arrays -> list of per-round dicts (K, sel, tau, restart, T_end, theta, ...)."""
    rows = []
    for i in range(len(tr["K"])):
        s0, s1 = int(tr["sel_off"][i]), int(tr["sel_off"][i + 1])
        r0, r1 = int(tr["rst_off"][i]), int(tr["rst_off"][i + 1])
        rows.append(dict(K=int(tr["K"][i]), sel=[int(x) for x in tr["sel_id"][s0:s1]],
                         tau=[int(x) for x in tr["sel_tau"][s0:s1]],
                         restart=[int(x) for x in tr["rst_id"][r0:r1]],
                         T_end=int(tr["T_end"][i]), theta=int(tr["theta"][i]),
                         loss_mean=float(tr["loss_mean"][i]), comm=int(tr["comm"][i]),
                         sel_loss=[float(x) for x in tr["sel_loss"][s0:s1]]))
    return rows


def context_from_config(cfg, X, y, w0, max_rounds=None, **kw):
    """Context for an `inputs.Config`; X, y as produced by `inputs.make_data` moved to the
    device by the caller (or numpy with data_on_host=True)."""
    return Context(cfg.kind, cfg.dims, X, y, w0, cfg.batch, cfg.lr, cfg.W, cfg.K0, cfg.S, cfg.time,
                   cfg.run_seed, max_rounds or cfg.rounds, dtype=cfg.dtype, conv=getattr(cfg, "conv", None), **kw)
