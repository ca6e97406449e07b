"""Host-side checks of the C-ABI library that need no GPU: it loads, exports
every declared symbol, sizes workspaces and rejects bad arguments."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2301_08895_b200 import abs as gpu
from paper_2301_08895_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "abs_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(abs_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_symbols()
    assert {"abs_init", "abs_run_rounds", "abs_get_params", "abs_get_trace"} <= set(names)
    l = gpu.lib()
    for name in names:
        assert getattr(l, name) is not None


def test_struct_sizes_match_header_layout(tmp_path):
    """The ctypes mirrors must have the layout the C compiler gives the header's structs: a small
    C program prints sizes and offsets taken from include/abs_b200.h."""
    import subprocess
    src = tmp_path / "layout.c"
    src.write_text(
        '#include <stdio.h>\n#include <stddef.h>\n#include "abs_b200.h"\n'
        'int main(void) { printf("%zu %zu %zu %zu %zu %zu %zu %zu %zu %zu\\n", sizeof(abs_time_dist), '
        'sizeof(abs_trace), sizeof(abs_model_desc), offsetof(abs_model_desc, X), '
        'offsetof(abs_model_desc, bound_offset), offsetof(abs_model_desc, max_rounds), '
        'offsetof(abs_model_desc, stream), offsetof(abs_time_dist, shape), '
        'offsetof(abs_time_dist, slow_factor), offsetof(abs_model_desc, sa_penalty)); return 0; }\n')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    got = [int(v) for v in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
    assert got == [C.sizeof(gpu.TimeDist), C.sizeof(gpu.Trace), C.sizeof(gpu.ModelDesc),
                   gpu.ModelDesc.X.offset, gpu.ModelDesc.bound_offset.offset,
                   gpu.ModelDesc.max_rounds.offset, gpu.ModelDesc.stream.offset,
                   gpu.TimeDist.shape.offset, gpu.TimeDist.slow_factor.offset, gpu.ModelDesc.sa_penalty.offset]
    assert C.sizeof(gpu.Trace) == 14 * 8


def test_workspace_bytes_grows_with_problem():
    a = gpu.workspace_bytes(gpu.LSQ, [64, 1], 32, gpu.FP32, 8, 4, 200, 8192)
    b = gpu.workspace_bytes(gpu.LSQ, [64, 1], 32, gpu.FP32, 8, 4, 400, 8192)
    c = gpu.workspace_bytes(gpu.MLP, [3072, 1024, 512, 10], 64, gpu.BF16_FP32MASTER, 128, 16, 2000,
                            50000)
    e = gpu.workspace_bytes(gpu.MLP, [3072, 1024, 512, 10], 64, gpu.BF16_FP32MASTER, 128, 16, 2000,
                            50000, data_on_host=1)
    assert 0 < a < b < c < e
    assert e - c >= 50000 * 3072 * 2
    d = 3072 * 1024 + 1024 + 1024 * 512 + 512 + 512 * 10 + 10
    assert c >= 17 * d * 2 + d * 4          # ring of S + 1 bf16 versions + fp32 master
    assert c < 4 << 30
    # local steps on a network: every worker's own copy (bf16) and its fp32 upload
    u = gpu.workspace_bytes(gpu.MLP, [3072, 1024, 512, 10], 64, gpu.BF16_FP32MASTER, 128, 16, 2000,
                            50000, local_steps=10)
    assert u - c >= 128 * d * 2 + (128 - 4) * d * 4 and u < 8 << 30


@pytest.mark.parametrize("kw,code", [
    (dict(W=0), gpu.EINVAL), (dict(W=1025), gpu.EINVAL), (dict(S=-1), gpu.EINVAL),
    (dict(S=256), gpu.EINVAL), (dict(batch=0), gpu.EINVAL), (dict(batch=2000), gpu.EINVAL),
    (dict(kind=9), gpu.EUNSUPPORTED), (dict(dtype=5), gpu.EUNSUPPORTED),
    (dict(dims=[64, 2]), gpu.EINVAL), (dict(max_rounds=0), gpu.EINVAL),
    (dict(n_samples=3), gpu.EINVAL),
])
def test_workspace_bytes_rejects(kw, code):
    args = dict(kind=gpu.LSQ, dims=[64, 1], batch=32, dtype=gpu.FP32, W=8, S=4, max_rounds=10,
                n_samples=8192)
    args.update(kw)
    with pytest.raises(gpu.AbsError) as e:
        gpu.workspace_bytes(**args)
    assert e.value.code == code and str(e.value)


def _init_args():
    m = gpu._desc(gpu.LSQ, [64, 1], 32, 0.05, gpu.FP32, 10, 8192, gpu.K_ADAPTIVE, gpu.BOUND_ADAPTIVE)
    w0 = np.zeros(64, np.float32)
    m.w0 = w0.ctypes.data
    m.X, m.y = 0x1000, 0x1000          # never dereferenced: checks fail first
    m.workspace, m.workspace_bytes = 0x10000, 1 << 30
    td = gpu.TimeDist(gpu.T_EXP, 0.0, 1.0, 1.0, 0, 0, 1.0)
    return m, td, w0


@pytest.mark.parametrize("mutate,code", [
    (lambda m, td: setattr(m, "local_steps", 0), gpu.EINVAL),
    (lambda m, td: setattr(m, "local_steps", 2000), gpu.EINVAL),
    (lambda m, td: (setattr(m, "local_steps", 4), setattr(m, "batch", 1024), m.dims.__setitem__(0, 20000)), gpu.EUNSUPPORTED),
    (lambda m, td: setattr(m, "restart_rule", 3), gpu.EINVAL),
    (lambda m, td: setattr(m, "sa_penalty", 2), gpu.EINVAL),
    (lambda m, td: setattr(m, "workspace", 0), gpu.EINVAL),
    (lambda m, td: setattr(m, "workspace", 0x10010), gpu.EINVAL),
    (lambda m, td: setattr(m, "workspace_bytes", 1024), gpu.ENOSPACE),
    (lambda m, td: setattr(m, "X", 0), gpu.EINVAL),
    (lambda m, td: setattr(m, "lr", float("nan")), gpu.EINVAL),
    (lambda m, td: setattr(td, "rate", 0.0), gpu.EINVAL),
    (lambda m, td: setattr(td, "kind", 7), gpu.EUNSUPPORTED),
    (lambda m, td: setattr(td, "slow_mod", -1), gpu.EINVAL),
    (lambda m, td: setattr(m, "k_mode", 3), gpu.EINVAL),
])
def test_init_rejects_before_touching_the_device(mutate, code):
    m, td, w0 = _init_args()
    mutate(m, td)
    ctx = C.c_void_p(None)
    rc = gpu.lib().abs_init(C.byref(ctx), C.byref(m), 8, 2, 4, C.byref(td), C.c_ulonglong(1))
    assert rc == code and not ctx.value
    assert gpu.last_error()


def test_init_rejects_k0():
    m, td, w0 = _init_args()
    ctx = C.c_void_p(None)
    for k0 in (0, 9):
        assert gpu.lib().abs_init(C.byref(ctx), C.byref(m), 8, k0, 4, C.byref(td),
                                  C.c_ulonglong(1)) == gpu.EINVAL


def test_null_context_calls():
    l = gpu.lib()
    assert l.abs_run_rounds(None, 1) == gpu.EINVAL
    assert l.abs_get_params(None, None, 0, None) == gpu.EINVAL
    assert l.abs_state_bytes(None, None) == gpu.EINVAL
    assert l.abs_save_state(None, None, 0, None) == gpu.EINVAL
    assert l.abs_restore_state(None, None, 0) == gpu.EINVAL
    assert l.abs_destroy(None) == gpu.OK
