"""Host-side checks that need no GPU: the C-ABI library loads and exports every symbol the
header declares, argument validation, workspace arithmetic, workload shapes."""
import os
import re

import numpy as np
import pytest

from paper_2008_11343_b200 import binding as B
from paper_2008_11343_b200 import build as libbuild
from paper_2008_11343_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return B.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "apms.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(apms_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_functions()
    assert len(names) >= 20
    for name in names:
        assert hasattr(lib, name), f"{name} declared in apms.h but not exported"
        assert name in B.SIGNATURES, f"{name} has no Python binding"
        assert callable(getattr(B, name)), f"binding lacks a function named {name}"
    assert sorted(B.SIGNATURES) == names


def test_workspace_bytes_is_pure_and_covers_the_state(lib):
    d, n, chunk = 335_141_888, 16, 32768
    nbytes = B.apms_workspace_bytes(d, n, chunk)
    C, W = -(-d // chunk), -(-d // 32)
    need = 4 * d * (n + 4 + 2 + 1) + 4 * W * (n + 1) + 4 * C * (n + 1)   # x, v, m, zbar, n z, 2 staging, sqrt(v) + eps
    need += 8 * n * -(-d // 512)                     # one binary64 partial sum per worker and 512 elements
    assert need <= nbytes <= need * 1.001 + (1 << 20)
    assert B.apms_workspace_bytes(d, n, chunk) == nbytes
    for bad in [(0, 1, 32), (1, 0, 32), (1, 65, 32), (1, 1, 31), (1, 1, 0), (1, 1, -32)]:
        assert B.apms_workspace_bytes(*bad) == 0


def test_create_validates_before_touching_the_device(lib):
    with pytest.raises(B.ApmsError) as e:
        B.apms_create(10, 1, 0.9, 0.999, 1e-8, 1e-3, 33)
    assert e.value.status == B.ERR_INVALID_ARG and "multiple of 32" in str(e.value)
    with pytest.raises(B.ApmsError) as e:
        B.apms_create(10, 1, 1.5, 0.999, 1e-8, 1e-3, 32)
    assert e.value.status == B.ERR_INVALID_ARG


def test_no_device_is_an_error_code_not_a_fallback(lib):
    import torch

    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(B.ApmsError) as e:
        B.apms_create(10, 1, 0.9, 0.999, 1e-8, 1e-3, 32)
    assert e.value.status == B.ERR_CUDA
    with pytest.raises(RuntimeError):
        B.Context(10, 1, 0.9, 0.999, 1e-8, 1e-3, 32)


def test_null_context_calls_return_invalid_arg(lib):
    assert lib.apms_freeze_v(None) == B.ERR_INVALID_ARG
    assert lib.apms_set_lr(None, 0.1) == B.ERR_INVALID_ARG
    assert lib.apms_get_phase(None) == B.PHASE_CREATED
    lib.apms_destroy(None)


def test_workload_shapes():
    assert wl.config(0).d == 1 << 20 and wl.config(0).n_chunks == 256
    w1 = wl.config(1)
    assert w1.d == 1 << 24 and len(w1.tensor_sizes) == 64 and w1.n_chunks == 2048
    w2, w3 = wl.config(2), wl.config(3)
    assert w2.d == 109_482_240 and w2.n_chunks == 6683
    assert w3.d == 335_141_888 and w3.n_chunks == 10228
    assert w3.d - (w3.n_chunks - 1) * w3.chunk == 23552            # ragged last chunk
    s = wl.sliced(w3, 5 * 32768 + 100)
    assert s.d == 5 * 32768 + 100


def test_host_gradients_are_seeded_and_shaped():
    w = wl.sliced(wl.config(1), 100_000)
    a, b = wl.host_gradient(w, 3, 1), wl.host_gradient(w, 3, 1)
    assert a.dtype == np.float32 and a.shape == (w.d,) and np.array_equal(a, b)
    assert not np.array_equal(a, wl.host_gradient(w, 3, 2))
    assert not np.array_equal(a, wl.host_gradient(w, 4, 1))
    assert 0.15 < (a == 0).mean() < 0.25                           # 20 % zero entries
    t = wl.host_gradient(wl.sliced(wl.config(3), 200_000), 0, 0)
    assert np.isfinite(t).all() and np.abs(t).max() > 8 * t.std()   # heavy tails (Student-t, nu = 3)
