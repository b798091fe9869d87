"""Host-only checks of the C ABI: the library loads, exports every symbol the header
declares, and validates arguments without touching a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2509_11254_b200 import build, binding

    build.build_library()
    return binding.lib()


def test_every_declared_symbol_is_exported(L):
    from paper_2509_11254_b200 import binding

    header = open(os.path.join(ROOT, "include", "psgd.h")).read()
    declared = set(re.findall(r"\b(psgd_[a-z0-9_]+)\s*\(", header))
    declared -= {"psgd_status", "psgd_handle", "psgd_stream"}
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} declared in psgd.h but not exported"
    assert declared == set(binding.SIGNATURES), "binding and header disagree"


def test_create_validates_arguments(L):
    h = C.c_void_p()
    ok = [(256, 128, 4, 4, 1, 5), (8, 8, 8, 1, 1, 0), (16384, 4096, 128, 4, 1, 100)]
    for m, n, r, N, cnt, tau in ok:
        assert L.psgd_create_batch(m, n, r, N, cnt, tau, 1, C.byref(h)) == 0
        assert L.psgd_destroy(h) == 0
    bad = [(100, 128, 4, 4, 1, 5),   # m < n
           (256, 128, 0, 4, 1, 5),   # r < 1
           (256, 128, 129, 4, 1, 5), # r > n
           (512, 512, 200, 4, 1, 5), # r > 128
           (256, 128, 4, 0, 1, 5),   # N < 1
           (256, 128, 4, 4, 0, 5),   # count < 1
           (256, 128, 4, 4, 1, -1)]  # negative period
    for m, n, r, N, cnt, tau in bad:
        assert L.psgd_create_batch(m, n, r, N, cnt, tau, 1, C.byref(h)) == -1
    assert L.psgd_create(256, 128, 4, 4, 5, 1, None) == -2


def test_sizes_and_unattached_calls(L):
    h = C.c_void_p()
    assert L.psgd_create_batch(2048, 768, 8, 8, 36, 50, 1, C.byref(h)) == 0
    e, q, w = C.c_size_t(), C.c_size_t(), C.c_size_t()
    assert L.psgd_sizes(h, C.byref(e), C.byref(q), C.byref(w)) == 0
    assert e.value == 36 * 8 * 2048 * 768 * 4
    assert q.value == 36 * 768 * 8 * 4
    assert w.value > 36 * 8 * 2048 * 8 * 4 and w.value % 256 == 0
    # nothing attached: every stream-ordered call refuses, nothing is launched
    assert L.psgd_step(h, None, None, None, None) == -3
    assert L.psgd_reset(h, None) == -3
    flags = C.c_int()
    assert L.psgd_last_status(h, None, C.byref(flags)) == -3
    assert L.psgd_attach(h, None, None, None, 0) == -2
    assert L.psgd_attach(h, 256, 512, 1024, 16) == -3          # workspace too small
    assert L.psgd_attach(h, 256, 512 + 4, 1024, w.value) == -1  # misaligned
    t = C.c_int64(-1)
    assert L.psgd_get_step(h, C.byref(t)) == 0 and t.value == 0
    assert L.psgd_set_step(h, 7) == 0 and L.psgd_get_step(h, C.byref(t)) == 0 and t.value == 7
    assert L.psgd_set_step(h, -1) == -1
    assert L.psgd_set_option(h, 1, 1) == 0 and L.psgd_set_option(h, 1, 2) == -1
    assert L.psgd_set_option(h, 99, 0) == -1
    n = C.c_int64(-1)
    assert L.psgd_launch_count(h, C.byref(n)) == 0 and n.value == 0
    assert L.psgd_last_cuda_error(h) == b"no error"
    assert L.psgd_destroy(h) == 0
    assert L.psgd_destroy(None) == -2


def test_binding_refuses_cpu_device():
    from paper_2509_11254_b200 import PowerSGDPlus, PSGDError

    with pytest.raises(PSGDError):
        PowerSGDPlus(64, 32, 2, 2, device="cpu")


def test_generators_are_deterministic_and_shaped():
    import numpy as np

    from paper_2509_11254_b200 import synth

    a = synth.make_gradients(2, 96, 64, 3, step=4, matrix_id=2)
    b = synth.make_gradients(2, 96, 64, 3, step=4, matrix_id=2)
    c = synth.make_gradients(2, 96, 64, 3, step=5, matrix_id=2)
    assert a.dtype == np.float32 and a.shape == (3, 96, 64)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    # workload 2: shared low-rank term, noise at 10 % of its Frobenius norm
    U, s, V = synth.low_rank_factors(2, 96, 64, 2)
    Lr = (U * s) @ V.T
    for i in range(3):
        assert np.linalg.norm(a[i] - Lr) == pytest.approx(0.1 * np.linalg.norm(Lr), rel=1e-4)
    np.testing.assert_allclose(s[:3], [1.0, 2 ** -1.5, 3 ** -1.5])
    # workload 3: node-specific leading subspace
    h = synth.make_gradients(3, 96, 64, 2, step=0)
    assert np.linalg.norm(h[0] - h[1]) > 0.5
    assert sum(cnt for _, _, cnt in synth.STACKS[2]) == 84 and sum(cnt for _, _, cnt in synth.STACKS[4]) == 168
