"""The allocation-free back-projection entry point against the handle-based step.

Some users of this library are not allowed to allocate GPU memory (their process has
handed the whole device to another allocator, or they run where an allocation would
stall the device), so `psgd_backproject_static` keeps its partial sums in a fixed array
inside the library instead of a caller-provided workspace.  This file checks, through
the C ABI, that it returns what `psgd_step` computes for the same inputs: Q_i = M_i^T P~
per node and their mean, twice in a row (the second call finds the first call's
leftovers in the shared array), and that oversized problems are refused.  Because the
two entry points share their kernels, the result is also compared with M_i^T P~ and its
node mean evaluated in double precision on the host.  The shapes include one where the
fixed array, not the GPU's size, limits the number of row chunks, and one with more
than 16 columns (several column chunks per launch).

Collected last on purpose (file name), and independent of every other test.
"""
import numpy as np
import pytest

from conftest import rel_fro

pytestmark = pytest.mark.gpu

TOL = 1e-5  # relative Frobenius error, the tolerance of the other parity tests


def _step_outputs(torch, m, n, r, N, seed):
    """Run one plain PowerSGD step from e = 0 (so M = G) and return (G, P~, Q_i, Q)."""
    from paper_2509_11254_b200 import PowerSGDPlus, synth

    G = torch.as_tensor(synth.make_gradients(2, m, n, N, step=0, seed=seed)[None], device="cuda:0")
    comp = PowerSGDPlus(m, n, r, N, refresh_period=0, seed=seed, device="cuda:0")
    comp.step(G)
    out = (G[0].contiguous(), comp.P_hat[0].clone(), comp.debug("Q_node")[0].clone(), comp.Q[0].clone())
    torch.cuda.synchronize()
    comp.close()
    return out


def test_static_backprojection_matches_step_twice_in_a_row():
    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2509_11254_b200.binding import backproject_static

    # (m, n, r, N, seed).  4096 x 1024, r = 16, N = 16: one row chunk of partial sums is 1 MiB, so the 8 MiB array allows
    # 8 chunks where the GPU alone would get 19; r = 24: two column chunks of 16
    problems = [(1024, 512, 8, 4, 21), (300, 130, 5, 3, 22), (4096, 1024, 16, 16, 23), (640, 256, 24, 2, 24), (1024, 512, 8, 4, 21)]
    prepared = [_step_outputs(torch, *p) for p in problems]
    # back-to-back calls on one stream: each finds the previous call's partial sums in the array
    results = []
    for (G, P_hat, _, _), (m, n, r, N, _) in zip(prepared, problems):
        Qn = torch.full((N, n, r), float("nan"), device="cuda:0")
        Qm = torch.full((n, r), float("nan"), device="cuda:0")
        backproject_static(G, P_hat, Qm, Qn)
        results.append((Qn, Qm))
    torch.cuda.synchronize()
    for (Qn, Qm), (G, P_hat, Qn_ref, Qm_ref) in zip(results, prepared):
        assert rel_fro(Qn.cpu().numpy(), Qn_ref.cpu().numpy()) <= TOL
        assert rel_fro(Qm.cpu().numpy(), Qm_ref.cpu().numpy()) <= TOL
        # the definition, in double on the host: Q_i = M_i^T P~, Q = (1/N) sum_i Q_i
        M64, P64 = G.cpu().numpy().astype(np.float64), P_hat.cpu().numpy().astype(np.float64)
        Q64 = np.stack([M64[i].T @ P64 for i in range(M64.shape[0])])
        assert rel_fro(Qn.cpu().numpy(), Q64) <= TOL
        assert rel_fro(Qm.cpu().numpy(), Q64.mean(axis=0)) <= TOL
    # Q_node is optional
    G, P_hat, _, Qm_ref = prepared[0]
    Qm = torch.empty_like(Qm_ref)
    backproject_static(G, P_hat, Qm, None)
    assert rel_fro(Qm.cpu().numpy(), Qm_ref.cpu().numpy()) <= TOL


def test_static_backprojection_refuses_oversized_problems():
    import ctypes as C

    import torch

    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2509_11254_b200 import binding

    L = binding.lib()
    d = torch.zeros(64, device="cuda:0")
    p = d.data_ptr()
    # N * n * r * 4 = 8 * 4096 * 128 * 4 = 16 MiB > 8 MiB of fixed scratch: refused before any launch
    assert L.psgd_backproject_static(p, p, p, p, 16384, 4096, 128, 8, None) == -6
    assert L.psgd_backproject_static(p, p, p, p, 100, 128, 4, 2, None) == -1      # m < n
    assert L.psgd_backproject_static(None, p, p, p, 256, 128, 4, 2, None) == -2
    torch.cuda.synchronize()
    assert float(d.sum()) == 0.0
