"""Pins for the CPU oracle: what the paper and the mathematics fix.

Each check is written against an oracle *module-like object* so that the last
test can re-run the checks on deliberately wrong variants of the oracle (planted
on the CPU) and show that every planted mistake trips at least one pin.
"""
import itertools
import os
import types
from fractions import Fraction

import numpy as np
import pytest

from oracle import psgd_oracle as orc
from paper_2509_11254_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _load_golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            p = line.split()
            vals[p[0]] = np.array([float(x) for x in p[3:]]).reshape(int(p[1]), int(p[2]))
    return vals


# --------------------------------------------------------------------------
# check functions (take the oracle module `o`)
# --------------------------------------------------------------------------
def check_counterexample_t0(o):
    """Appendix A, Claim 1, t = 0: printed closed-form values."""
    gold = _load_golden("counterexample_t0.txt")
    sigma, N = 3.0, 3
    X0 = np.array([[0.3, -0.2], [0.1, 0.7]])
    xi = np.ones((1, N))
    hist, _ = o.run_counterexample(X0, np.array([[0.5], [1.5]]), xi, sigma, tau=0, eta=0.1, mu=0.9)
    h = hist[0]
    for i in range(N):
        np.testing.assert_allclose(h["M"][i], gold["Delta0"], atol=1e-14)
        np.testing.assert_allclose(h["Dhat_i"][i], gold["Dhat0"], atol=1e-13)
        np.testing.assert_allclose(h["E"][i], gold["E1"], atol=1e-13)
    np.testing.assert_allclose(h["P"], gold["P0"], atol=1e-14)
    np.testing.assert_allclose(h["P_hat"], gold["Phat0"], atol=1e-15)
    np.testing.assert_allclose(h["Q"], gold["Q0"], atol=1e-14)
    np.testing.assert_allclose(h["mom"], gold["m0"], atol=1e-13)


def check_counterexample_induction(o):
    """Appendix A, Claim 1, t >= 1 and the conclusion of Theorem 1.

    With xi_0 = +1 on every node and arbitrary later draws (odd N so that the
    node-sum of beta never vanishes): P~_t = +-C, Q_t in span(C), e_{t+1} in
    span(A), the local reconstruction is beta_t^(i) B with beta = +-sigma,
    m_t in span(B), X_t - X_0 in span(B) and ||grad f(X_t)||_F^2 stays at
    4 psi'(a-b-c+d)^2.
    The trap is an unstable equilibrium in floating point: a rounding error along
    D = (1,-1) is multiplied by |sum(lambda+gamma)| / |sum(beta)| every step, so the
    run is kept short and sigma large enough that this factor stays below one.
    """
    rng = np.random.default_rng(5)
    sigma, N, T = 200.0, 5, 12
    X0 = np.array([[0.9, -0.4], [0.3, 0.2]])          # a-b-c+d = 1.2  -> psi' = 2
    xi = rng.choice([-1.0, 1.0], size=(T, N))
    xi[0] = 1.0
    hist, _ = o.run_counterexample(X0, np.array([[0.7], [-0.2]]), xi, sigma, tau=0, eta=0.05, mu=0.9)
    A, B, C = o.A_MAT, o.B_MAT, o.C_VEC
    arg0 = X0[0, 0] - X0[0, 1] - X0[1, 0] + X0[1, 1]
    g2 = 4.0 * o.psi_prime(arg0) ** 2
    assert g2 == pytest.approx(16.0)

    def in_span(M, S):
        c = np.sum(M * S) / np.sum(S * S)
        return np.linalg.norm(M - c * S) <= 1e-11 * max(1.0, np.linalg.norm(M))

    for t, h in enumerate(hist):
        assert np.allclose(np.abs(h["P_hat"]), C, atol=1e-12)
        assert np.linalg.norm(h["Q"] - C * (C.T @ h["Q"])) < 1e-10 * sigma
        assert in_span(h["mom"], B)
        assert in_span(h["X"] - X0, B)
        assert np.sum(h["grad"] ** 2) == pytest.approx(g2, rel=1e-12)
        for i in range(N):
            assert in_span(h["E"][i], A)
            beta = sigma if xi[t, i] > 0 else -sigma
            np.testing.assert_allclose(h["Dhat_i"][i], beta * B, atol=1e-10 * sigma)


def check_refresh_escapes(o):
    """Algorithm 2, green branch: with tau > 0 the same run leaves the trap.

    The residuals accumulate along A until the node-mean's leading singular
    direction is A's; the next refresh then picks it and the gradient starts to
    shrink, whereas with tau = 0 it never does (Theorem 1 vs Theorem 2).
    """
    sigma, N, T = 2.5, 5, 6
    X0 = np.array([[0.9, -0.4], [0.3, 0.2]])
    # fixed draws: all +1 at t = 0; at t = 1 two nodes draw -1, at t = 2 four do.
    xi = np.array([[1, 1, 1, 1, 1], [1, -1, 1, -1, 1], [-1, -1, 1, -1, -1],
                   [1, -1, -1, 1, -1], [1, 1, -1, -1, -1], [-1, 1, 1, -1, -1]], dtype=float)
    args = dict(X0=X0, Q_init=np.array([[0.7], [-0.2]]), xi=xi, sigma=sigma, eta=0.05, mu=0.0)
    h0, X_plain = o.run_counterexample(tau=0, **args)
    h1, X_plus = o.run_counterexample(tau=2, **args)
    g_plain = np.linalg.norm(o.counter_grad(X_plain))
    assert g_plain == pytest.approx(4.0, rel=1e-6)
    # by hand: at t = 2 the node mean is 4.8 A - 1.5 B, so SVD-Comp picks A's direction,
    # the compressed update is 4.8 A and D^T X D drops from 1.2 by 4 * 0.05 * 4.8 = 0.96
    np.testing.assert_allclose(h1[2]["Dbar"], 4.8 * o.A_MAT - 1.5 * o.B_MAT, atol=1e-12)
    np.testing.assert_allclose(h1[2]["Dhat"], 4.8 * o.A_MAT, atol=1e-12)
    arg3 = float((o.D_VEC.T @ h1[3]["X"] @ o.D_VEC)[0, 0])
    assert arg3 == pytest.approx(0.24, abs=1e-12)
    assert np.linalg.norm(h1[3]["grad"]) == pytest.approx(2 * 0.48, rel=1e-10)
    # schedule: SVD-Comp exactly at t = 0, 2, 4
    assert [h["refresh"] for h in h1] == [t % 2 == 0 for t in range(T)]
    assert not any(h["refresh"] for h in h0)


def check_exact_recovery(o):
    """Rank-r input on every node, zero residual, generic Q: one SSP step is exact."""
    m, n, r, N = 12, 9, 3, 4
    G = synth.exact_rank_r(m, n, r, N).astype(np.float64)
    Q0 = np.random.default_rng(2).standard_normal((n, r))
    st = o.PowerSGDPlusOracle(m, n, r, N, 0, Q0)
    out = st.step(G)
    np.testing.assert_allclose(out["Dhat"], G[0], atol=1e-12)
    assert np.linalg.norm(out["E"]) < 1e-11
    st = o.PowerSGDPlusOracle(m, n, r, N, 1, Q0)
    out = st.step(G)
    assert out["refresh"]
    np.testing.assert_allclose(out["Dhat"], G[0], atol=1e-12)


def check_qr(o):
    """QR(.) of Sec. 2: orthonormal factor, positive diagonal, against LAPACK and exact GS."""
    rng = np.random.default_rng(3)
    for rows, cols in [(7, 1), (5, 5), (40, 6), (33, 17)]:
        A = rng.standard_normal((rows, cols))
        Qh, R = o.householder_qr(A)
        np.testing.assert_allclose(Qh.T @ Qh, np.eye(cols), atol=1e-13)
        np.testing.assert_allclose(Qh @ R, A, atol=1e-13)
        assert np.allclose(R, np.triu(R)) and np.all(np.diag(R) > 0)
        ql, rl = np.linalg.qr(A)
        sg = np.sign(np.diag(rl))
        np.testing.assert_allclose(Qh, ql * sg[None, :], atol=1e-12)
        np.testing.assert_allclose(o.qr_orth(A), Qh, atol=0)
    # exact-rational classical Gram-Schmidt on a small integer matrix
    Ai = [[2, -1, 3], [1, 4, 0], [-3, 2, 1], [0, 5, -2], [1, 1, 1]]
    cols = [[Fraction(Ai[i][j]) for i in range(5)] for j in range(3)]
    basis = []
    for c in cols:
        v = list(c)
        for b in basis:
            coef = sum(x * y for x, y in zip(c, b)) / sum(y * y for y in b)
            v = [x - coef * y for x, y in zip(v, b)]
        basis.append(v)
    ref = np.array([[float(x) for x in b] for b in basis]).T
    ref /= np.linalg.norm(ref, axis=0, keepdims=True)
    Qh, R = o.householder_qr(np.array(Ai, dtype=float))
    np.testing.assert_allclose(Qh, ref, atol=1e-14)
    # r = 1: plain normalisation; zero matrix: still orthonormal
    v = rng.standard_normal((9, 1))
    np.testing.assert_allclose(o.qr_orth(v), v / np.linalg.norm(v), atol=1e-15)
    Z = o.qr_orth(np.zeros((6, 2)))
    np.testing.assert_allclose(Z.T @ Z, np.eye(2), atol=1e-14)
    # rank-deficient: span is kept, factor is orthonormal
    a = rng.standard_normal((8, 1))
    Ad = np.hstack([a, 2 * a, rng.standard_normal((8, 1))])
    Qd, Rd = o.householder_qr(Ad)
    np.testing.assert_allclose(Qd.T @ Qd, np.eye(3), atol=1e-13)
    np.testing.assert_allclose(Qd @ Rd, Ad, atol=1e-13)


def check_error_identities(o):
    """Eq. (4), Appendix B linearity, and the residual identities, SSP and SVD steps."""
    m, n, r, N = 24, 10, 3, 4
    G = synth.make_gradients(1, m, n, N, step=0).astype(np.float64)
    rng = np.random.default_rng(4)
    st = o.PowerSGDPlusOracle(m, n, r, N, 3, rng.standard_normal((n, r)))
    st.E = rng.standard_normal((N, m, n)) * 0.1
    for t in range(4):
        E_before = st.E.copy()
        out = st.step(G * (1 + 0.1 * t))
        M, Ph = out["M"], out["P_hat"]
        np.testing.assert_allclose(M, G * (1 + 0.1 * t) + E_before, atol=0)
        np.testing.assert_allclose(Ph.T @ Ph, np.eye(r), atol=1e-12)
        for i in range(N):
            np.testing.assert_allclose(out["E"][i] + Ph @ out["Q_i"][i].T, M[i], atol=1e-12)
            assert np.linalg.norm(Ph.T @ out["E"][i]) < 1e-11
            assert np.sum(out["E"][i] ** 2) + np.sum(out["Dhat_i"][i] ** 2) == pytest.approx(np.sum(M[i] ** 2), rel=1e-12)
            np.testing.assert_allclose(out["Q_i"][i], M[i].T @ Ph, atol=1e-12)
            np.testing.assert_allclose(out["Dhat_i"][i], Ph @ Ph.T @ M[i], atol=1e-12)
        Mbar = M.mean(axis=0)
        np.testing.assert_allclose(out["Dhat_i"].mean(axis=0), out["Dhat"], atol=1e-12)
        np.testing.assert_allclose(out["E"].mean(axis=0), Mbar - Ph @ (Ph.T @ Mbar), atol=1e-12)
        np.testing.assert_allclose(out["Q"], Mbar.T @ Ph, atol=1e-12)
        if not out["refresh"]:   # state wiring: this step projected with the previous step's Q_t
            np.testing.assert_allclose(out["P"], Mbar @ Q_prev, atol=1e-12)
        Q_prev = out["Q"].copy()
    # SSP: P is the node mean of M_i Q_{t-1}
    Qprev = rng.standard_normal((n, r))
    st = o.PowerSGDPlusOracle(m, n, r, N, 0, Qprev)
    out = st.step(G)
    np.testing.assert_allclose(out["P"], G.mean(axis=0) @ Qprev, atol=1e-12)
    for i in range(N):
        np.testing.assert_allclose(out["P_i"][i], G[i] @ Qprev, atol=1e-12)
    # the "mean" error form subtracts the averaged reconstruction
    st2 = o.PowerSGDPlusOracle(m, n, r, N, 0, Qprev, error_form="mean")
    out2 = st2.step(G)
    for i in range(N):
        np.testing.assert_allclose(out2["E"][i], G[i] - out2["P_hat"] @ out2["Q"].T, atol=1e-12)
    np.testing.assert_allclose(out2["E"].mean(axis=0), out["E"].mean(axis=0), atol=1e-12)


def check_svd_tiny(o):
    """Definition 3 / Eq. (5)-(6): brute force on tiny inputs."""
    rng = np.random.default_rng(6)
    for (m, n, r) in [(6, 4, 1), (8, 6, 2), (7, 5, 3), (5, 5, 4)]:
        W = rng.standard_normal((m, n))
        P, s = o.svd_top_r(W, r)
        np.testing.assert_allclose(P.T @ P, np.eye(r), atol=1e-13)
        # independent eigen-solve of W W^T
        lam, vec = np.linalg.eigh(W @ W.T)
        order = np.argsort(lam)[::-1]
        lam, vec = lam[order], vec[:, order]
        np.testing.assert_allclose(s ** 2, lam[:n], atol=1e-10)
        np.testing.assert_allclose(P @ P.T, vec[:, :r] @ vec[:, :r].T, atol=1e-9)
        res = np.linalg.norm(P @ (P.T @ W) - W) ** 2
        assert res == pytest.approx(np.sum(s[r:] ** 2), rel=1e-10, abs=1e-12)
        assert res <= (1 - r / n) * np.linalg.norm(W) ** 2 + 1e-12
        # exhaustive: no other r-subset of eigenvectors does better
        for sub in itertools.combinations(range(m), r):
            Ps = vec[:, list(sub)]
            assert np.linalg.norm(Ps @ (Ps.T @ W) - W) ** 2 >= res - 1e-10
        # random semi-orthogonal competitors never win
        for _ in range(50):
            Pr = np.linalg.qr(rng.standard_normal((m, r)))[0]
            assert np.linalg.norm(Pr @ (Pr.T @ W) - W) ** 2 >= res - 1e-10
    # constructed spectrum
    U = synth.random_orthonormal(20, 6, rng)
    V = synth.random_orthonormal(9, 6, rng)
    s = np.array([5.0, 3.0, 2.0, 0.5, 0.25, 0.1])
    W = (U * s) @ V.T
    P, sv = o.svd_top_r(W, 3)
    np.testing.assert_allclose(sv[:6], s, atol=1e-12)
    np.testing.assert_allclose(P @ P.T, U[:, :3] @ U[:, :3].T, atol=1e-12)
    # SVD-Comp uses the node MEAN (not a single node, not the sum)
    D = rng.standard_normal((3, 8, 5))
    out = o.svd_comp(D, 2)
    Pm, _ = o.svd_top_r(D.mean(axis=0), 2)
    np.testing.assert_allclose(out["P_hat"] @ out["P_hat"].T, Pm @ Pm.T, atol=1e-11)
    np.testing.assert_allclose(out["Dbar"], D.mean(axis=0), atol=1e-15)


def check_fixed_point(o):
    """Eq. (9): started from Q = V_r Sigma_r the SSP step reproduces the SVD compressor."""
    rng = np.random.default_rng(7)
    m, n, r, N = 16, 8, 3, 2
    D = rng.standard_normal((N, m, n))
    Dbar = D.mean(axis=0)
    U, s, Vt = np.linalg.svd(Dbar, full_matrices=False)
    Q0 = Vt[:r].T * s[:r]
    a = o.ssp_comp(Q0, D)
    b = o.svd_comp(D, r)
    np.testing.assert_allclose(a["P_hat"] @ a["P_hat"].T, b["P_hat"] @ b["P_hat"].T, atol=1e-11)
    np.testing.assert_allclose(a["Dhat"], b["Dhat"], atol=1e-11)
    np.testing.assert_allclose(a["Dhat"], (U[:, :r] * s[:r]) @ Vt[:r], atol=1e-11)
    # N = 1, K-step power iteration with K = 1 is the same thing as SSP-Comp
    P1, Q1 = o.power_iteration(D[0], Q0, 1)
    c = o.ssp_comp(Q0, D[:1])
    np.testing.assert_allclose(P1, c["P_hat"], atol=1e-13)
    np.testing.assert_allclose(Q1, c["Q"], atol=1e-13)
    # many power steps converge to the optimal compressor (Eq. (8))
    Pk, Qk = o.power_iteration(Dbar, rng.standard_normal((n, r)), 400)
    np.testing.assert_allclose(Pk @ Qk.T, (U[:, :r] * s[:r]) @ Vt[:r], atol=1e-8)
    # K power steps across the nodes (means of per-node products) are K power steps on the node mean
    Qs = rng.standard_normal((n, r))
    for K in (2, 5):
        d = o.ssp_comp(Qs, D, power_steps=K)
        Pk, Qk = o.power_iteration(Dbar, Qs, K)
        np.testing.assert_allclose(d["P_hat"], Pk, atol=1e-12)
        np.testing.assert_allclose(d["Q"], Qk, atol=1e-12)


def check_counter_function(o):
    """Eq. (10a): psi, its derivative, and the gradient against finite differences."""
    for x in [-3.0, -1.0, -0.4, 0.0, 0.7, 1.0, 2.5]:
        assert o.psi(x) == pytest.approx(x * x if abs(x) <= 1 else 2 * abs(x) - 1)
    rng = np.random.default_rng(8)
    for _ in range(5):
        X = rng.standard_normal((2, 2)) * 0.3
        g = o.counter_grad(X)
        fd = np.zeros((2, 2))
        for i in range(2):
            for j in range(2):
                d = np.zeros((2, 2)); d[i, j] = 1e-6
                fd[i, j] = (o.counter_f(X + d) - o.counter_f(X - d)) / 2e-6
        np.testing.assert_allclose(g, fd, atol=1e-6)
    X = np.array([[2.0, -1.0], [-1.0, 2.0]])   # argument 6 -> linear branch
    np.testing.assert_allclose(o.counter_grad(X), 2.0 * o.A_MAT, atol=0)
    gs = o.counter_stoch_grad(X, [1.0, -1.0], 1.5)
    np.testing.assert_allclose(gs[0], 1.5 * o.B_MAT, atol=1e-15)
    np.testing.assert_allclose(gs[1], 2 * o.counter_grad(X) - 1.5 * o.B_MAT, atol=1e-15)
    np.testing.assert_allclose(gs.mean(axis=0), o.counter_grad(X), atol=1e-15)  # unbiased


def check_tf32_product(o):
    """TF32 keeps 1 sign + 8 exponent + 10 mantissa bits of a float32 and drops the 13 low ones by truncation.
    Values the format fixes, chosen so that a mask one bit too short or too long, or rounding instead of
    truncation, gives a different answer; then a 2 x 2 x 2 product worked out by hand."""
    one = 1.0
    keep = np.float32(1.0 + 2.0 ** -10)                     # last kept bit
    drop = np.float32(1.0 + 2.0 ** -11)                     # first dropped bit: truncates to 1, rounding would not
    drop2 = np.float32(1.0 + 2.0 ** -11 + 2.0 ** -12)       # above half an ulp: still truncates down
    top = np.float32(2.0 - 2.0 ** -23)                      # all mantissa bits set -> 2 - 2^-10
    x = np.array([keep, drop, drop2, top, -drop2, -top, 0.0, np.float32(2.0 ** -120) * drop2, np.float32(2.0 ** 100) * top], dtype=np.float32)
    want = np.array([1.0 + 2.0 ** -10, one, one, 2.0 - 2.0 ** -10, -one, -(2.0 - 2.0 ** -10), 0.0,
                     2.0 ** -120, 2.0 ** 100 * (2.0 - 2.0 ** -10)])
    got = o.tf32_truncate(x)
    assert got.dtype == np.float64
    np.testing.assert_array_equal(got, want)                 # sign and exponent untouched, magnitude never grows
    # every TF32 number is a fixed point; truncation is idempotent
    rng = np.random.default_rng(12)
    y = (rng.standard_normal(1000) * 10.0 ** rng.integers(-20, 20, 1000)).astype(np.float32)
    t = o.tf32_truncate(y)
    np.testing.assert_array_equal(o.tf32_truncate(t.astype(np.float32)), t)
    assert np.all(np.abs(t) <= np.abs(y.astype(np.float64))) and np.all(np.abs(y - t) < 2.0 ** -10 * np.abs(y) + 1e-300)
    assert np.all(np.mod(np.frexp(t)[0] * 2.0 ** 11, 1.0) == 0.0)      # at most 11 significant bits
    # hand-computed product: a11 = 1 + 2^-10 (kept), a12 = 1 + 2^-11 (-> 1), a21 = 3, a22 = -(1 + 2^-11 + 2^-12) (-> -1);
    # b11 = 2, b12 = 1 + 2^-10 + 2^-13 (-> 1 + 2^-10), b21 = -0.5, b22 = 4.   C = A B^T, C[i][j] = sum_k a[i][k] b[j][k]
    A = np.array([[keep, drop], [3.0, -drop2]], dtype=np.float32)
    B = np.array([[2.0, 1.0 + 2.0 ** -10 + 2.0 ** -13], [-0.5, 4.0]], dtype=np.float32)
    e = 2.0 ** -10
    C = np.array([[(1 + e) * 2 + 1 * (1 + e), (1 + e) * -0.5 + 1 * 4.0],
                  [3 * 2 - 1 * (1 + e), 3 * -0.5 - 1 * 4.0]])
    np.testing.assert_array_equal(o.gemm_nt_tf32(A, B), C)
    # not transposed by mistake: a non-square case against the definition on already-representable operands
    A2 = np.array([[1.0, 2.0, 3.0]], dtype=np.float32)
    B2 = np.array([[1.0, 0.0, 0.0], [0.0, 0.0, 2.0]], dtype=np.float32)
    np.testing.assert_array_equal(o.gemm_nt_tf32(A2, B2), np.array([[1.0, 6.0]]))


ALL_CHECKS = [
    check_counterexample_t0,
    check_counterexample_induction,
    check_refresh_escapes,
    check_exact_recovery,
    check_qr,
    check_error_identities,
    check_svd_tiny,
    check_fixed_point,
    check_counter_function,
    check_tf32_product,
]


@pytest.mark.parametrize("check", ALL_CHECKS, ids=lambda f: f.__name__)
def test_oracle_pin(check):
    check(orc)


# --------------------------------------------------------------------------
# planted mistakes (in the oracle, on the CPU): every one must trip a pin
# --------------------------------------------------------------------------
def _mutant(**overrides):
    """A copy of the oracle module with some functions replaced."""
    src = open(orc.__file__).read()
    mod = types.ModuleType("oracle_mutant")
    mod.__file__ = orc.__file__
    exec(compile(src, orc.__file__, "exec"), mod.__dict__)
    for k, v in overrides.items():
        v(mod) if k.startswith("patch") else setattr(mod, k, v)
    return mod


def _patch_tail_transposed(mod):
    def _tail(P_hat, Delta):
        out = mod._orig_tail(P_hat, Delta)
        N = Delta.shape[0]
        # wrong operand: Delta P~ is not even shaped right unless m == n; emulate
        # the classic slip of projecting with the mean matrix instead of node i
        Dm = Delta.mean(axis=0)
        out["Q_i"] = np.stack([Dm.T @ P_hat for _ in range(N)])
        out["Dhat_i"] = np.stack([P_hat @ out["Q_i"][i].T for i in range(N)])
        return out
    mod._orig_tail = mod._tail
    mod._tail = _tail


def _patch_no_sign_fix(mod):
    def hq(A):
        q, r = np.linalg.qr(np.asarray(A, dtype=float))
        return q, r                       # LAPACK's sign, not diag(R) >= 0
    mod.householder_qr = hq


def _patch_sum_not_mean(mod):
    mod._mean = lambda X: np.sum(X, axis=0)


def _patch_no_error_feedback(mod):
    orig = mod.PowerSGDPlusOracle.step
    def step(self, G, force_svd=False):
        self.E = np.zeros_like(self.E)    # dropped term: e_t never added
        return orig(self, G, force_svd)
    mod.PowerSGDPlusOracle.step = step


def _patch_refresh_off_by_one(mod):
    mod.PowerSGDPlusOracle.is_refresh_step = lambda self: self.tau > 0 and (self.t + 1) % self.tau == 0


def _patch_svd_right_vectors(mod):
    def svd_top_r(W, r):
        U, s, Vt = np.linalg.svd(np.asarray(W, dtype=float), full_matrices=False)
        return U[:, -r:].copy(), s        # trailing instead of leading vectors
    mod.svd_top_r = svd_top_r


def _patch_stale_q(mod):
    orig = mod.PowerSGDPlusOracle.step
    def step(self, G, force_svd=False):
        q = self.Q.copy()
        out = orig(self, G, force_svd)
        self.Q = q                        # forgot to carry Q_t forward
        return out
    mod.PowerSGDPlusOracle.step = step


def _patch_psi_wrong_arg(mod):
    # the garbled sign pattern that appears once in Appendix A
    mod.counter_grad = lambda X: mod.psi_prime(X[0, 0] + X[0, 1] - X[1, 0] - X[1, 1]) * mod.A_MAT


def _patch_tf32_mask(bits_dropped):
    def patch(mod):
        mask = np.uint32((0xFFFFFFFF << bits_dropped) & 0xFFFFFFFF)
        mod.tf32_truncate = lambda X: (np.ascontiguousarray(X, dtype=np.float32).view(np.uint32) & mask).view(np.float32).astype(np.float64)
    return patch


def _patch_tf32_rounds(mod):
    def rn(X):      # round to nearest instead of truncation
        b = np.ascontiguousarray(X, dtype=np.float32).view(np.uint32)
        return ((b + np.uint32(0x1000)) & np.uint32(0xFFFFE000)).view(np.float32).astype(np.float64)
    mod.tf32_truncate = rn


def _patch_gemm_not_transposed(mod):
    mod.gemm_nt_tf32 = lambda A, B: mod.tf32_truncate(A) @ mod.tf32_truncate(B)


MUTANTS = {
    "node_mean_used_for_local_Q": _patch_tail_transposed,
    "qr_sign_not_fixed": _patch_no_sign_fix,
    "sum_instead_of_mean": _patch_sum_not_mean,
    "error_feedback_dropped": _patch_no_error_feedback,
    "refresh_off_by_one": _patch_refresh_off_by_one,
    "svd_trailing_vectors": _patch_svd_right_vectors,
    "psi_argument_garbled": _patch_psi_wrong_arg,
    "stale_Q_state": _patch_stale_q,
    "tf32_mask_12_bits": _patch_tf32_mask(12),
    "tf32_mask_14_bits": _patch_tf32_mask(14),
    "tf32_rounds_to_nearest": _patch_tf32_rounds,
    "tf32_product_not_transposed": _patch_gemm_not_transposed,
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(name):
    mod = _mutant(**{"patch_" + name: MUTANTS[name]})
    tripped = []
    for chk in ALL_CHECKS:
        try:
            chk(mod)
        except Exception:
            tripped.append(chk.__name__)
    assert tripped, f"no pin caught the planted mistake {name}"


def test_msgd_update_closed_form():
    """Eq. (7c) with a constant reconstruction D and m_{-1} = 0: m_t = D (1 - mu^(t+1)) / (1 - mu) and
    X_T = X_0 - eta D sum_{t<T} (1 - mu^(t+1)) / (1 - mu); with mu = 0 plain SGD, X_T = X_0 - T eta D."""
    rng = np.random.default_rng(3)
    X0, D = rng.standard_normal((5, 4)), rng.standard_normal((5, 4))
    for mu, eta, T in [(0.9, 0.05, 7), (0.0, 0.1, 4), (0.5, 1.0, 3)]:
        X, mom = X0.copy(), np.zeros_like(X0)
        for _ in range(T):
            X, mom = orc.msgd_update(X, mom, D, eta, mu)
        geo = [(1 - mu ** (t + 1)) / (1 - mu) for t in range(T)]
        np.testing.assert_allclose(mom, D * geo[-1], rtol=1e-13, atol=1e-15)
        np.testing.assert_allclose(X, X0 - eta * D * sum(geo), rtol=1e-13, atol=1e-13)
