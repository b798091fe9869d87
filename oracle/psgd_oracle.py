"""CPU oracle for the PowerSGD+ compression path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, double-precision restatement of what the compression path
computes, written from the paper's statement of the method.  It shares no
code with the CUDA library and must never be imported by it: only the test
suite, the smoke check and the benchmark's CPU-baseline leg may call it.

What follows the paper, and where:

* error-feedback add  Delta_i = g_i + e_i ........................ Eq. (7a)
* SSP-Comp  (P_i = Delta_i Q, mean, QR, Q_i = Delta_i^T P~, mean) . Algorithm 1
* SVD-Comp  (mean of Delta_i, SVD, P~ = U[:, :r], Q_i, mean) ...... Algorithm 1
* QR(.) = economy QR that returns only the orthonormal factor ..... Sec. 2 "QR decomposition"
* optimal rank-r compressor = leading r left singular vectors ..... Definition 3, Eq. (5)-(6)
* schedule: SVD-Comp iff mod(t, tau) == 0, else SSP-Comp .......... Algorithm 2
* residual  e_i <- Delta_i - Delta^_i ............................. Algorithm 2, last line
* K-step power iteration ......................................... Eq. (8)
* MSGD update (used only by the counterexample driver) ............ Eq. (7c)
* counterexample objective and stochastic gradient ............... Eq. (10a)-(10b), Appendix A

Readings taken where the paper is silent (each is listed in the design notes):
the QR factor is made unique by diag(R) >= 0; t = 0 is a refresh step when
tau > 0; one shared Q on every node; means are plain left-to-right sums in
double; psi'(x) = 2x on |x| <= 1 and 2 sign(x) outside; the argument of psi is
x11 - x12 - x21 + x22 (= D^T X D).

Pins (tests/test_oracle_*.py): the counterexample's closed-form values, exact
recovery of exactly-rank-r input, orthonormality, the Pythagoras identity
Eq. (4), linearity of the compressor (Appendix B), Eq. (6), comparison with an
independent eigen-solve and exhaustive subset search on tiny inputs, LAPACK QR
with sign fix, exact-rational Gram-Schmidt, and for the TF32 product the values
the number format fixes (last kept and first dropped mantissa bit, truncation
not rounding) with a hand-computed 2 x 2 x 2 product.  Nothing here is "parity
unpinned" except the trajectories of the large synthetic workloads, for which
no published values exist.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# QR(.) of Sec. 2: economy Householder QR, R discarded by the callers.
# --------------------------------------------------------------------------
def householder_qr(A):
    """Economy QR of A (rows >= cols) by Householder reflections.

    Returns (Qhat, R) with Qhat^T Qhat = I, Qhat R = A, R upper triangular and
    diag(R) >= 0.  The sign convention makes the factor unique for full column
    rank; for a rank-deficient A the reflections still deliver an orthonormal
    completion.
    """
    A = np.array(A, dtype=F64, copy=True)
    rows, cols = A.shape
    if rows < cols:
        raise ValueError("householder_qr needs rows >= cols")
    V = []  # reflector vectors
    for k in range(cols):
        x = A[k:, k].copy()
        alpha = np.linalg.norm(x)
        v = x.copy()
        if alpha == 0.0:
            # zero column: the identity is a valid reflection choice
            V.append(None)
            continue
        # reflect x onto -sign(x0)*alpha*e1 (the numerically stable choice)
        s = 1.0 if x[0] >= 0 else -1.0
        v[0] += s * alpha
        v /= np.linalg.norm(v)
        V.append(v)
        A[k:, k:] -= 2.0 * np.outer(v, v @ A[k:, k:])
    R = np.triu(A[:cols, :])
    # accumulate Qhat = H_0 H_1 ... H_{cols-1} [I; 0]
    Qh = np.zeros((rows, cols), dtype=F64)
    Qh[:cols, :cols] = np.eye(cols)
    for k in reversed(range(cols)):
        v = V[k]
        if v is None:
            continue
        Qh[k:, :] -= 2.0 * np.outer(v, v @ Qh[k:, :])
    # make diag(R) non-negative: flip column k of Qhat and row k of R together
    for k in range(cols):
        if R[k, k] < 0:
            R[k, :] = -R[k, :]
            Qh[:, k] = -Qh[:, k]
    return Qh, R


def qr_orth(A):
    """QR(.) as the paper uses it: only the orthonormal factor is returned."""
    return householder_qr(A)[0]


# --------------------------------------------------------------------------
# Optimal rank-r compressor, Definition 3 / Eq. (5): P~ = U[:, :r].
# --------------------------------------------------------------------------
def svd_top_r(W, r):
    """Leading r left singular vectors of W and all singular values (descending)."""
    W = np.asarray(W, dtype=F64)
    U, s, _Vt = np.linalg.svd(W, full_matrices=False)
    return U[:, :r].copy(), s


# --------------------------------------------------------------------------
# Product with TF32 operands: what the tensor-core sweeps of the refresh compute
# for one contraction of the subspace iteration (any basis of the subspace is a
# valid SVD-Comp result, so the sweeps themselves need no oracle; this function
# defines the single product so that the kernel can be checked in isolation).
# --------------------------------------------------------------------------
def tf32_truncate(X):
    """float32 values with the 13 low mantissa bits cleared (TF32: 1 + 8 + 10 bits), as float64."""
    bits = np.ascontiguousarray(X, dtype=np.float32).view(np.uint32) & np.uint32(0xFFFFE000)
    return bits.view(np.float32).astype(F64)


def gemm_nt_tf32(A, B):
    """C = A B^T with both operands truncated to TF32 and exact (double) accumulation."""
    return tf32_truncate(A) @ tf32_truncate(B).T


# --------------------------------------------------------------------------
# Algorithm 1, both compressors.  Delta has shape [N, m, n].
# --------------------------------------------------------------------------
def ssp_comp(Q, Delta, power_steps=1):
    """SSP-Comp of Algorithm 1.  Returns a dict of every intermediate.

    power_steps = K > 1 runs the K-step power iteration of Eq. (8) across the nodes: the first K - 1
    rounds only carry Q forward (Q <- mean_i Delta_i^T P~), the K-th is the round Algorithm 1 states.
    """
    Delta = np.asarray(Delta, dtype=F64)
    Q = np.asarray(Q, dtype=F64)
    N = Delta.shape[0]
    for _ in range(power_steps - 1):
        P_hat = qr_orth(_mean(np.stack([Delta[i] @ Q for i in range(N)])))
        Q = _mean(np.stack([Delta[i].T @ P_hat for i in range(N)]))
    P_i = np.stack([Delta[i] @ Q for i in range(N)])           # P^(i) <- Delta^(i) Q
    P = _mean(P_i)                                              # All-Reduce Mean
    P_hat, R = householder_qr(P)                                # P~ <- QR(P)
    out = _tail(P_hat, Delta)
    out.update(P_i=P_i, P=P, R=R)
    return out


def svd_comp(Delta, r):
    """SVD-Comp of Algorithm 1."""
    Delta = np.asarray(Delta, dtype=F64)
    Dbar = _mean(Delta)                                         # All-Reduce Mean
    P_hat, s = svd_top_r(Dbar, r)                               # U[:, :r]
    out = _tail(P_hat, Delta)
    out.update(Dbar=Dbar, sigma=s)
    return out


def _mean(X):
    """Plain left-to-right mean over the leading (node) axis."""
    acc = np.zeros_like(X[0], dtype=F64)
    for i in range(X.shape[0]):
        acc = acc + X[i]
    return acc / X.shape[0]


def _tail(P_hat, Delta):
    """Last three lines shared by both compressors of Algorithm 1."""
    N = Delta.shape[0]
    Q_i = np.stack([Delta[i].T @ P_hat for i in range(N)])      # Q^(i) <- Delta^(i)^T P~
    Q = _mean(Q_i)                                              # All-Reduce Mean
    Dhat_i = np.stack([P_hat @ Q_i[i].T for i in range(N)])     # P~ Q^(i)^T
    Dhat = P_hat @ Q.T                                          # P~ Q^T
    return dict(P_hat=P_hat, Q_i=Q_i, Q=Q, Dhat_i=Dhat_i, Dhat=Dhat)


def power_iteration(Dbar, Q_init, K):
    """K-step power iteration of Eq. (8) on one matrix; K = 1 is Eq. (9)."""
    Q = np.asarray(Q_init, dtype=F64)
    Dbar = np.asarray(Dbar, dtype=F64)
    P_hat = None
    for _ in range(K):
        P_hat = qr_orth(Dbar @ Q)
        Q = Dbar.T @ P_hat
    return P_hat, Q


# --------------------------------------------------------------------------
# Algorithm 2: the per-iteration compression with error feedback.
# --------------------------------------------------------------------------
class PowerSGDPlusOracle:
    """State (t, Q, e_i) of Algorithm 2 for ONE matrix variable on N nodes.

    tau = 0 means "never refresh", i.e. plain PowerSGD (the red branch of
    Algorithm 2).  `error_form` selects which reconstruction the residual
    subtracts: "local" is the paper's e_i <- Delta_i - P~ Q_i^T; "mean"
    subtracts P~ Q^T with the node-averaged Q instead.
    """

    def __init__(self, m, n, r, N, tau, Q_init, error_form="local", power_steps=1):
        if not (m >= n >= r >= 1 and N >= 1 and tau >= 0):
            raise ValueError("need m >= n >= r >= 1, N >= 1, tau >= 0")
        if error_form not in ("local", "mean"):
            raise ValueError("error_form")
        self.m, self.n, self.r, self.N, self.tau = m, n, r, N, tau
        self.error_form = error_form
        self.power_steps = power_steps
        self.t = 0
        self.Q = np.array(Q_init, dtype=F64).reshape(n, r).copy()
        self.E = np.zeros((N, m, n), dtype=F64)                 # e_0^(i) = 0

    def is_refresh_step(self):
        return self.tau > 0 and self.t % self.tau == 0

    def step(self, G, force_svd=False):
        """One iteration t of Algorithm 2 (without the optimizer update).

        G: [N, m, n] stochastic gradients g_t^(i).  Returns the dict of
        intermediates; the state (t, Q, E) is advanced in place.
        """
        G = np.asarray(G, dtype=F64).reshape(self.N, self.m, self.n)
        M = G + self.E                                          # Eq. (7a)
        refresh = force_svd or self.is_refresh_step()
        out = svd_comp(M, self.r) if refresh else ssp_comp(self.Q, M, self.power_steps)
        if self.error_form == "local":
            E_new = M - out["Dhat_i"]                           # e_{t+1}^(i)
        else:
            E_new = M - out["Dhat"][None, :, :]
        out.update(M=M, E=E_new, refresh=refresh, t=self.t)
        self.Q = out["Q"].copy()
        self.E = E_new
        self.t += 1
        return out


# --------------------------------------------------------------------------
# The counterexample of Eq. (10) / Appendix A (2x2 variable, rank 1).
# --------------------------------------------------------------------------
A_MAT = np.array([[1.0, -1.0], [-1.0, 1.0]])
B_MAT = np.array([[1.0, 1.0], [1.0, 1.0]])
C_VEC = np.array([[np.sqrt(2.0) / 2.0], [np.sqrt(2.0) / 2.0]])
D_VEC = np.array([[1.0], [-1.0]])


def psi(x):
    return x * x if abs(x) <= 1.0 else 2.0 * abs(x) - 1.0


def psi_prime(x):
    return 2.0 * x if abs(x) <= 1.0 else 2.0 * np.sign(x)


def counter_f(X):
    """f(X) = psi(D^T X D) = psi(x11 - x12 - x21 + x22)."""
    return psi(float((D_VEC.T @ X @ D_VEC)[0, 0]))


def counter_grad(X):
    """grad f(X) = psi'(D^T X D) * D D^T = psi'(.) * A."""
    return psi_prime(float((D_VEC.T @ X @ D_VEC)[0, 0])) * A_MAT


def counter_stoch_grad(X, xi, sigma):
    """Eq. (10b): grad f + xi (sigma B - grad f), one matrix per node."""
    g = counter_grad(X)
    return np.stack([g + x * (sigma * B_MAT - g) for x in xi])


def msgd_update(X, mom, Dhat, eta, mu):
    """Eq. (7c): m_t = mu m_{t-1} + Dhat_t;  X_{t+1} = X_t - eta m_t.  Returns (X_{t+1}, m_t)."""
    mom = mu * np.asarray(mom, dtype=F64) + np.asarray(Dhat, dtype=F64)
    return np.asarray(X, dtype=F64) - eta * mom, mom


def run_counterexample(X0, Q_init, xi, sigma, tau, eta, mu, error_form="local"):
    """Algorithm 2 with the MSGD update of Eq. (7c) on the counterexample.

    xi: [T, N] array of +-1 draws.  Returns per-step records (X_t before the
    update, the compressor's outputs, the momentum after the update).
    """
    xi = np.asarray(xi, dtype=F64)
    T, N = xi.shape
    orc = PowerSGDPlusOracle(2, 2, 1, N, tau, Q_init, error_form)
    X = np.array(X0, dtype=F64)
    mom = np.zeros((2, 2))
    hist = []
    for t in range(T):
        G = counter_stoch_grad(X, xi[t], sigma)
        out = orc.step(G)
        Xn, mom = msgd_update(X, mom, out["Dhat"], eta, mu)
        rec = dict(X=X.copy(), grad=counter_grad(X), mom=mom.copy(), **out)
        X = Xn
        hist.append(rec)
    return hist, X
