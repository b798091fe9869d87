"""Seeded synthetic gradients shaped like the paper's LLM workloads.

This module only *generates inputs*.  It contains none of the compression
method's arithmetic and is the one module that both the CUDA path's callers
and the CPU oracle's callers may import.  Every random slab is drawn from a
counter-based generator (Philox) keyed by
(master seed, workload id, matrix id, node, step, purpose), so any slab can be
regenerated independently of the others.

The paper trains LLaMA-60M/130M on C4 and RoBERTa-Base on GLUE (Sec. 5); none of
that data is used here.  The workloads below stand in for it: they take the
*shapes* of such models' weight matrices and fill them with a decaying-spectrum
low-rank term plus Gaussian noise.
"""
from __future__ import annotations

import numpy as np

MASTER_SEED = 20250911

_PURPOSE = {"U": 1, "V": 2, "noise": 3, "Q": 4, "Unode": 5, "misc": 6}


def rng_for(workload, matrix_id, node, step, purpose, seed=MASTER_SEED):
    """Independent generator for one slab."""
    key = (np.uint64(seed) << np.uint64(8)) ^ np.uint64(workload)
    ctr = [int(matrix_id), int(node) + 1, int(step) + 1, _PURPOSE[purpose]]
    return np.random.Generator(np.random.Philox(key=int(key), counter=ctr))


def random_orthonormal(rows, cols, rng):
    """Orthonormal columns: the Q factor of a Gaussian matrix."""
    q, rr = np.linalg.qr(rng.standard_normal((rows, cols)))
    return q * np.sign(np.diag(rr))[None, :]


def spectrum(kind, K):
    k1 = np.arange(1, K + 1, dtype=np.float64)
    if kind == "pow2":        # s_k = 2^-k, k = 0..K-1
        return 2.0 ** (-(k1 - 1))
    if kind == "k^-1.5":      # s_k = k^-1.5, k = 1..K
        return k1 ** -1.5
    if kind == "k^-1":
        return k1 ** -1.0
    if kind == "0.9^k":       # s_k = 0.9^k, k = 0..K-1
        return 0.9 ** (k1 - 1)
    raise ValueError(kind)


# workload id -> recipe.  noise: ("abs", c) adds c * Z / sqrt(n);
# ("rel", x) rescales Z_i so that ||Z_i||_F = x * ||L||_F.
WORKLOADS = {
    1: dict(name="tiny", spec="pow2", K=16, noise=("abs", 0.05), hetero=0),
    2: dict(name="llama130m", spec="k^-1.5", K=64, noise=("rel", 0.10), hetero=0),
    3: dict(name="llama130m-hetero", spec="k^-1.5", K=64, noise=("rel", 0.10), hetero=8),
    4: dict(name="llama1b", spec="k^-1", K=64, noise=("rel", 0.05), hetero=0),
    5: dict(name="sweep", spec="0.9^k", K=256, noise=("rel", 0.05), hetero=0),
}

# (m, n, count) shape classes of the stacks (matrices stored so that m >= n)
STACKS = {
    2: [(768, 768, 48), (2048, 768, 36)],
    3: [(768, 768, 48), (2048, 768, 36)],
    4: [(2048, 2048, 96), (5504, 2048, 72)],
    5: [(16384, 4096, 1)],
    1: [(256, 128, 1)],
}


def low_rank_factors(workload, m, n, matrix_id=0, seed=MASTER_SEED):
    """(U [m,K], s [K], V [n,K]) of the step-independent low-rank term."""
    w = WORKLOADS[workload]
    K = min(w["K"], n)
    U = random_orthonormal(m, K, rng_for(workload, matrix_id, -1, -1, "U", seed))
    V = random_orthonormal(n, K, rng_for(workload, matrix_id, -1, -1, "V", seed))
    return U, spectrum(w["spec"], K), V


def make_gradients(workload, m, n, N, step, matrix_id=0, seed=MASTER_SEED):
    """Per-node gradients g_t^(i), float32 [N, m, n]."""
    w = WORKLOADS[workload]
    U, s, V = low_rank_factors(workload, m, n, matrix_id, seed)
    L = (U * s[None, :]) @ V.T
    normL = np.linalg.norm(L)
    G = np.empty((N, m, n), dtype=np.float32)
    for i in range(N):
        Li = L
        if w["hetero"]:
            h = min(w["hetero"], U.shape[1])
            Ui = U.copy()
            Ui[:, :h] = random_orthonormal(m, h, rng_for(workload, matrix_id, i, -1, "Unode", seed))
            Li = (Ui * s[None, :]) @ V.T
        Z = rng_for(workload, matrix_id, i, step, "noise", seed).standard_normal((m, n))
        kind, c = w["noise"]
        if kind == "abs":
            Z *= c / np.sqrt(n)
        else:
            Z *= c * normL / np.linalg.norm(Z)
        G[i] = (Li + Z).astype(np.float32)
    return G


def init_Q(n, r, matrix_id=0, workload=0, seed=MASTER_SEED):
    """Initial auxiliary basis Q_{-1} ~ N(0,1), float32 [n, r], shared by all nodes."""
    return rng_for(workload, matrix_id, -1, -1, "Q", seed).standard_normal((n, r)).astype(np.float32)


def exact_rank_r(m, n, r, N, seed=MASTER_SEED):
    """One exactly-rank-r matrix replicated on N nodes, float32-representable factors."""
    rng = rng_for(0, 0, -1, -1, "misc", seed)
    A = np.round(rng.standard_normal((m, r)) * 8) / 8
    B = np.round(rng.standard_normal((r, n)) * 8) / 8
    G = (A @ B).astype(np.float32)
    return np.broadcast_to(G, (N, m, n)).copy()


# ---------------------------------------------------------------------------
# Device-side generation for the full-size workloads (benchmark, full-size
# parity).  torch is used purely as an allocator and random-number source.
# ---------------------------------------------------------------------------
def make_gradients_torch(workload, m, n, N, count, step, device, seed=MASTER_SEED, out=None):
    """float32 [count, N, m, n] on `device`, same recipe as make_gradients.

    The streams differ from the numpy generator's (different engine); full-size
    tests copy what they need back to the host, so both sides still see
    identical values.
    """
    import torch

    w = WORKLOADS[workload]
    g = torch.Generator(device=device)
    K = min(w["K"], n)
    s = torch.tensor(spectrum(w["spec"], K), dtype=torch.float32, device=device)
    if out is None:
        out = torch.empty((count, N, m, n), dtype=torch.float32, device=device)
    for c in range(count):
        g.manual_seed(seed * 1000003 + workload * 7919 + c * 31 + m)
        U = torch.linalg.qr(torch.randn((m, K), generator=g, device=device))[0]
        V = torch.linalg.qr(torch.randn((n, K), generator=g, device=device))[0]
        L = (U * s[None, :]) @ V.T
        normL = torch.linalg.norm(L)
        g.manual_seed(seed * 1000003 + workload * 7919 + c * 31 + m + 104729 * (step + 1))
        for i in range(N):
            Li = L
            if w["hetero"]:
                h = min(w["hetero"], K)
                gi = torch.Generator(device=device)
                gi.manual_seed(seed + 17 * c + 1009 * i + m)
                Ui = U.clone()
                Ui[:, :h] = torch.linalg.qr(torch.randn((m, h), generator=gi, device=device))[0]
                Li = (Ui * s[None, :]) @ V.T
            Z = torch.randn((m, n), generator=g, device=device)
            kind, cc = w["noise"]
            if kind == "abs":
                Z *= cc / np.sqrt(n)
            else:
                Z *= cc * normL / torch.linalg.norm(Z)
            out[c, i] = Li + Z
    return out
