"""Nodes spread over processes, on CPU: two gloo ranks, each holding two of four nodes, against the oracle on all four.

`ExchangedStack` lays the arrays that Algorithm 2 averages over the nodes (P, Q and, at a refresh, the error-compensated
gradient) into one flat buffer per exchange and all-reduces it.  Here the handles are CPU stand-ins with the same four
`exchange_*` methods, doing each phase with the oracle's own routines in double precision, so that the test covers what
the module adds: the slot layout, the order of the phases, the mean over processes with equal node counts, and that
several handles (different shapes, one a refresh step while the other is not) share one exchange.
"""
import os
import socket
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

SHAPES = [(48, 20, 3, 3), (33, 33, 5, 0)]     # (m, n, r, tau): the first refreshes at t = 0 and 3, the second never
N_TOTAL, STEPS = 4, 5


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _gradients(shape_id, step):
    m, n, _, _ = SHAPES[shape_id]
    rng = np.random.default_rng(1000 * shape_id + step)
    low = rng.standard_normal((N_TOTAL, m, 4)) @ rng.standard_normal((4, n))
    return low + 0.1 * rng.standard_normal((N_TOTAL, m, n))


def _q0(shape_id):
    _, n, r, _ = SHAPES[shape_id]
    return np.random.default_rng(77 + shape_id).standard_normal((n, r))


class _StubHandle:
    """The local nodes of one matrix on CPU; every phase uses the oracle's routines on float64 arrays."""

    def __init__(self, orc, torch, m, n, r, nodes, tau, Q0):
        self.orc, self.torch = orc, torch
        self.m, self.n, self.r, self.N, self.tau = m, n, r, nodes, tau
        self.device = "cpu"
        self.t = 0
        self.Q = np.array(Q0, dtype=np.float64)
        self.E = np.zeros((nodes, m, n))
        self.phase = 0

    def exchange_plan(self, force_refresh=False):
        rf = self.refresh if self.phase else (bool(force_refresh) or (self.tau > 0 and self.t % self.tau == 0))
        return rf, self.m * (self.n if rf else self.r), self.n * self.r

    def exchange_begin(self, G, first, force_refresh=False):
        assert self.phase == 0
        self.refresh = self.exchange_plan(force_refresh)[0]
        self.M = np.asarray(G, dtype=np.float64) + self.E
        local = self.M.mean(axis=0) if self.refresh else np.stack([Mi @ self.Q for Mi in self.M]).mean(axis=0)
        first.copy_(self.torch.from_numpy(local.reshape(-1)))
        self.phase = 1

    def exchange_orth(self, first, second):
        assert self.phase == 1
        X = first.numpy().astype(np.float64)
        if self.refresh:
            self.P_hat = self.orc.svd_top_r(X.reshape(self.m, self.n), self.r)[0]
        else:
            self.P_hat = self.orc.qr_orth(X.reshape(self.m, self.r))
        self.Q_i = np.stack([Mi.T @ self.P_hat for Mi in self.M])
        second.copy_(self.torch.from_numpy(self.Q_i.mean(axis=0).reshape(-1)))
        self.phase = 2

    def exchange_end(self, second):
        assert self.phase == 2
        self.Q = second.numpy().astype(np.float64).reshape(self.n, self.r).copy()
        self.E = self.M - np.stack([self.P_hat @ Qi.T for Qi in self.Q_i])
        self.phase = 0
        self.t += 1


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import torch
    import torch.distributed as dist

    from oracle import psgd_oracle as orc
    from paper_2509_11254_b200.exchange import ExchangedStack

    dist.init_process_group("gloo")
    per = N_TOTAL // world
    mine = slice(rank * per, (rank + 1) * per)
    hs = [_StubHandle(orc, torch, m, n, r, per, tau, _q0(i)) for i, (m, n, r, tau) in enumerate(SHAPES)]
    stack = ExchangedStack(hs, device="cpu", dtype=torch.float64)      # the stand-ins work in double
    refreshes = []
    for step in range(STEPS):
        refreshes.append(stack.step([_gradients(i, step)[mine] for i in range(len(SHAPES))]))
    res = dict(rank=rank, refreshes=refreshes, exchanges=stack.exchanges,
               Q=[h.Q for h in hs], P_hat=[h.P_hat for h in hs], E=[h.E for h in hs])
    dist.barrier()
    dist.destroy_process_group()
    out.put(res)


def test_slot_offsets_are_aligned_and_disjoint():
    from paper_2509_11254_b200.exchange import ALIGN_FLOATS, slot_offsets

    sizes = [1, 64, 65, 0, 1000, 3]
    offs, total = slot_offsets(sizes)
    assert all(o % ALIGN_FLOATS == 0 for o in offs) and total % ALIGN_FLOATS == 0
    ends = [o + s for o, s in zip(offs, sizes)]
    assert all(e <= o2 for e, o2 in zip(ends, offs[1:])) and ends[-1] <= total
    assert offs == [0, 64, 128, 256, 256, 1280] and total == 1344
    assert slot_offsets([]) == ([], 0)
    with pytest.raises(ValueError):
        slot_offsets([4, -1])


def test_two_gloo_ranks_equal_the_oracle_on_all_nodes():
    import torch.multiprocessing as mp

    from oracle import psgd_oracle as orc

    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((out.get(timeout=180) for _ in procs), key=lambda d: d["rank"])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the whole job in one process: Algorithm 2 on all four nodes
    oracles = [orc.PowerSGDPlusOracle(m, n, r, N_TOTAL, tau, _q0(i)) for i, (m, n, r, tau) in enumerate(SHAPES)]
    expect_refresh = []
    for step in range(STEPS):
        outs = [o.step(_gradients(i, step)) for i, o in enumerate(oracles)]
        expect_refresh.append([bool(o["refresh"]) for o in outs])
    per = N_TOTAL // 2
    for d in res:
        assert d["refreshes"] == expect_refresh and d["exchanges"] == 2 * STEPS
        for i, o in enumerate(oracles):
            assert np.allclose(d["Q"][i], o.Q, rtol=0, atol=1e-10 * np.abs(o.Q).max())
            mine = slice(d["rank"] * per, (d["rank"] + 1) * per)
            assert np.allclose(d["E"][i], o.E[mine], rtol=0, atol=1e-10 * np.abs(o.E).max())
            P = outs[i]["P_hat"]
            assert np.allclose(d["P_hat"][i] @ d["P_hat"][i].T, P @ P.T, atol=1e-10)
    # both ranks hold the same Q and P~ bit for bit (same averaged input, same deterministic routine)
    for i in range(len(SHAPES)):
        assert np.array_equal(res[0]["Q"][i], res[1]["Q"][i]) and np.array_equal(res[0]["P_hat"][i], res[1]["P_hat"][i])


def test_single_process_needs_no_process_group():
    import torch

    from oracle import psgd_oracle as orc
    from paper_2509_11254_b200.exchange import ExchangedStack

    m, n, r, tau = SHAPES[0]
    h = _StubHandle(orc, torch, m, n, r, N_TOTAL, tau, _q0(0))
    stack = ExchangedStack([h], device="cpu", dtype=torch.float64)
    o = orc.PowerSGDPlusOracle(m, n, r, N_TOTAL, tau, _q0(0))
    for step in range(4):
        stack.step([_gradients(0, step)])
        o.step(_gradients(0, step))
        assert np.allclose(h.Q, o.Q, atol=1e-10 * np.abs(o.Q).max()) and np.allclose(h.E, o.E, atol=1e-10)
    assert stack.world == 1 and stack.exchanges == 8
