"""ctypes binding of the C ABI in include/psgd.h (same names, argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))

PSGD_W_RANK_DEFICIENT = 1
PSGD_W_NOT_CONVERGED = 2
PSGD_W_TIMEOUT = 4
PSGD_OPT_ERROR_FORM, PSGD_OPT_MODE, PSGD_OPT_REFRESH_ITERS, PSGD_OPT_REFRESH_OVERSAMPLE, PSGD_OPT_REFRESH_TC = 1, 2, 3, 4, 5
PSGD_OPT_POWER_STEPS = 6
PSGD_OPT_REFRESH_ADAPTIVE = 7
PSGD_OPT_GRAD_BF16 = 8
PSGD_OPT_SINGLE_PASS = 9
PSGD_OPT_TRANSPOSED = 10
PSGD_OPT_PENDING_TC = 11
PSGD_OPT_BACKPROJECT_TMA = 12
PSGD_BUF = {"P_node": 1, "Q_node": 2, "P_hat": 3, "Dbar": 4, "P_mean": 5}
KERNEL_FAMILIES = ["project", "orth", "backproject", "residual", "refresh", "misc"]

_STATUS = {0: "PSGD_OK", -1: "PSGD_E_INVALID", -2: "PSGD_E_NULL", -3: "PSGD_E_WORKSPACE",
           -4: "PSGD_E_CUDA", -5: "PSGD_E_STATE", -6: "PSGD_E_TOO_LARGE"}

# every symbol include/psgd.h declares: name -> (restype, argtypes)
_vp, _i64, _u64, _int, _sz = C.c_void_p, C.c_int64, C.c_uint64, C.c_int, C.c_size_t
SIGNATURES = {
    "psgd_create": (_int, [_i64, _i64, _int, _int, _int, _u64, C.POINTER(_vp)]),
    "psgd_create_batch": (_int, [_i64, _i64, _int, _int, _int, _int, _u64, C.POINTER(_vp)]),
    "psgd_set_option": (_int, [_vp, _int, _int]),
    "psgd_sizes": (_int, [_vp, C.POINTER(_sz), C.POINTER(_sz), C.POINTER(_sz)]),
    "psgd_attach": (_int, [_vp, _vp, _vp, _vp, _sz]),
    "psgd_reset": (_int, [_vp, _vp]),
    "psgd_step": (_int, [_vp, _vp, _vp, _vp, _vp]),
    "psgd_refresh": (_int, [_vp, _vp, _vp, _vp, _vp]),
    "psgd_step_host": (_int, [_vp, _vp, _vp, _vp, _vp, _vp]),
    "psgd_msgd_update": (_int, [_vp, _vp, _vp, C.c_float, C.c_float, _vp]),
    "psgd_materialize_error": (_int, [_vp, _vp]),
    "psgd_state_written": (_int, [_vp]),
    "psgd_get_step": (_int, [_vp, C.POINTER(_i64)]),
    "psgd_set_step": (_int, [_vp, _i64]),
    "psgd_last_status": (_int, [_vp, _vp, C.POINTER(_int)]),
    "psgd_debug_ptr": (_int, [_vp, _int, C.POINTER(_vp), C.POINTER(_sz)]),
    "psgd_plan_info": (_int, [_vp, C.POINTER(_int)]),
    "psgd_launch_count": (_int, [_vp, C.POINTER(_i64)]),
    "psgd_profile_begin": (_int, [_vp]),
    "psgd_profile_read": (_int, [_vp, C.POINTER(C.c_float), C.POINTER(_int)]),
    "psgd_last_cuda_error": (C.c_char_p, [_vp]),
    "psgd_destroy": (_int, [_vp]),
    "psgd_gemm_nt_tf32_scratch": (_int, [_i64, _i64, _i64, _int, C.POINTER(_sz)]),
    "psgd_gemm_nt_tf32": (_int, [_vp, _vp, _vp, _i64, _i64, _i64, _int, _vp, _sz, _vp]),
    "psgd_backproject_static": (_int, [_vp, _vp, _vp, _vp, _i64, _i64, _int, _int, _vp]),
    "psgd_exchange_plan": (_int, [_vp, _int, C.POINTER(_int), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "psgd_exchange_begin": (_int, [_vp, _vp, _int, _vp, _vp]),
    "psgd_exchange_orth": (_int, [_vp, _vp, _vp, _vp]),
    "psgd_exchange_end": (_int, [_vp, _vp, _vp, _vp, _vp]),
    "psgd_group_create": (_int, [C.POINTER(_vp), _int, C.POINTER(_vp)]),
    "psgd_group_step": (_int, [_vp, C.POINTER(_vp), C.POINTER(_vp), _vp]),
    "psgd_group_destroy": (_int, [_vp]),
}


class PSGDError(RuntimeError):
    pass


def library_path():
    return os.path.join(HERE, "libpsgd.so")


_lib = None


def lib():
    """The loaded C library.  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise PSGDError(f"{path} is missing: build it with `python -m paper_2509_11254_b200.build`")
        L = C.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(code, h=None):
    if code != 0:
        msg = _STATUS.get(code, str(code))
        if code == -4 and h is not None:
            msg += ": " + lib().psgd_last_cuda_error(h).decode()
        raise PSGDError(msg)


class PowerSGDPlus:
    """`count` equally shaped m x n matrix variables on N simulated nodes (one GPU).

    Owns the torch tensors that back the library's caller-owned buffers:
    E [count,N,m,n], Q [count,n,r] and the workspace.
    """

    def __init__(self, m, n, r, N, refresh_period=0, seed=0, count=1, device="cuda:0", error_form="local",
                 mode="eager", refresh_iters=None, oversample=None, reset=True, refresh_tc=None, power_steps=None, refresh_adaptive=None,
                 grad_dtype="float32", single_pass=None, transposed=False, pending_tc=None, backproject_tma=None):
        import torch

        self.torch = torch
        self.m, self.n, self.r, self.N, self.count, self.tau = m, n, r, N, count, refresh_period
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise PSGDError("PowerSGDPlus needs a CUDA device; there is no CPU path")
        L = lib()
        h = _vp()
        _check(L.psgd_create_batch(m, n, r, N, count, refresh_period, seed, C.byref(h)))
        self.h = h
        _check(L.psgd_set_option(h, PSGD_OPT_ERROR_FORM, {"local": 0, "mean": 1}[error_form]))
        _check(L.psgd_set_option(h, PSGD_OPT_MODE, {"eager": 0, "deferred": 1}[mode]))
        if refresh_iters is not None:
            _check(L.psgd_set_option(h, PSGD_OPT_REFRESH_ITERS, refresh_iters))
        if oversample is not None:
            _check(L.psgd_set_option(h, PSGD_OPT_REFRESH_OVERSAMPLE, oversample))
        if refresh_tc is not None:
            _check(L.psgd_set_option(h, PSGD_OPT_REFRESH_TC, int(bool(refresh_tc))))
        if power_steps is not None:
            _check(L.psgd_set_option(h, PSGD_OPT_POWER_STEPS, int(power_steps)))
        if refresh_adaptive is not None:
            _check(L.psgd_set_option(h, PSGD_OPT_REFRESH_ADAPTIVE, int(bool(refresh_adaptive))))
        self.transposed = bool(transposed)
        if self.transposed:
            _check(L.psgd_set_option(h, PSGD_OPT_TRANSPOSED, 1))
        if single_pass is not None:
            _check(L.psgd_set_option(h, PSGD_OPT_SINGLE_PASS, {"auto": 0, "cluster": 1, "none": 2, "l2": 3}[single_pass]))
        if pending_tc is not None:      # "auto" | "always" | "never": which projection folds in the pending residual of the two-pass form
            _check(L.psgd_set_option(h, PSGD_OPT_PENDING_TC, {"auto": 0, "always": 1, "never": 2}[pending_tc]))
        if backproject_tma is not None:
            _check(L.psgd_set_option(h, PSGD_OPT_BACKPROJECT_TMA, int(bool(backproject_tma))))
        self.grad_dtype = {"float32": torch.float32, "bfloat16": torch.bfloat16}[grad_dtype]
        if self.grad_dtype is torch.bfloat16:
            _check(L.psgd_set_option(h, PSGD_OPT_GRAD_BF16, 1))
        eb, qb, wb = _sz(), _sz(), _sz()
        _check(L.psgd_sizes(h, C.byref(eb), C.byref(qb), C.byref(wb)))
        with torch.cuda.device(self.device):
            self.E = torch.empty((count, N, n, m) if self.transposed else (count, N, m, n), dtype=torch.float32, device=self.device)
            self.Q = torch.empty((count, n, r), dtype=torch.float32, device=self.device)
            self.ws = torch.empty((wb.value,), dtype=torch.uint8, device=self.device)
            self.P_hat = torch.empty((count, m, r), dtype=torch.float32, device=self.device)
            _check(L.psgd_attach(h, self.E.data_ptr(), self.Q.data_ptr(), self.ws.data_ptr(), wb.value), h)
            if reset:
                self.reset()

    # -- helpers ----------------------------------------------------------
    def _stream(self, stream=None):
        s = stream if stream is not None else self.torch.cuda.current_stream(self.device)
        return _vp(s.cuda_stream)

    def _g(self, G):
        t = self.torch
        if not (isinstance(G, t.Tensor) and G.is_cuda and G.dtype == self.grad_dtype and G.is_contiguous()):
            raise PSGDError(f"G must be a contiguous {self.grad_dtype} CUDA tensor")
        if G.numel() != self.count * self.N * self.m * self.n:
            raise PSGDError("G has the wrong number of elements")
        return G

    # -- the C ABI, one method per entry point ------------------------------
    def reset(self, stream=None):
        with self.torch.cuda.device(self.device):
            _check(lib().psgd_reset(self.h, self._stream(stream)), self.h)

    def step(self, G, D_hat=None, stream=None, force_refresh=False):
        G = self._g(G)
        fn = lib().psgd_refresh if force_refresh else lib().psgd_step
        with self.torch.cuda.device(self.device):
            _check(fn(self.h, G.data_ptr(), self.P_hat.data_ptr(), D_hat.data_ptr() if D_hat is not None else None,
                      self._stream(stream)), self.h)

    def refresh(self, G, D_hat=None, stream=None):
        self.step(G, D_hat, stream, force_refresh=True)

    def step_host(self, G_host, G_stage, P_hat_host=None, Q_host=None, stream=None):
        with self.torch.cuda.device(self.device):
            _check(lib().psgd_step_host(self.h, G_host.data_ptr(), G_stage.data_ptr(),
                                        P_hat_host.data_ptr() if P_hat_host is not None else None,
                                        Q_host.data_ptr() if Q_host is not None else None,
                                        self._stream(stream)), self.h)

    # One iteration with the nodes spread over several processes: the caller averages `first` and `second` over the
    # processes between the phases (exchange.ExchangedStack does, with torch.distributed).
    def exchange_plan(self, force_refresh=False):
        """(refresh, first_floats, second_floats) of the next step."""
        rf, a, b = _int(), C.c_size_t(), C.c_size_t()
        _check(lib().psgd_exchange_plan(self.h, int(bool(force_refresh)), C.byref(rf), C.byref(a), C.byref(b)))
        return bool(rf.value), a.value, b.value

    def _slot(self, t, floats):
        tt = self.torch
        if not (isinstance(t, tt.Tensor) and t.is_cuda and t.dtype == tt.float32 and t.is_contiguous() and t.numel() >= floats):
            raise PSGDError(f"an exchange array must be a contiguous float32 CUDA tensor of at least {floats} elements")
        return t.data_ptr()

    def exchange_begin(self, G, first, force_refresh=False, stream=None):
        G = self._g(G)
        floats = self.exchange_plan(force_refresh)[1]
        with self.torch.cuda.device(self.device):
            _check(lib().psgd_exchange_begin(self.h, G.data_ptr(), int(bool(force_refresh)), self._slot(first, floats),
                                             self._stream(stream)), self.h)

    def exchange_orth(self, first, second, stream=None):
        _, a, b = self.exchange_plan()
        with self.torch.cuda.device(self.device):
            _check(lib().psgd_exchange_orth(self.h, self._slot(first, a), self._slot(second, b), self._stream(stream)), self.h)

    def exchange_end(self, second, D_hat=None, stream=None):
        b = self.exchange_plan()[2]
        with self.torch.cuda.device(self.device):
            _check(lib().psgd_exchange_end(self.h, self._slot(second, b), self.P_hat.data_ptr(),
                                           D_hat.data_ptr() if D_hat is not None else None, self._stream(stream)), self.h)

    def msgd_update(self, X, mom, eta, mu, stream=None):
        """Eq. (7c) with the reconstruction of the last step: mom <- mu mom + P~ Q^T, X <- X - eta mom (in place)."""
        t = self.torch
        for a in (X, mom):
            if not (isinstance(a, t.Tensor) and a.is_cuda and a.dtype == t.float32 and a.is_contiguous()
                    and a.numel() == self.count * self.m * self.n):
                raise PSGDError("X and mom must be contiguous float32 CUDA tensors of count*m*n elements")
        with t.cuda.device(self.device):
            _check(lib().psgd_msgd_update(self.h, X.data_ptr(), mom.data_ptr(), float(eta), float(mu), self._stream(stream)), self.h)

    def materialize_error(self, stream=None):
        with self.torch.cuda.device(self.device):
            _check(lib().psgd_materialize_error(self.h, self._stream(stream)), self.h)

    def set_state(self, E=None, Q=None, t=None):
        """Overwrite the persistent state (e_t, Q_{t-1}, t) from host or device arrays."""
        tc = self.torch
        if E is not None:
            self.E.copy_(tc.as_tensor(E, dtype=tc.float32).reshape(self.E.shape))
        if Q is not None:
            self.Q.copy_(tc.as_tensor(Q, dtype=tc.float32).reshape(self.Q.shape))
        _check(lib().psgd_state_written(self.h))
        if t is not None:
            _check(lib().psgd_set_step(self.h, int(t)))

    @property
    def t(self):
        v = _i64()
        _check(lib().psgd_get_step(self.h, C.byref(v)))
        return v.value

    def last_status(self, stream=None):
        v = _int()
        with self.torch.cuda.device(self.device):
            _check(lib().psgd_last_status(self.h, self._stream(stream), C.byref(v)), self.h)
        return v.value

    def debug(self, name):
        """Copy of an internal buffer as a torch tensor (test hook)."""
        tc = self.torch
        p, b = _vp(), _sz()
        _check(lib().psgd_debug_ptr(self.h, PSGD_BUF[name], C.byref(p), C.byref(b)))
        off = p.value - self.ws.data_ptr()
        flat = self.ws[off:off + b.value].view(tc.float32)
        shape = {"P_node": (self.count, self.N, self.m, self.r), "Q_node": (self.count, self.N, self.n, self.r),
                 "P_hat": (self.count, self.m, self.r), "Dbar": (self.count, self.m, self.n),
                 "P_mean": (self.count, self.m, self.r)}[name]
        return flat.view(shape).clone()

    def plan_info(self):
        v = (_int * 12)()
        _check(lib().psgd_plan_info(self.h, v))
        keys = ("single_pass", "RP", "WC", "CS", "KC", "active_clusters", "smem_bytes", "S", "pending", "pending_single_pass",
                "sm_count", "step_kernel")
        return dict(zip(keys, list(v)))

    def launch_count(self):
        v = _i64()
        _check(lib().psgd_launch_count(self.h, C.byref(v)))
        return v.value

    def profile_begin(self):
        _check(lib().psgd_profile_begin(self.h))

    def profile_read(self):
        ms = (C.c_float * len(KERNEL_FAMILIES))()
        ln = (_int * len(KERNEL_FAMILIES))()
        _check(lib().psgd_profile_read(self.h, ms, ln), self.h)
        return {k: (ms[i], ln[i]) for i, k in enumerate(KERNEL_FAMILIES)}

    def close(self):
        if getattr(self, "h", None) is not None and self.h.value:
            lib().psgd_destroy(self.h)
            self.h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class StepGroup:
    """Handles of different shapes stepped by one call (psgd_group_*): each on a stream of the group's own,
    forked from and joined into the caller's stream."""

    def __init__(self, handles):
        import torch

        self.torch = torch
        self.handles = list(handles)
        arr = (_vp * len(self.handles))(*[h.h for h in self.handles])
        g = _vp()
        with torch.cuda.device(self.handles[0].device):
            _check(lib().psgd_group_create(arr, len(self.handles), C.byref(g)))
        self.g = g

    def step(self, G_list, stream=None):
        hs = self.handles
        Gs = (_vp * len(hs))(*[h._g(g).data_ptr() for h, g in zip(hs, G_list)])
        Ps = (_vp * len(hs))(*[h.P_hat.data_ptr() for h in hs])
        with self.torch.cuda.device(hs[0].device):
            _check(lib().psgd_group_step(self.g, Gs, Ps, hs[0]._stream(stream)))

    def close(self):
        if getattr(self, "g", None) is not None and self.g.value:
            lib().psgd_group_destroy(self.g)
            self.g = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def gemm_nt_tf32(A, B, stream=None):
    """C[c] = A[c] @ B[c].T on the tensor cores (TF32 operands, float32 accumulation).

    A [count,M,K], B [count,Nc,K]: contiguous float32 CUDA tensors.  Returns C [count,M,Nc].
    """
    import torch

    count, M, K = A.shape
    Nc = B.shape[1]
    for t in (A, B):
        if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
            raise PSGDError("tensors must be contiguous float32 CUDA tensors")
    nb = _sz()
    _check(lib().psgd_gemm_nt_tf32_scratch(M, Nc, K, count, C.byref(nb)))
    s = stream if stream is not None else torch.cuda.current_stream(A.device)
    with torch.cuda.device(A.device):
        scratch = torch.empty((nb.value,), dtype=torch.uint8, device=A.device)
        out = torch.empty((count, M, Nc), dtype=torch.float32, device=A.device)
        _check(lib().psgd_gemm_nt_tf32(A.data_ptr(), B.data_ptr(), out.data_ptr(), M, Nc, K, count,
                                       scratch.data_ptr(), nb.value, _vp(s.cuda_stream)))
    return out


def backproject_static(M, P_hat, Q_mean, Q_node=None, stream=None):
    """Q_node[i] = M[i]^T P_hat and their mean, through the entry point that allocates nothing.

    M [N,m,n], P_hat [m,r], Q_mean [n,r], Q_node [N,n,r] or None: contiguous float32 CUDA tensors
    owned by the caller.  Raises PSGDError(PSGD_E_TOO_LARGE) when N*n*r*4 exceeds the fixed scratch.
    """
    import torch

    N, m, n = M.shape
    r = P_hat.shape[1]
    for t in (M, P_hat, Q_mean) + ((Q_node,) if Q_node is not None else ()):
        if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
            raise PSGDError("tensors must be contiguous float32 CUDA tensors")
    s = stream if stream is not None else torch.cuda.current_stream(M.device)
    with torch.cuda.device(M.device):
        _check(lib().psgd_backproject_static(M.data_ptr(), P_hat.data_ptr(),
                                             Q_node.data_ptr() if Q_node is not None else None,
                                             Q_mean.data_ptr(), m, n, r, N, _vp(s.cuda_stream)))
