"""ctypes binding of libsolon.so: same names as the C interface (include/solon.h), marshalling only.

Torch is used for device memory and streams; every step of the path runs in the library's kernels.
The library is loaded on first use and a missing build raises: there is no fallback of any kind.
"""

from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_double, c_float, c_int, c_int64, c_uint8, c_uint64, c_void_p

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsolon.so")

OK = 0
ERR_INVALID_ARG = -1
ERR_INFEASIBLE = -2
ERR_CUDA = -3
ERR_UNDECODABLE = -4
ERR_INTERNAL = -5
ERR_NOMEM = -6
F32 = 0
F64 = 1

# name -> (restype, argtypes); every symbol the header declares
SIGNATURES = {
    "solon_check_params": (c_int, [c_int, c_int, c_int, c_int, c_int64]),
    "solon_group_layout": (c_int, [c_int, c_int, POINTER(c_int), c_int, POINTER(c_int)]),
    "solon_node_scalars": (c_int, [c_int, c_int, POINTER(c_double)]),
    "solon_locate_host": (c_int, [c_int, c_int, c_int, c_int, POINTER(c_double), POINTER(c_double), POINTER(c_double),
                                  c_double, POINTER(c_uint8), POINTER(c_int), POINTER(c_int), POINTER(c_int),
                                  POINTER(c_double)]),
    "solon_strerror": (c_char_p, [c_int]),
    "solon_plan_create": (c_int, [c_int, c_int, c_int, c_int, c_int64, c_uint64, POINTER(c_void_p)]),
    "solon_plan_create_ex": (c_int, [c_int, c_int, c_int, c_int, c_int64, c_uint64, c_int, POINTER(c_void_p)]),
    "solon_float64_m_supported": (c_int, [c_int]),
    "solon_plan_dtype": (c_int, [c_void_p]),
    "solon_plan_destroy": (c_int, [c_void_p]),
    "solon_plan_set_stream": (c_int, [c_void_p, c_void_p]),
    "solon_plan_set_num_projections": (c_int, [c_void_p, c_int]),
    "solon_plan_reseed": (c_int, [c_void_p, c_uint64]),
    "solon_plan_set_fresh_projections": (c_int, [c_void_p, c_int]),
    "solon_plan_set_tolerance": (c_int, [c_void_p, c_double]),
    "solon_plan_set_early_locator": (c_int, [c_void_p, c_int]),
    "solon_plan_set_optimistic": (c_int, [c_void_p, c_int]),
    "solon_plan_get_optimistic_outcome": (c_int, [c_void_p, POINTER(c_int)]),
    "solon_plan_set_lsq_rows": (c_int, [c_void_p, c_int]),
    "solon_plan_dc": (c_int64, [c_void_p]),
    "solon_plan_num_groups": (c_int, [c_void_p]),
    "solon_plan_group_of": (c_int, [c_void_p, c_int]),
    "solon_plan_group_start": (c_int, [c_void_p, c_int]),
    "solon_plan_group_size": (c_int, [c_void_p, c_int]),
    "solon_plan_num_projections": (c_int, [c_void_p]),
    "solon_plan_get_node_scalars": (c_int, [c_void_p, POINTER(c_double)]),
    "solon_plan_get_projection_vectors": (c_int, [c_void_p, POINTER(c_float)]),
    "solon_encode": (c_int, [c_void_p, c_void_p, c_void_p]),
    "solon_decode": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p]),
    "solon_encode_f64": (c_int, [c_void_p, c_void_p, c_void_p]),
    "solon_decode_f64": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p]),
    "solon_overwrite_rows_f64": (c_int, [c_void_p, c_void_p, c_int, c_void_p, c_void_p]),
    "solon_step_host_f64": (c_int, [c_void_p, c_void_p, c_int, POINTER(c_int), c_void_p, c_void_p, c_void_p]),
    "solon_decode_status": (c_int, [c_void_p]),
    "solon_plan_status": (c_int, [c_void_p]),
    "solon_decode_project": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p]),
    "solon_decode_finish": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "solon_lsq_grads": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "solon_overwrite_rows": (c_int, [c_void_p, c_void_p, c_int, c_void_p, c_void_p]),
    "solon_step_host": (c_int, [c_void_p, c_void_p, c_int, POINTER(c_int), c_void_p, c_void_p, c_void_p]),
    "solon_plan_get_projections": (c_int, [c_void_p, POINTER(c_double), POINTER(c_double)]),
    "solon_plan_get_recovery": (c_int, [c_void_p, POINTER(c_int), POINTER(c_int), POINTER(c_int), POINTER(c_double)]),
    "solon_plan_get_early_outcome": (c_int, [c_void_p, POINTER(c_int)]),
    "solon_plan_kernel_launches": (c_int64, [c_void_p]),
    "solon_plan_set_profiling": (c_int, [c_void_p, c_int]),
    "solon_plan_get_timings": (c_int, [c_void_p, POINTER(c_float)]),
    "solon_project_noalloc": (c_int, [c_void_p, c_void_p, c_int64, c_int, c_int64, c_int, c_void_p, c_void_p, c_void_p]),
}

_lib = None


class SolonError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} ({status})")


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it has not been built (python -m paper_2110_01595_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2110_01595_b200.build`")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (restype, argtypes) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = restype
            fn.argtypes = argtypes
        _lib = handle
    return _lib


def strerror(status: int) -> str:
    return lib().solon_strerror(status).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise SolonError(status, where)


def _dptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(POINTER(ctype))


# ------------------------------------------------------------------ plan-free helpers


def solon_check_params(P: int, s: int, m: int, r: int, d: int) -> int:
    return lib().solon_check_params(P, s, m, r, d)


def solon_group_layout(P: int, r: int) -> list[int]:
    starts = np.zeros(P + 2, dtype=np.int32)
    q = c_int(0)
    _check(lib().solon_group_layout(P, r, _dptr(starts, c_int), len(starts), byref(q)), "solon_group_layout")
    return starts[:q.value + 1].tolist()


def solon_node_scalars(P: int, r: int) -> np.ndarray:
    w = np.zeros(P, dtype=np.float64)
    _check(lib().solon_node_scalars(P, r, _dptr(w, c_double)), "solon_node_scalars")
    return w


def solon_locate_host(rho: np.ndarray, nu: np.ndarray, w_g: np.ndarray, m: int, s: int, tau: float):
    """Host mirror of the device locator for one group.  Returns (status, mask, t, rec_rows, coeff[n_rec, m])."""
    rho = np.ascontiguousarray(np.atleast_2d(rho), dtype=np.float64)
    nu = np.ascontiguousarray(nu, dtype=np.float64)
    w_g = np.ascontiguousarray(w_g, dtype=np.float64)
    K, n = rho.shape
    mask = np.zeros(n, dtype=np.uint8)
    rows = np.zeros(n, dtype=np.int32)
    coeff = np.zeros(n * m, dtype=np.float64)
    t = c_int(0)
    n_rec = c_int(0)
    status = lib().solon_locate_host(n, m, s, K, _dptr(rho, c_double), _dptr(nu, c_double), _dptr(w_g, c_double), tau,
                                     _dptr(mask, c_uint8), byref(t), _dptr(rows, c_int), byref(n_rec),
                                     _dptr(coeff, c_double))
    if status not in (OK, ERR_UNDECODABLE):
        raise SolonError(status, "solon_locate_host")
    return status, mask, t.value, rows[:n_rec.value].copy(), coeff[:n_rec.value * m].reshape(n_rec.value, m).copy()


def solon_project_noalloc(received, f, rho, nu, stream=None) -> int:
    """Projections through the entry point that allocates nothing.

    received: P x d_c float32 CUDA tensor; f: K x f_pitch float32 CUDA tensor (f_pitch >= d_c, multiple of 4);
    rho (K x P) and nu (P): float64 CUDA tensors the caller has already allocated.  Returns the status code.
    """
    import torch

    P, d_c = received.shape
    K, f_pitch = f.shape
    for t, dt in ((received, torch.float32), (f, torch.float32), (rho, torch.float64), (nu, torch.float64)):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == dt):
            raise ValueError("solon_project_noalloc takes contiguous CUDA tensors (float32 in, float64 out)")
    if tuple(rho.shape) != (K, P) or tuple(nu.shape) != (P,):
        raise ValueError("rho must be K x P and nu must have P entries")
    stream = stream if stream is not None else torch.cuda.current_stream()
    return lib().solon_project_noalloc(c_void_p(received.data_ptr()), c_void_p(f.data_ptr()), f_pitch, P, d_c, K,
                                       c_void_p(rho.data_ptr()), c_void_p(nu.data_ptr()), c_void_p(stream.cuda_stream))


# ------------------------------------------------------------------ plan


class Plan:
    """Owner of a solon_plan*.  Methods mirror the C calls; tensors are torch CUDA tensors (float32, contiguous)."""

    def __init__(self, P: int, s: int, m: int, r: int, d: int, seed: int = 0, stream=None, dtype: str = "f32"):
        import torch

        self._torch = torch
        if dtype not in ("f32", "f64"):
            raise ValueError("dtype must be 'f32' or 'f64'")
        self.dtype = dtype
        self.tdtype = torch.float64 if dtype == "f64" else torch.float32     # element type of gradients, coded vectors, aggregate
        handle = c_void_p()
        _check(lib().solon_plan_create_ex(P, s, m, r, d, seed, F64 if dtype == "f64" else F32, byref(handle)), "solon_plan_create_ex")
        self._h = handle
        self.P, self.s, self.m, self.r, self.d = P, s, m, r, d
        self.d_c = int(lib().solon_plan_dc(self._h))
        self.q = int(lib().solon_plan_num_groups(self._h))
        self.set_stream(stream if stream is not None else torch.cuda.current_stream())

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib().solon_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- configuration
    def set_stream(self, stream) -> None:
        raw = stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)
        _check(lib().solon_plan_set_stream(self._h, c_void_p(raw)), "solon_plan_set_stream")
        self.stream_handle = int(raw)      # the cudaStream_t the plan's calls enqueue on

    def set_num_projections(self, K: int) -> None:
        _check(lib().solon_plan_set_num_projections(self._h, K), "solon_plan_set_num_projections")

    def reseed(self, seed: int) -> None:
        _check(lib().solon_plan_reseed(self._h, seed), "solon_plan_reseed")

    def set_fresh_projections(self, on: bool) -> None:
        """True: every decode projects with projection vectors no earlier decode used; False (default): the ones in memory
        are reused until reseed()."""
        _check(lib().solon_plan_set_fresh_projections(self._h, 1 if on else 0), "solon_plan_set_fresh_projections")

    def set_tolerance(self, tau: float) -> None:
        _check(lib().solon_plan_set_tolerance(self._h, tau), "solon_plan_set_tolerance")

    def set_early_locator(self, mode: int) -> None:
        """0: never start the locator on a partial projection; 1 (default): when the projection pass is long; 2: always;
        3: diagnostic, the locator's wait for the partial sums runs out (outcome 3), results unchanged."""
        _check(lib().solon_plan_set_early_locator(self._h, mode), "solon_plan_set_early_locator")

    def set_optimistic(self, mode: int) -> None:
        """0: the projection pass never recovers the aggregate itself; 1 (default): it does so, from the rows of the previous
        decode's recovery table, when in each of the last two decodes the table of the decode before would have served; 2: always.  The recovery
        kernel is skipped when the locator finds those rows trusted in this decode."""
        _check(lib().solon_plan_set_optimistic(self._h, mode), "solon_plan_set_optimistic")

    def optimistic_outcome(self) -> bool:
        """True if the recovery kernel of the most recent decode had nothing to do."""
        out = c_int(0)
        _check(lib().solon_plan_get_optimistic_outcome(self._h, byref(out)), "solon_plan_get_optimistic_outcome")
        return bool(out.value)

    def early_outcome(self) -> np.ndarray:
        """Per group: 0 no early run, 1 early answer confirmed, 2 not confirmed, 3 wait expired (last decode)."""
        out = np.zeros(self.q, dtype=np.int32)
        _check(lib().solon_plan_get_early_outcome(self._h, _dptr(out, c_int)), "solon_plan_get_early_outcome")
        return out

    def set_lsq_rows(self, rows: int) -> None:
        _check(lib().solon_plan_set_lsq_rows(self._h, rows), "solon_plan_set_lsq_rows")

    # -- queries
    @property
    def K(self) -> int:
        return int(lib().solon_plan_num_projections(self._h))

    def group_starts(self) -> list[int]:
        starts = [lib().solon_plan_group_start(self._h, g) for g in range(self.q)]
        return starts + [self.P]

    def group_sizes(self) -> list[int]:
        return [lib().solon_plan_group_size(self._h, g) for g in range(self.q)]

    def group_of(self, node: int) -> int:
        return lib().solon_plan_group_of(self._h, node)

    def node_scalars(self) -> np.ndarray:
        w = np.zeros(self.P, dtype=np.float64)
        _check(lib().solon_plan_get_node_scalars(self._h, _dptr(w, c_double)), "solon_plan_get_node_scalars")
        return w

    def projection_vectors(self) -> np.ndarray:
        f = np.zeros((self.K, self.d_c), dtype=np.float32)
        _check(lib().solon_plan_get_projection_vectors(self._h, _dptr(f, c_float)), "solon_plan_get_projection_vectors")
        return f

    def set_profiling(self, on: bool) -> None:
        _check(lib().solon_plan_set_profiling(self._h, 1 if on else 0), "solon_plan_set_profiling")

    def timings(self) -> dict:
        """Milliseconds of the most recent encode / projection / locator / recovery kernels (profiling on)."""
        ms = np.zeros(4, dtype=np.float32)
        _check(lib().solon_plan_get_timings(self._h, _dptr(ms, c_float)), "solon_plan_get_timings")
        return {"encode": float(ms[0]), "project": float(ms[1]), "locate": float(ms[2]), "recover": float(ms[3])}

    def kernel_launches(self) -> int:
        return int(lib().solon_plan_kernel_launches(self._h))

    # -- hot path
    def _dev(self, t, shape, dtype=None):
        dtype = dtype or self.tdtype
        if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype and tuple(t.shape) == tuple(shape)):
            raise ValueError(f"expected a contiguous CUDA {dtype} tensor of shape {tuple(shape)}, got {tuple(t.shape)} {t.dtype}")
        return c_void_p(t.data_ptr())

    def encode(self, partition_grads, coded=None):
        torch = self._torch
        if coded is None:
            coded = torch.empty((self.P, self.d_c), dtype=self.tdtype, device=partition_grads.device)
        fn = lib().solon_encode_f64 if self.dtype == "f64" else lib().solon_encode
        _check(fn(self._h, self._dev(partition_grads, (self.P, self.d)), self._dev(coded, (self.P, self.d_c))),
               "solon_encode")
        return coded

    def decode(self, received, agg_grad=None, byz_mask=None):
        torch = self._torch
        if agg_grad is None:
            agg_grad = torch.empty(self.d, dtype=self.tdtype, device=received.device)
        if byz_mask is None:
            byz_mask = torch.empty(self.P, dtype=torch.uint8, device=received.device)
        fn = lib().solon_decode_f64 if self.dtype == "f64" else lib().solon_decode
        _check(fn(self._h, self._dev(received, (self.P, self.d_c)), self._dev(agg_grad, (self.d,)),
                                  self._dev(byz_mask, (self.P,), torch.uint8)), "solon_decode")
        return agg_grad, byz_mask

    def decode_project(self, received, rho, nu):
        """First half of the decode: rho (K x P) and nu (P), float64 device tensors, receive this plan's projections."""
        torch = self._torch
        _check(lib().solon_decode_project(self._h, self._dev(received, (self.P, self.d_c)),
                                          self._dev(rho, (self.K, self.P), torch.float64),
                                          self._dev(nu, (self.P,), torch.float64)), "solon_decode_project")
        return rho, nu

    def decode_finish(self, rho, nu, received, agg_grad=None, byz_mask=None):
        """Second half: locator and recovery from the given (summed) projections."""
        torch = self._torch
        if agg_grad is None:
            agg_grad = torch.empty(self.d, dtype=torch.float32, device=received.device)
        if byz_mask is None:
            byz_mask = torch.empty(self.P, dtype=torch.uint8, device=received.device)
        _check(lib().solon_decode_finish(self._h, self._dev(rho, (self.K, self.P), torch.float64),
                                         self._dev(nu, (self.P,), torch.float64),
                                         self._dev(received, (self.P, self.d_c)), self._dev(agg_grad, (self.d,)),
                                         self._dev(byz_mask, (self.P,), torch.uint8)), "solon_decode_finish")
        return agg_grad, byz_mask

    def overwrite_rows(self, matrix, nodes, rows):
        """matrix[nodes[i]] = rows[i] on the plan's stream (the adversary of a device-resident simulation).
        nodes: int32 CUDA tensor; rows: len(nodes) x d_c float32 CUDA tensor."""
        torch = self._torch
        n = int(nodes.numel())
        if n == 0:
            return matrix
        fn = lib().solon_overwrite_rows_f64 if self.dtype == "f64" else lib().solon_overwrite_rows
        _check(fn(self._h, self._dev(matrix, (self.P, self.d_c)), n, self._dev(nodes, (n,), torch.int32),
                                          self._dev(rows, (n, self.d_c))), "solon_overwrite_rows")
        return matrix

    def decode_status(self) -> int:
        return lib().solon_decode_status(self._h)

    def status(self) -> int:
        """solon_plan_status: OK, or ERR_INTERNAL once a bounded wait inside one of the plan's kernels has run out."""
        return lib().solon_plan_status(self._h)

    def lsq_grads(self, X, y, w, grads=None, rows: int | None = None):
        torch = self._torch
        if rows is not None:
            self.set_lsq_rows(rows)
        n = X.shape[0]
        if grads is None:
            grads = torch.empty((self.P, self.d), dtype=torch.float32, device=X.device)
        _check(lib().solon_lsq_grads(self._h, self._dev(X, (n, self.d)), self._dev(y, (n,)), self._dev(w, (self.d,)),
                                     self._dev(grads, (self.P, self.d))), "solon_lsq_grads")
        return grads

    def step_host(self, grads_host, byz_nodes, byz_rows_host, agg_host, mask_host) -> int:
        """solon_step_host: host tensors in (ideally pinned), host tensors out; returns the decode status."""
        torch = self._torch
        for t in (grads_host, agg_host, mask_host):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("solon_step_host takes contiguous host tensors")
        n_byz = len(byz_nodes)
        nodes = np.asarray(byz_nodes, dtype=np.int32)
        rows_ptr = c_void_p(byz_rows_host.data_ptr()) if n_byz else c_void_p(0)
        fn = lib().solon_step_host_f64 if self.dtype == "f64" else lib().solon_step_host
        return fn(self._h, c_void_p(grads_host.data_ptr()), n_byz,
                                     _dptr(nodes, c_int) if n_byz else None, rows_ptr,
                                     c_void_p(agg_host.data_ptr()), c_void_p(mask_host.data_ptr()))

    # -- introspection of the last decode
    def projections(self):
        rho = np.zeros((self.K, self.P), dtype=np.float64)
        nu = np.zeros(self.P, dtype=np.float64)
        _check(lib().solon_plan_get_projections(self._h, _dptr(rho, c_double), _dptr(nu, c_double)), "solon_plan_get_projections")
        return rho, nu

    def recovery(self):
        """Returns (n_rec[q], t[q], rec_rows (concatenated), coeff (sum n_rec x m))."""
        n_rec = np.zeros(self.q, dtype=np.int32)
        t = np.zeros(self.q, dtype=np.int32)
        rows = np.zeros(self.P, dtype=np.int32)
        coeff = np.zeros(self.P * self.m, dtype=np.float64)
        _check(lib().solon_plan_get_recovery(self._h, _dptr(n_rec, c_int), _dptr(t, c_int), _dptr(rows, c_int),
                                             _dptr(coeff, c_double)), "solon_plan_get_recovery")
        total = int(n_rec.sum())
        return n_rec, t, rows[:total].copy(), coeff[:total * self.m].reshape(total, self.m).copy()


# C-named aliases for callers that prefer the flat interface
def solon_plan_create(P, s, m, r, d, seed=0) -> Plan:
    return Plan(P, s, m, r, d, seed)


def solon_encode(plan: Plan, partition_grads, coded=None):
    return plan.encode(partition_grads, coded)


def solon_decode(plan: Plan, received, agg_grad=None, byz_mask=None):
    return plan.decode(received, agg_grad, byz_mask)


def solon_lsq_grads(plan: Plan, X, y, w, grads=None):
    return plan.lsq_grads(X, y, w, grads)
