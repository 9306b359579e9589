"""ctypes binding of the CORE C ABI (``include/core.h``): argument marshalling only.

Every function has the name of the C entry point it calls and takes torch tensors (device
memory for ``*_dev`` arguments, host memory for ``*_host``).  Nothing is computed here, and
there is no fallback: if ``libcore_b200.so`` cannot be loaded the import of a symbol raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

CORE_OK, CORE_EINVAL, CORE_ENOMEM, CORE_ECUDA, CORE_ELIMIT = 0, -1, -2, -3, -4
CORE_STATIC_SCRATCH_FLOATS = 1 << 20
CORE_F32, CORE_BF16 = 0, 1

_lib = None

_c = ctypes
_SIGNATURES = {
    "core_init": ([_c.POINTER(_c.c_void_p), _c.c_uint64, _c.c_int64, _c.c_int32], _c.c_int),
    "core_destroy": ([_c.c_void_p], _c.c_int),
    "core_set_stream": ([_c.c_void_p, _c.c_void_p], _c.c_int),
    "core_set_round": ([_c.c_void_p, _c.c_uint32], _c.c_int),
    "core_get_round": ([_c.c_void_p], _c.c_uint32),
    "core_workspace_bytes": ([_c.c_void_p], _c.c_size_t),
    "core_strerror": ([_c.c_int], _c.c_char_p),
    "core_last_cuda_error": ([_c.c_void_p], _c.c_int),
    "core_device_status": ([_c.POINTER(_c.c_int32)], _c.c_int),
    "core_project": ([_c.c_void_p, _c.c_void_p, _c.c_int, _c.c_int32, _c.c_int64, _c.c_void_p], _c.c_int),
    "core_aggregate": ([_c.c_void_p, _c.c_void_p, _c.c_int32, _c.c_void_p], _c.c_int),
    "core_reconstruct": ([_c.c_void_p, _c.c_void_p, _c.c_void_p], _c.c_int),
    "core_round": ([_c.c_void_p, _c.c_void_p, _c.c_int, _c.c_int32, _c.c_int64, _c.c_void_p, _c.c_void_p],
                   _c.c_int),
    "core_round_host": ([_c.c_void_p, _c.c_void_p, _c.c_int, _c.c_int32, _c.c_int64, _c.c_void_p,
                         _c.c_void_p], _c.c_int),
    "core_ls_create": ([_c.POINTER(_c.c_void_p), _c.c_void_p, _c.c_void_p, _c.c_int32, _c.c_int32, _c.c_int64],
                       _c.c_int),
    "core_ls_destroy": ([_c.c_void_p], _c.c_int),
    "core_gd_step": ([_c.c_void_p, _c.c_void_p, _c.c_float, _c.c_void_p], _c.c_int),
    "core_agd_step": ([_c.c_void_p, _c.c_void_p, _c.c_float, _c.c_float, _c.c_void_p, _c.c_void_p], _c.c_int),
    "core_gd_step_guarded": ([_c.c_void_p, _c.c_void_p, _c.c_float, _c.c_void_p, _c.c_void_p, _c.c_void_p],
                             _c.c_int),
    "core_gd_step_option1": ([_c.c_void_p, _c.c_void_p, _c.c_double, _c.c_double, _c.c_double, _c.c_void_p, _c.c_void_p,
                              _c.c_void_p, _c.c_void_p, _c.c_void_p], _c.c_int),
    "core_gossip_round": ([_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_int32, _c.c_void_p], _c.c_int),
    "core_decentralized_step": ([_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_int32, _c.c_int32, _c.c_int, _c.c_float,
                                 _c.c_void_p, _c.c_void_p], _c.c_int),
    "core_ls_loss": ([_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_void_p], _c.c_int),
    "core_ls_loss_host": ([_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_void_p], _c.c_int),
    "core_reserve_workspace": ([_c.c_void_p, _c.c_int32, _c.c_int], _c.c_int),
    "core_debug_fail_allocations": ([_c.c_int], _c.c_int),
    "core_debug_force_project_kernel": ([_c.c_int], _c.c_int),
    "core_debug_wait_timeout": ([_c.c_uint32, _c.c_int32, _c.POINTER(_c.c_uint32)], _c.c_int),
    "core_ls_gradients": ([_c.c_void_p, _c.c_void_p, _c.c_void_p, _c.c_void_p], _c.c_int),
    "core_debug_philox": ([_c.c_void_p, _c.c_uint32, _c.c_uint64, _c.c_int64, _c.c_void_p], _c.c_int),
    "core_debug_gaussians": ([_c.c_void_p, _c.c_uint32, _c.c_uint64, _c.c_int64, _c.c_void_p], _c.c_int),
    "core_debug_box_muller": ([_c.c_void_p, _c.c_void_p, _c.c_int64, _c.c_void_p], _c.c_int),
    "core_project_static": ([_c.c_uint64, _c.c_uint32, _c.c_int64, _c.c_int32, _c.c_void_p, _c.c_int, _c.c_int32,
                             _c.c_int64, _c.c_void_p, _c.c_void_p, _c.POINTER(_c.c_int)], _c.c_int),
    "core_debug_pipe_kinds": ([], _c.c_int),
    "core_debug_pipe_mix": ([_c.c_int, _c.POINTER(_c.c_int32)], _c.c_int),
    "core_debug_pipe_cycles": ([_c.c_int, _c.c_int, _c.c_int, _c.c_uint32, _c.POINTER(_c.c_double),
                                _c.POINTER(_c.c_uint32)], _c.c_int),
    "core_debug_project_plan": ([_c.c_int32, _c.c_int32, _c.c_int64, _c.c_int, _c.c_int32,
                                 _c.POINTER(_c.c_int64)], _c.c_int),
}


class CoreError(RuntimeError):
    def __init__(self, code: int, where: str, cuda: int = 0):
        self.code = code
        self.cuda = cuda
        msg = lib().core_strerror(code).decode()
        super().__init__(f"{where}: {msg} (code {code}" + (f", CUDA error {cuda})" if cuda else ")"))


def library_path() -> str:
    return _build.LIB


def lib() -> ctypes.CDLL:
    """The loaded shared library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not os.path.exists(path):
            raise RuntimeError(
                f"{path} is missing: build it with `python -m paper_2309_13307_b200.build` "
                "(needs nvcc); the CORE library has no non-CUDA path")
        L = ctypes.CDLL(path)
        for name, (argtypes, restype) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.argtypes = argtypes
            fn.restype = restype
        _lib = L
    return _lib


def exported_symbols():
    return list(_SIGNATURES)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return CORE_F32
    if t.dtype == torch.bfloat16:
        return CORE_BF16
    raise TypeError(f"gradients must be float32 or bfloat16, not {t.dtype}")


def _rows(G: torch.Tensor):
    """(pointer, dtype code, n, ld) of a 2-D tensor whose rows are contiguous."""
    if G.dim() != 2 or G.stride(1) != 1:
        raise ValueError("G must be 2-D with unit stride along coordinates")
    n = G.shape[0]
    ld = G.stride(0) if n > 1 else max(G.stride(0), G.shape[1])
    return G.data_ptr(), _dtype_code(G), n, ld


def _dev(t: torch.Tensor, dtype, numel=None) -> int:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"expected a contiguous CUDA tensor of {dtype}")
    if numel is not None and t.numel() < numel:
        raise ValueError(f"tensor too small: {t.numel()} < {numel}")
    return t.data_ptr()


def core_debug_project_plan(n: int, m: int, d: int, dtype: int = CORE_F32, sm_count: int = 148) -> dict:
    out = (ctypes.c_int64 * 10)()
    rc = lib().core_debug_project_plan(n, m, d, dtype, sm_count, out)
    if rc != CORE_OK:
        raise CoreError(rc, "core_debug_project_plan")
    keys = ("nb", "jt", "uq", "tile_q", "tj", "tq", "grid_x", "grid_y", "tiles", "smem")
    return dict(zip(keys, (int(v) for v in out)))


def core_debug_pipe_kinds() -> int:
    return int(lib().core_debug_pipe_kinds())


def core_debug_pipe_mix(kind: int) -> tuple:
    out = (ctypes.c_int32 * 7)()
    rc = lib().core_debug_pipe_mix(kind, out)
    if rc != CORE_OK:
        raise CoreError(rc, "core_debug_pipe_mix")
    return tuple(int(v) for v in out)


def core_debug_pipe_cycles(kind: int, warps_per_scheduler: int = 4, iters: int = 2048, seed: int = 1):
    """(SM cycles a scheduler spends per loop body and warp, checksum of the loop results)."""
    cyc, chk = ctypes.c_double(0.0), ctypes.c_uint32(0)
    rc = lib().core_debug_pipe_cycles(kind, warps_per_scheduler, iters, seed, ctypes.byref(cyc), ctypes.byref(chk))
    if rc != CORE_OK:
        raise CoreError(rc, "core_debug_pipe_cycles")
    return float(cyc.value), int(chk.value)


def core_debug_force_project_kernel(kind: int) -> None:
    """-1: by shape (default); 0: scalar; 1: warp-level tensor cores; 2: tensor-memory kernel."""
    rc = lib().core_debug_force_project_kernel(int(kind))
    if rc != CORE_OK:
        raise CoreError(rc, "core_debug_force_project_kernel")


def core_debug_fail_allocations(count: int) -> None:
    """The next `count` device allocations of the library fail (0 switches this off)."""
    rc = lib().core_debug_fail_allocations(int(count))
    if rc != CORE_OK:
        raise CoreError(rc, "core_debug_fail_allocations")


def core_debug_wait_timeout(limit_us: int, code: int) -> tuple:
    """(wait was served, second warp saw the abort flag) of the bounded-wait test kernel."""
    out = (ctypes.c_uint32 * 2)()
    rc = lib().core_debug_wait_timeout(int(limit_us), int(code), out)
    if rc != CORE_OK:
        raise CoreError(rc, "core_debug_wait_timeout")
    return int(out[0]), int(out[1])


def core_device_status() -> int:
    """Synchronises the current device; returns and clears the status word that a kernel raises
    when one of its bounded waits runs out (0: every wait was served)."""
    out = ctypes.c_int32(0)
    rc = lib().core_device_status(ctypes.byref(out))
    if rc != CORE_OK:
        raise CoreError(rc, "core_device_status")
    return int(out.value)


def core_project_static(seed: int, t: int, m: int, G_dev: torch.Tensor, P_dev: torch.Tensor,
                        stream: torch.cuda.Stream | None = None) -> torch.Tensor:
    """Projection for callers that must not allocate device memory (no context, no workspace):
    P_dev (caller-allocated, [n, m] float32) receives <g_i, xi_j>.  This wrapper allocates nothing
    either.  Raises CoreError with code CORE_ELIMIT when n > 16 or n*m exceeds the fixed scratch."""
    ptr, code, n, ld = _rows(G_dev)
    if not G_dev.is_cuda:
        raise ValueError("G must be a CUDA tensor")
    stream = stream if stream is not None else torch.cuda.current_stream()
    cuda_err = ctypes.c_int(0)
    rc = lib().core_project_static(int(seed), int(t), int(G_dev.shape[1]), int(m), ptr, code, n, ld,
                                   _dev(P_dev, torch.float32, n * m), ctypes.c_void_p(stream.cuda_stream),
                                   ctypes.byref(cuda_err))
    if rc != CORE_OK:
        raise CoreError(rc, "core_project_static", cuda_err.value)
    return P_dev


class Core:
    """A ``core_ctx``: fixed (seed, d, m), a round counter t, a stream and a workspace."""

    def __init__(self, seed: int, d: int, m: int, stream: torch.cuda.Stream | None = None):
        self._h = ctypes.c_void_p()
        self.seed, self.d, self.m = int(seed), int(d), int(m)
        rc = lib().core_init(ctypes.byref(self._h), self.seed, self.d, self.m)
        if rc != CORE_OK:
            self._h = ctypes.c_void_p()
            raise CoreError(rc, "core_init")
        self.core_set_stream(stream if stream is not None else torch.cuda.current_stream())

    def _check(self, rc: int, where: str):
        if rc != CORE_OK:
            raise CoreError(rc, where, lib().core_last_cuda_error(self._h))

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            lib().core_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- context ------------------------------------------------------------------
    def core_set_stream(self, stream: torch.cuda.Stream):
        self._check(lib().core_set_stream(self._h, ctypes.c_void_p(stream.cuda_stream)), "core_set_stream")

    def core_set_round(self, t: int):
        self._check(lib().core_set_round(self._h, int(t)), "core_set_round")

    def core_get_round(self) -> int:
        return int(lib().core_get_round(self._h))

    def core_workspace_bytes(self) -> int:
        return int(lib().core_workspace_bytes(self._h))

    def core_reserve_workspace(self, n: int, dtype: int = CORE_F32):
        self._check(lib().core_reserve_workspace(self._h, int(n), int(dtype)), "core_reserve_workspace")

    # -- the round ------------------------------------------------------------------
    def core_project(self, G_dev: torch.Tensor, P_dev: torch.Tensor | None = None) -> torch.Tensor:
        ptr, code, n, ld = _rows(G_dev)
        if not G_dev.is_cuda or G_dev.shape[1] != self.d:
            raise ValueError("G must be a CUDA tensor of shape [n, d]")
        if P_dev is None:
            P_dev = torch.empty((n, self.m), dtype=torch.float32, device=G_dev.device)
        self._check(lib().core_project(self._h, ptr, code, n, ld, _dev(P_dev, torch.float32, n * self.m)),
                    "core_project")
        return P_dev

    def core_aggregate(self, P_dev: torch.Tensor, pbar_dev: torch.Tensor | None = None) -> torch.Tensor:
        n = P_dev.shape[0]
        if pbar_dev is None:
            pbar_dev = torch.empty(self.m, dtype=torch.float32, device=P_dev.device)
        self._check(lib().core_aggregate(self._h, _dev(P_dev, torch.float32, n * self.m), n,
                                         _dev(pbar_dev, torch.float32, self.m)), "core_aggregate")
        return pbar_dev

    def core_reconstruct(self, pbar_dev: torch.Tensor, gtilde_dev: torch.Tensor | None = None) -> torch.Tensor:
        if gtilde_dev is None:
            gtilde_dev = torch.empty(self.d, dtype=torch.float32, device=pbar_dev.device)
        self._check(lib().core_reconstruct(self._h, _dev(pbar_dev, torch.float32, self.m),
                                           _dev(gtilde_dev, torch.float32, self.d)), "core_reconstruct")
        return gtilde_dev

    def core_round(self, G_dev: torch.Tensor, pbar_dev: torch.Tensor | None = None,
                   gtilde_dev: torch.Tensor | None = None):
        ptr, code, n, ld = _rows(G_dev)
        if not G_dev.is_cuda or G_dev.shape[1] != self.d:
            raise ValueError("G must be a CUDA tensor of shape [n, d]")
        if pbar_dev is None:
            pbar_dev = torch.empty(self.m, dtype=torch.float32, device=G_dev.device)
        if gtilde_dev is None:
            gtilde_dev = torch.empty(self.d, dtype=torch.float32, device=G_dev.device)
        self._check(lib().core_round(self._h, ptr, code, n, ld, _dev(pbar_dev, torch.float32, self.m),
                                     _dev(gtilde_dev, torch.float32, self.d)), "core_round")
        return pbar_dev, gtilde_dev

    def core_round_host(self, G_host: torch.Tensor, pbar_host: torch.Tensor, gtilde_host: torch.Tensor):
        ptr, code, n, ld = _rows(G_host)
        if G_host.is_cuda or pbar_host.is_cuda or gtilde_host.is_cuda or G_host.shape[1] != self.d:
            raise ValueError("core_round_host takes host tensors, G of shape [n, d]")
        if pbar_host.dtype != torch.float32 or gtilde_host.dtype != torch.float32 or \
                pbar_host.numel() < self.m or gtilde_host.numel() < self.d or \
                not pbar_host.is_contiguous() or not gtilde_host.is_contiguous():
            raise ValueError("pbar_host [m] and gtilde_host [d] must be contiguous float32")
        self._check(lib().core_round_host(self._h, ptr, code, n, ld, pbar_host.data_ptr(),
                                          gtilde_host.data_ptr()), "core_round_host")
        return pbar_host, gtilde_host

    # -- least squares ------------------------------------------------------------
    def core_gd_step(self, ls: "LeastSquares", h: float, x_dev: torch.Tensor):
        self._check(lib().core_gd_step(self._h, ls._h, float(h), _dev(x_dev, torch.float32, self.d)),
                    "core_gd_step")
        return x_dev

    def core_agd_step(self, ls: "LeastSquares", h: float, beta: float, x_dev: torch.Tensor, x_prev_dev: torch.Tensor):
        self._check(lib().core_agd_step(self._h, ls._h, float(h), float(beta), _dev(x_dev, torch.float32, self.d),
                                        _dev(x_prev_dev, torch.float32, self.d)), "core_agd_step")
        return x_dev, x_prev_dev

    def core_gd_step_guarded(self, ls: "LeastSquares", h: float, x_dev: torch.Tensor, f_dev: torch.Tensor,
                             accepted_dev: torch.Tensor | None = None):
        acc = ctypes.c_void_p(_dev(accepted_dev, torch.int32, 1)) if accepted_dev is not None else None
        self._check(lib().core_gd_step_guarded(self._h, ls._h, float(h), _dev(x_dev, torch.float32, self.d),
                                               _dev(f_dev, torch.float64, 1), acc), "core_gd_step_guarded")
        return x_dev, f_dev

    def core_gd_step_option1(self, ls: "LeastSquares", r1: float, H: float, c: float, x_dev: torch.Tensor,
                             f_dev: torch.Tensor, accepted_dev: torch.Tensor | None = None,
                             p_dev: torch.Tensor | None = None, h_dev: torch.Tensor | None = None):
        opt = lambda t, dt: ctypes.c_void_p(_dev(t, dt, 1)) if t is not None else None
        self._check(lib().core_gd_step_option1(self._h, ls._h, float(r1), float(H), float(c),
                                               _dev(x_dev, torch.float32, self.d), _dev(f_dev, torch.float64, 1),
                                               opt(accepted_dev, torch.int32), opt(p_dev, torch.float32),
                                               opt(h_dev, torch.float32)), "core_gd_step_option1")
        return x_dev, f_dev

    def core_gossip_round(self, W_dev: torch.Tensor, P_in_dev: torch.Tensor, P_out_dev: torch.Tensor | None = None):
        n = P_in_dev.shape[0]
        if P_out_dev is None:
            P_out_dev = torch.empty_like(P_in_dev)
        self._check(lib().core_gossip_round(self._h, _dev(W_dev, torch.float32, n * n),
                                            _dev(P_in_dev, torch.float32, n * self.m), n,
                                            _dev(P_out_dev, torch.float32, n * self.m)), "core_gossip_round")
        return P_out_dev

    def core_decentralized_step(self, ls: "LeastSquares", W_dev: torch.Tensor, rounds: int, h: float, x_dev: torch.Tensor,
                                reader: int = 0, as_printed: bool = False, spread_dev: torch.Tensor | None = None):
        sp = ctypes.c_void_p(_dev(spread_dev, torch.float32, 1)) if spread_dev is not None else None
        self._check(lib().core_decentralized_step(self._h, ls._h, _dev(W_dev, torch.float32, ls.n * ls.n), int(rounds),
                                                  int(reader), 1 if as_printed else 0, float(h),
                                                  _dev(x_dev, torch.float32, self.d), sp), "core_decentralized_step")
        return x_dev

    def core_ls_loss(self, ls: "LeastSquares", x_dev: torch.Tensor, loss_dev: torch.Tensor | None = None):
        if loss_dev is None:
            loss_dev = torch.empty(1, dtype=torch.float64, device=x_dev.device)
        self._check(lib().core_ls_loss(self._h, ls._h, _dev(x_dev, torch.float32, self.d),
                                       _dev(loss_dev, torch.float64, 1)), "core_ls_loss")
        return loss_dev

    def core_ls_loss_host(self, ls: "LeastSquares", x_dev: torch.Tensor, loss_host: torch.Tensor):
        if loss_host.is_cuda or loss_host.dtype != torch.float64 or loss_host.numel() < 1:
            raise ValueError("loss_host must be a host float64 tensor")
        self._check(lib().core_ls_loss_host(self._h, ls._h, _dev(x_dev, torch.float32, self.d), loss_host.data_ptr()),
                    "core_ls_loss_host")
        return loss_host

    def core_ls_gradients(self, ls: "LeastSquares", x_dev: torch.Tensor, G_out_dev: torch.Tensor | None = None):
        if G_out_dev is None:
            G_out_dev = torch.empty((ls.n, self.d), dtype=torch.float32, device=x_dev.device)
        self._check(lib().core_ls_gradients(self._h, ls._h, _dev(x_dev, torch.float32, self.d),
                                            _dev(G_out_dev, torch.float32, ls.n * self.d)), "core_ls_gradients")
        return G_out_dev

    # -- generator windows ----------------------------------------------------------
    def core_debug_philox(self, j: int, q0: int, nq: int) -> torch.Tensor:
        words = torch.empty((nq, 4), dtype=torch.int32, device="cuda")
        self._check(lib().core_debug_philox(self._h, j, q0, nq, words.data_ptr()), "core_debug_philox")
        return words

    def core_debug_gaussians(self, j: int, q0: int, nq: int) -> torch.Tensor:
        z = torch.empty((nq, 4), dtype=torch.float32, device="cuda")
        self._check(lib().core_debug_gaussians(self._h, j, q0, nq, z.data_ptr()), "core_debug_gaussians")
        return z

    def core_debug_box_muller(self, words_dev: torch.Tensor) -> torch.Tensor:
        nb = words_dev.numel() // 4
        z = torch.empty((nb, 4), dtype=torch.float32, device=words_dev.device)
        self._check(lib().core_debug_box_muller(self._h, _dev(words_dev, torch.int32, 4 * nb), nb, z.data_ptr()),
                    "core_debug_box_muller")
        return z


class LeastSquares:
    """A ``core_ls``: borrows A[n, rows, d] and b[n, rows] (kept alive here), owns the gradient scratch."""

    def __init__(self, A_dev: torch.Tensor, b_dev: torch.Tensor):
        if A_dev.dim() != 3 or b_dev.shape != A_dev.shape[:2]:
            raise ValueError("A must be [n, rows, d] and b [n, rows]")
        self.A, self.b = A_dev, b_dev
        self.n, self.rows, self.d = (int(s) for s in A_dev.shape)
        self._h = ctypes.c_void_p()
        rc = lib().core_ls_create(ctypes.byref(self._h), _dev(A_dev, torch.float32), _dev(b_dev, torch.float32),
                                  self.n, self.rows, self.d)
        if rc != CORE_OK:
            self._h = ctypes.c_void_p()
            raise CoreError(rc, "core_ls_create")

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            lib().core_ls_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
