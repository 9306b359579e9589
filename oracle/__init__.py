"""CORE oracle -- TEST INFRASTRUCTURE, not a product path.

ctypes access to the plain fp64 C restatement of the CORE round in
``core_oracle.c`` (Algorithm 1, Algorithm 2 and the Section-4 estimator of the
paper).  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import this package; the CUDA library never does.

``build()`` compiles the C file with gcc into ``libcore_oracle.so`` next to it;
``lib()`` loads it (building first when the shared object is missing or older
than its sources).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = [os.path.join(_HERE, "core_oracle.c"), os.path.join(_HERE, "core_oracle.h")]
_SO = os.path.join(_HERE, "libcore_oracle.so")
_lock = threading.Lock()
_lib = None

F32, BF16, F64 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle (strict IEEE: no fast-math, no contraction)."""
    stale = force or not os.path.exists(_SO) or any(
        os.path.getmtime(s) > os.path.getmtime(_SO) for s in _SRC
    )
    if stale:
        tmp = _SO + f".tmp{os.getpid()}"
        cmd = ["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-ffp-contract=off", "-Wall",
               "-Wextra", "-o", tmp, _SRC[0], "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _SO)
    return _SO


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(build())
            u32, u64, i32, i64 = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int32, ctypes.c_int64
            dbl, vp, ci = ctypes.c_double, ctypes.c_void_p, ctypes.c_int
            L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
            L.oracle_philox4x32_10.restype = None
            L.oracle_philox_round.argtypes = [vp, vp, vp]
            L.oracle_philox_round.restype = None
            L.oracle_uniform.argtypes = [u32]
            L.oracle_uniform.restype = dbl
            L.oracle_box_muller.argtypes = [vp, vp]
            L.oracle_box_muller.restype = None
            L.oracle_xi_words.argtypes = [u64, u32, u32, u64, vp]
            L.oracle_xi_words.restype = None
            L.oracle_xi_block.argtypes = [u64, u32, u32, u64, vp]
            L.oracle_xi_block.restype = None
            L.oracle_xi_range.argtypes = [u64, u32, u32, i64, i64, vp]
            L.oracle_xi_range.restype = None
            L.oracle_xi_words_many.argtypes = [u64, u32, u32, u64, i64, vp]
            L.oracle_xi_words_many.restype = None
            L.oracle_box_muller_many.argtypes = [vp, i64, vp]
            L.oracle_box_muller_many.restype = None
            L.oracle_project_slice.argtypes = [u64, u32, u32, vp, ci, i64, i64]
            L.oracle_project_slice.restype = dbl
            L.oracle_project.argtypes = [u64, u32, i64, i32, i32, vp, ci, i64, vp]
            L.oracle_project.restype = None
            L.oracle_aggregate.argtypes = [vp, i32, i32, vp]
            L.oracle_aggregate.restype = None
            L.oracle_reconstruct_slice.argtypes = [u64, u32, i32, vp, i64, i64, vp]
            L.oracle_reconstruct_slice.restype = None
            L.oracle_ls_loss.argtypes = [vp, vp, i32, i32, i64, vp]
            L.oracle_ls_loss.restype = dbl
            L.oracle_ls_grad.argtypes = [vp, vp, i32, i32, i64, vp, vp]
            L.oracle_ls_grad.restype = None
            L.oracle_gd_step.argtypes = [u64, u32, i32, vp, vp, i32, i32, i64, dbl, vp, vp, ci]
            L.oracle_gd_step.restype = None
            L.oracle_agd_step.argtypes = [u64, u32, i32, vp, vp, i32, i32, i64, dbl, dbl, vp, vp, vp, ci]
            L.oracle_agd_step.restype = None
            L.oracle_gd_step_guarded.argtypes = [u64, u32, i32, vp, vp, i32, i32, i64, dbl, vp, vp, vp]
            L.oracle_gd_step_guarded.restype = ci
            L.oracle_message_norm.argtypes = [vp, i32]
            L.oracle_message_norm.restype = dbl
            L.oracle_option1_step.argtypes = [dbl, i32, i64, dbl, dbl, dbl]
            L.oracle_option1_step.restype = dbl
            L.oracle_gd_step_option1.argtypes = [u64, u32, i32, vp, vp, i32, i32, i64, dbl, dbl, dbl, vp, vp, vp, vp, vp]
            L.oracle_gd_step_option1.restype = ci
            L.oracle_gossip_round.argtypes = [vp, vp, i32, i32, vp]
            L.oracle_gossip_round.restype = None
            L.oracle_gossip_average.argtypes = [vp, i32, i32, i32, vp, vp]
            L.oracle_gossip_average.restype = None
            L.oracle_decentralized_step.argtypes = [u64, u32, i32, vp, vp, i32, i32, i64, vp, i32, i32, ci, dbl, vp, vp]
            L.oracle_decentralized_step.restype = dbl
            _lib = L
    return _lib


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _grad_array(G: np.ndarray):
    """Return (contiguous 2-D array, dtype code).  uint16 arrays hold bf16 bit patterns."""
    G = np.ascontiguousarray(G)
    if G.ndim == 1:
        G = G[None, :]
    code = {np.dtype(np.float32): F32, np.dtype(np.uint16): BF16, np.dtype(np.float64): F64}
    return G, code[G.dtype]


# ---- generator ---------------------------------------------------------------

def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def philox_round(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox_round(_ptr(c), _ptr(k), _ptr(out))
    return out


def uniform(w: int) -> float:
    return lib().oracle_uniform(int(w) & 0xFFFFFFFF)


def box_muller(w) -> np.ndarray:
    w = np.asarray(w, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.float64)
    lib().oracle_box_muller(_ptr(w), _ptr(out))
    return out


def xi_words(seed: int, t: int, j: int, q: int) -> np.ndarray:
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_xi_words(seed, t, j, q, _ptr(out))
    return out


def xi_words_range(seed: int, t: int, j: int, q0: int, q1: int) -> np.ndarray:
    """Raw words of blocks q0..q1-1 of vector j, shape [q1-q0, 4]."""
    out = np.zeros((q1 - q0, 4), dtype=np.uint32)
    lib().oracle_xi_words_many(seed, t, j, q0, q1 - q0, _ptr(out))
    return out


def box_muller_many(words: np.ndarray) -> np.ndarray:
    """Box-Muller of an [nb, 4] uint32 array of words; returns [nb, 4] float64."""
    words = np.ascontiguousarray(words, dtype=np.uint32).reshape(-1, 4)
    out = np.zeros(words.shape, dtype=np.float64)
    lib().oracle_box_muller_many(_ptr(words), words.shape[0], _ptr(out))
    return out


def xi_block(seed: int, t: int, j: int, q: int) -> np.ndarray:
    out = np.zeros(4, dtype=np.float64)
    lib().oracle_xi_block(seed, t, j, q, _ptr(out))
    return out


def xi_range(seed: int, t: int, j: int, k0: int, k1: int) -> np.ndarray:
    out = np.zeros(max(k1 - k0, 0), dtype=np.float64)
    lib().oracle_xi_range(seed, t, j, k0, k1, _ptr(out))
    return out


# ---- the round ---------------------------------------------------------------

def project_slice(seed: int, t: int, j: int, g: np.ndarray, k0: int, k1: int) -> float:
    """sum_{k0 <= k < k1} g[k] xi_j[k]; g is one machine's whole gradient."""
    G, code = _grad_array(g)
    return lib().oracle_project_slice(seed, t, j, _ptr(G), code, k0, k1)


def project(seed: int, t: int, m: int, G: np.ndarray) -> np.ndarray:
    """P[n, m] from G[n, d] (float32, float64, or uint16 holding bf16 bits)."""
    G, code = _grad_array(G)
    n, d = G.shape
    P = np.zeros((n, m), dtype=np.float64)
    lib().oracle_project(seed, t, d, m, n, _ptr(G), code, d, _ptr(P))
    return P


def aggregate(P: np.ndarray) -> np.ndarray:
    P = np.ascontiguousarray(P, dtype=np.float64)
    n, m = P.shape
    pbar = np.zeros(m, dtype=np.float64)
    lib().oracle_aggregate(_ptr(P), n, m, _ptr(pbar))
    return pbar


def reconstruct_slice(seed: int, t: int, pbar: np.ndarray, k0: int, k1: int) -> np.ndarray:
    pbar = np.ascontiguousarray(pbar, dtype=np.float64)
    out = np.zeros(max(k1 - k0, 0), dtype=np.float64)
    lib().oracle_reconstruct_slice(seed, t, pbar.shape[0], _ptr(pbar), k0, k1, _ptr(out))
    return out


def reconstruct(seed: int, t: int, pbar: np.ndarray, d: int) -> np.ndarray:
    return reconstruct_slice(seed, t, pbar, 0, d)


def core_round(seed: int, t: int, m: int, G: np.ndarray):
    """project -> aggregate -> reconstruct; returns (P, pbar, gtilde)."""
    G2, _ = _grad_array(G)
    P = project(seed, t, m, G2)
    pbar = aggregate(P)
    return P, pbar, reconstruct(seed, t, pbar, G2.shape[1])


# ---- least-squares CORE-GD driver ---------------------------------------------

def _ls_arrays(A, b):
    A = np.ascontiguousarray(A, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    n, rows, d = A.shape
    assert b.shape == (n, rows)
    return A, b, n, rows, d


def ls_loss(A, b, x) -> float:
    A, b, n, rows, d = _ls_arrays(A, b)
    x = np.ascontiguousarray(x, dtype=np.float64)
    return lib().oracle_ls_loss(_ptr(A), _ptr(b), n, rows, d, _ptr(x))


def ls_grad(A, b, x) -> np.ndarray:
    A, b, n, rows, d = _ls_arrays(A, b)
    x = np.ascontiguousarray(x, dtype=np.float64)
    G = np.zeros((n, d), dtype=np.float64)
    lib().oracle_ls_grad(_ptr(A), _ptr(b), n, rows, d, _ptr(x), _ptr(G))
    return G


def gd_step(seed: int, t: int, m: int, A, b, h: float, x: np.ndarray, exact: bool = False) -> np.ndarray:
    """One Algorithm-2 iteration with round index t; returns the new iterate."""
    A, b, n, rows, d = _ls_arrays(A, b)
    x = np.array(x, dtype=np.float64, copy=True)
    work = np.zeros(n * d + n * m + m + d, dtype=np.float64)
    lib().oracle_gd_step(seed, t, m, _ptr(A), _ptr(b), n, rows, d, float(h), _ptr(x), _ptr(work),
                         1 if exact else 0)
    return x


def agd_step(seed: int, t: int, m: int, A, b, h: float, beta: float, x: np.ndarray, x_prev: np.ndarray,
             exact: bool = False):
    """One Algorithm-4 iteration with round index t; returns (x_new, x)."""
    A, b, n, rows, d = _ls_arrays(A, b)
    x = np.array(x, dtype=np.float64, copy=True)
    x_prev = np.array(x_prev, dtype=np.float64, copy=True)
    work = np.zeros(d + n * d + n * m + m + d, dtype=np.float64)
    lib().oracle_agd_step(seed, t, m, _ptr(A), _ptr(b), n, rows, d, float(h), float(beta), _ptr(x), _ptr(x_prev),
                          _ptr(work), 1 if exact else 0)
    return x, x_prev


def gd_step_guarded(seed: int, t: int, m: int, A, b, h: float, x: np.ndarray, f_x: float):
    """One Algorithm-3 iteration (caller-fixed step): returns (x_kept, f(x_kept), accepted)."""
    A, b, n, rows, d = _ls_arrays(A, b)
    x = np.array(x, dtype=np.float64, copy=True)
    f = np.array([f_x], dtype=np.float64)
    work = np.zeros(d + n * d + n * m + m + d, dtype=np.float64)
    acc = lib().oracle_gd_step_guarded(seed, t, m, _ptr(A), _ptr(b), n, rows, d, float(h), _ptr(x), _ptr(f),
                                       _ptr(work))
    return x, float(f[0]), bool(acc)


# ---- Algorithm 3, Option I -------------------------------------------------------

def message_norm(pbar: np.ndarray) -> float:
    """sqrt((1/m) sum_j pbar_j^2): the statistic p of Algorithm 3 in the reading taken here."""
    pbar = np.ascontiguousarray(pbar, dtype=np.float64)
    return lib().oracle_message_norm(_ptr(pbar), pbar.shape[0])


def option1_step(p: float, m: int, d: int, r1: float, H: float, c: float = 1.0 / 1600.0) -> float:
    return lib().oracle_option1_step(float(p), int(m), int(d), float(r1), float(H), float(c))


def gd_step_option1(seed: int, t: int, m: int, A, b, r1: float, H: float, c: float, x: np.ndarray, f_x: float):
    """One Algorithm-3 iteration with Option I: returns (x_kept, f(x_kept), accepted, p, h)."""
    A, b, n, rows, d = _ls_arrays(A, b)
    x = np.array(x, dtype=np.float64, copy=True)
    f = np.array([f_x], dtype=np.float64)
    p = np.zeros(1, dtype=np.float64)
    h = np.zeros(1, dtype=np.float64)
    work = np.zeros(n * d + n * m + m + 2 * d, dtype=np.float64)
    acc = lib().oracle_gd_step_option1(seed, t, m, _ptr(A), _ptr(b), n, rows, d, float(r1), float(H), float(c),
                                       _ptr(x), _ptr(f), _ptr(p), _ptr(h), _ptr(work))
    return x, float(f[0]), bool(acc), float(p[0]), float(h[0])


# ---- Algorithm 5: decentralised CORE-GD --------------------------------------------

def gossip_round(W: np.ndarray, P: np.ndarray) -> np.ndarray:
    W = np.ascontiguousarray(W, dtype=np.float64)
    P = np.ascontiguousarray(P, dtype=np.float64)
    n, m = P.shape
    assert W.shape == (n, n)
    out = np.zeros_like(P)
    lib().oracle_gossip_round(_ptr(W), _ptr(P), n, m, _ptr(out))
    return out


def gossip_average(W: np.ndarray, P: np.ndarray, rounds: int) -> np.ndarray:
    W = np.ascontiguousarray(W, dtype=np.float64)
    P = np.array(P, dtype=np.float64, copy=True, order="C")
    n, m = P.shape
    assert W.shape == (n, n)
    scratch = np.zeros_like(P)
    lib().oracle_gossip_average(_ptr(W), int(rounds), n, m, _ptr(P), _ptr(scratch))
    return P


def decentralized_step(seed: int, t: int, m: int, A, b, W: np.ndarray, rounds: int, h: float, x: np.ndarray,
                       reader: int = 0, as_printed: bool = False):
    """One Algorithm-5 iteration; returns (x_new, spread of the machines' estimates around the reader's)."""
    A, b, n, rows, d = _ls_arrays(A, b)
    W = np.ascontiguousarray(W, dtype=np.float64)
    assert W.shape == (n, n)
    x = np.array(x, dtype=np.float64, copy=True)
    work = np.zeros(n * d + 2 * n * m + d, dtype=np.float64)
    spread = lib().oracle_decentralized_step(seed, t, m, _ptr(A), _ptr(b), n, rows, d, _ptr(W), int(rounds),
                                             int(reader), 1 if as_printed else 0, float(h), _ptr(x), _ptr(work))
    return x, float(spread)
