"""ctypes loader for the float64 CPU oracle (``adwin_oracle.c``).

TEST INFRASTRUCTURE, not the product: only the tests, the smoke check and the benchmark's
CPU-baseline leg import this module.  It imports nothing from the CUDA package.  The arithmetic
lives in the C file; this module only compiles it with gcc, marshals numpy arrays and returns
numpy float64 results.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "adwin_oracle.c"
_LIB = _HERE / "libadwin_oracle.so"

F32, BF16 = 0, 1
MODE_FULL_KL, MODE_SAMPLED = 0, 1
FLAG_ZERO_TAIL, FLAG_RANGE_FULL = 1, 2
ALIGN_DEGENERATE, ALIGN_NONE_ADMISSIBLE = 1, 2

_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (OpenMP over rows when available)."""
    if not force and _LIB.exists() and _LIB.stat().st_mtime >= _SRC.stat().st_mtime:
        return _LIB
    tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
           str(_SRC), "-o", str(tmp), "-lm"]
    subprocess.run(cmd, check=True, capture_output=True)
    os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(str(_LIB))
        L.adwin_oracle_logsumexp.restype = ctypes.c_double
        L.adwin_oracle_literal_cosine.restype = ctypes.c_double
        L.adwin_oracle_opd_kl_fwd_bwd.restype = ctypes.c_int
        L.adwin_oracle_num_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def num_threads() -> int:
    return int(lib().adwin_oracle_num_threads())


def logsumexp(v) -> float:
    v = _f64(v)
    return float(lib().adwin_oracle_logsumexp(_p(v), ctypes.c_int64(v.size)))


def row(z, u, y: int, alpha: float = 1.0, mode: int = MODE_FULL_KL):
    """One position: returns dict(kl, c, lse_s, lse_t, gsq, g)."""
    z, u = _f64(z), _f64(u)
    V = z.size
    g = np.empty(V, dtype=np.float64)
    out = [ctypes.c_double() for _ in range(5)]
    lib().adwin_oracle_row(_p(z), _p(u), ctypes.c_int64(V), ctypes.c_int64(int(y)),
                           ctypes.c_double(alpha), ctypes.c_int(mode),
                           *[ctypes.byref(o) for o in out], _p(g))
    kl, c, ls, lt, gsq = [o.value for o in out]
    return dict(kl=kl, c=c, lse_s=ls, lse_t=lt, gsq=gsq, g=g)


def _logit_array(a):
    """Accept float32 arrays, or uint16/int16 arrays holding bf16 bit patterns."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.float32:
        return a, F32
    if a.dtype in (np.uint16, np.int16):
        return a.view(np.uint16), BF16
    raise TypeError(f"logits must be float32 or bf16 bits (uint16), got {a.dtype}")


def opd_kl_fwd_bwd(student, teacher, tokens, window, rollout_len=None, grad_scale: float = 1.0,
                   grad_mode: int = MODE_FULL_KL, flags: int = 0, want_grad: bool = True,
                   grad_init=None, ld: int | None = None):
    """Whole batch.  student/teacher: [B,T,V] (float32, or uint16 bf16 bits).

    Returns dict(kl, logratio, gsq, lse_s, lse_t [B,T] float64, grad [B,T,V] float64 or None).
    ``grad_init`` pre-fills the gradient buffer (to observe which rows are left untouched).
    """
    s, dt = _logit_array(student)
    t, dt2 = _logit_array(teacher)
    assert dt == dt2 and s.shape == t.shape and s.ndim == 3
    B, T, V = s.shape
    ld = V if ld is None else ld
    tokens = _i32(tokens)
    window = _i32(window)
    rollout_len = _i32(rollout_len)
    kl = np.empty((B, T), dtype=np.float64)
    c = np.empty((B, T), dtype=np.float64)
    gsq = np.empty((B, T), dtype=np.float64)
    ls = np.empty((B, T), dtype=np.float64)
    lt = np.empty((B, T), dtype=np.float64)
    grad = None
    if want_grad:
        grad = (np.array(grad_init, dtype=np.float64, copy=True) if grad_init is not None
                else np.full((B, T, V), np.nan, dtype=np.float64))
        assert grad.shape == (B, T, V)
    rc = lib().adwin_oracle_opd_kl_fwd_bwd(
        _p(s), _p(t), ctypes.c_int(dt), ctypes.c_int64(B), ctypes.c_int64(T), ctypes.c_int64(V),
        ctypes.c_int64(ld), _p(tokens), _p(window), _p(rollout_len), ctypes.c_double(grad_scale),
        ctypes.c_int(grad_mode), ctypes.c_int(flags), _p(grad), ctypes.c_int64(V), _p(kl), _p(c),
        _p(gsq), _p(ls), _p(lt))
    if rc != 0:
        raise ValueError(f"oracle rejected window / rollout lengths (code {rc})")
    return dict(kl=kl, logratio=c, gsq=gsq, lse_s=ls, lse_t=lt, grad=grad)


def window_reduce(kl, logratio, gsq, window, rollout_len=None):
    kl, logratio = _f64(kl), _f64(logratio)
    gsq = None if gsq is None else _f64(gsq)
    B, T = kl.shape
    window, rollout_len = _i32(window), _i32(rollout_len)
    seq = np.empty((B, 4), dtype=np.float64)
    batch = np.empty(4, dtype=np.float64)
    lib().adwin_oracle_window_reduce(_p(kl), _p(logratio), _p(gsq), _p(window), _p(rollout_len),
                                     ctypes.c_int64(B), ctypes.c_int64(T), _p(seq), _p(batch))
    return seq, batch


def probe_align(kl, logratio, gsq, window, rollout_len, candidates, rho_star: float):
    kl, logratio, gsq = _f64(kl), _f64(logratio), _f64(gsq)
    B, T = kl.shape
    window, rollout_len, candidates = _i32(window), _i32(rollout_len), _i32(candidates)
    K = int(candidates.size)
    seq_stats = np.empty((B, K + 1, 4), dtype=np.float64)
    seq_full = np.empty((B, 3), dtype=np.float64)
    batch_stats = np.empty((K + 1, 5), dtype=np.float64)
    L_next = ctypes.c_int32()
    flags = ctypes.c_int32()
    lib().adwin_oracle_probe_align(_p(kl), _p(logratio), _p(gsq), _p(window), _p(rollout_len),
                                   ctypes.c_int64(B), ctypes.c_int64(T), _p(candidates),
                                   ctypes.c_int32(K), ctypes.c_double(rho_star), _p(seq_stats),
                                   _p(seq_full), _p(batch_stats), ctypes.byref(L_next),
                                   ctypes.byref(flags))
    return dict(seq_stats=seq_stats, seq_full=seq_full, batch_stats=batch_stats,
                L_next=int(L_next.value), flags=int(flags.value))


def literal_cosine(grad, rollout_len, L: int):
    grad = _f64(grad)
    B, T, V = grad.shape
    rollout_len = _i32(rollout_len)
    per_seq = np.empty(B, dtype=np.float64)
    micro = lib().adwin_oracle_literal_cosine(_p(grad), _p(rollout_len), ctypes.c_int64(B),
                                              ctypes.c_int64(T), ctypes.c_int64(V),
                                              ctypes.c_int64(int(L)), _p(per_seq))
    return float(micro), per_seq


def return_to_go(logratio, window, rollout_len=None, gamma: float = 0.0, flags: int = 0):
    """Discounted return-to-go G[b,t] of the per-token costs over each sequence's range (Eq. 3)."""
    c = _f64(logratio)
    B, T = c.shape
    window, rollout_len = _i32(window), _i32(rollout_len)
    G = np.empty((B, T), dtype=np.float64)
    lib().adwin_oracle_return_to_go(_p(c), _p(window), _p(rollout_len), ctypes.c_int64(B),
                                    ctypes.c_int64(T), ctypes.c_double(gamma), ctypes.c_int(flags),
                                    _p(G))
    return G


def row_weighted(z, y: int, alpha: float, w: float):
    """Sampled-token gradient of one position with coefficient w in place of c: (g, gsq)."""
    z = _f64(z)
    g = np.empty(z.size, dtype=np.float64)
    gsq = ctypes.c_double()
    lib().adwin_oracle_row_weighted(_p(z), ctypes.c_int64(z.size), ctypes.c_int64(int(y)),
                                    ctypes.c_double(alpha), ctypes.c_double(w), ctypes.byref(gsq),
                                    _p(g))
    return g, gsq.value


def teacher_drift_row(u, y: int):
    """Entropy (nats) of softmax(u) and the rank of token y under it (Section 3.1)."""
    u = _f64(u)
    H = ctypes.c_double()
    r = ctypes.c_int64()
    lib().adwin_oracle_teacher_drift_row(_p(u), ctypes.c_int64(u.size), ctypes.c_int64(int(y)),
                                         ctypes.byref(H), ctypes.byref(r))
    return H.value, int(r.value)


def topk_survival(rank, rollout_len, k: int):
    """S_T^(k) for every position T: [T] float64 (Section 3.1)."""
    rank = np.ascontiguousarray(rank, dtype=np.int64)
    B, T = rank.shape
    rollout_len = _i32(rollout_len)
    out = np.empty(T, dtype=np.float64)
    lib().adwin_oracle_topk_survival(_p(rank), _p(rollout_len), ctypes.c_int64(B),
                                     ctypes.c_int64(T), ctypes.c_int64(int(k)), _p(out))
    return out
