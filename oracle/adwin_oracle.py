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
        L.adwin_oracle_gsq_term_scale.restype = ctypes.c_double
        L.adwin_oracle_gsq_term_scale_batch.restype = ctypes.c_int
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


def gsq_term_scale(student, teacher, tokens, window, rollout_len=None, grad_scale: float = 1.0,
                   grad_mode: int = MODE_FULL_KL, flags: int = 0):
    """Conditioning scale of a one-sweep evaluation of gsq, per processed position ([B,T] float64):
    the magnitude of the terms such an evaluation adds and subtracts (see the C function)."""
    s, dt = _logit_array(student)
    t, dt2 = _logit_array(teacher)
    assert dt == dt2 and s.shape == t.shape and s.ndim == 3
    B, T, V = s.shape
    tokens, window, rollout_len = _i32(tokens), _i32(window), _i32(rollout_len)
    out = np.empty((B, T), dtype=np.float64)
    rc = lib().adwin_oracle_gsq_term_scale_batch(
        _p(s), _p(t), ctypes.c_int(dt), ctypes.c_int64(B), ctypes.c_int64(T), ctypes.c_int64(V),
        ctypes.c_int64(V), _p(tokens), _p(window), _p(rollout_len), ctypes.c_double(grad_scale),
        ctypes.c_int(grad_mode), ctypes.c_int(flags), _p(out))
    if rc != 0:
        raise ValueError(f"oracle rejected window / rollout lengths (code {rc})")
    return out


def row_gsq_term_scale(z, u, y: int, alpha: float = 1.0, mode: int = MODE_FULL_KL) -> float:
    z, u = _f64(z), _f64(u)
    return float(lib().adwin_oracle_gsq_term_scale(_p(z), _p(u), ctypes.c_int64(z.size),
                                                   ctypes.c_int64(int(y)), ctypes.c_double(alpha),
                                                   ctypes.c_int(mode)))


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


# --------------------------------------------------------------------------------------------
# Fused LM-head form: the two policies of Eq. 2 are softmax(H W^T), hidden states times an output
# embedding, and the quantities wanted are the same per-token scalars plus the gradients of the
# windowed loss with respect to the student's hidden states and LM-head weight.  Written as the
# definition: form the logits with a float64 matrix product (numpy's matmul is the library
# primitive of this step), hand every processed row to the per-row definition above, then apply
# the chain rule  dH_s = G W_s,  dW_s = G^T H_s  with G the window-masked logit gradient.
# --------------------------------------------------------------------------------------------
F64 = 2


def widen(a):
    """Stored values (float32 / float64, or uint16 bf16 bit patterns) exactly as float64."""
    a = np.ascontiguousarray(a)
    if a.dtype in (np.uint16, np.int16):
        return (a.view(np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    if a.dtype in (np.float32, np.float64):
        return a.astype(np.float64)
    raise TypeError(f"expected float32/float64 or bf16 bits (uint16), got {a.dtype}")


def _rows_f64_logits(z, u, tokens, window, rollout_len, grad_scale, grad_mode, flags):
    """Per-row definition on float64 logits z, u [B,T,V]; gradient zero outside the window."""
    B, T, V = z.shape
    kl = np.empty((B, T)); c = np.empty((B, T)); gsq = np.empty((B, T))
    ls = np.empty((B, T)); lt = np.empty((B, T))
    grad = np.zeros((B, T, V), dtype=np.float64)
    rc = lib().adwin_oracle_opd_kl_fwd_bwd(
        _p(z), _p(u), ctypes.c_int(F64), ctypes.c_int64(B), ctypes.c_int64(T), ctypes.c_int64(V),
        ctypes.c_int64(V), _p(tokens), _p(window), _p(rollout_len), ctypes.c_double(grad_scale),
        ctypes.c_int(grad_mode), ctypes.c_int(flags), _p(grad), ctypes.c_int64(V), _p(kl), _p(c),
        _p(gsq), _p(ls), _p(lt))
    if rc != 0:
        raise ValueError(f"oracle rejected window / rollout lengths (code {rc})")
    return kl, c, gsq, ls, lt, grad


def lmhead_logits(H, W):
    """z[b,t,k] = sum_j H[b,t,j] W[k,j] in float64 (stored values widened exactly)."""
    return widen(H) @ widen(W).T


def lmhead_fwd_bwd(Hs, Ws, Ht, Wt, tokens, window, rollout_len=None, grad_scale: float = 1.0,
                   grad_mode: int = MODE_FULL_KL, flags: int = 0):
    """The OPD divergence of Eq. 2 with both policies given as hidden states times an LM head.

    Hs [B,T,d_s], Ws [V,d_s] (student), Ht [B,T,d_t], Wt [V,d_t] (teacher); tokens, window,
    rollout_len, grad_scale, grad_mode as in opd_kl_fwd_bwd; flags: FLAG_RANGE_FULL only.
    One sequence at a time:
      z = Hs[b] Ws^T, u = Ht[b] Wt^T                       (the logits of Eq. 2's two policies)
      kl, logratio, gsq, lse per processed position        (the per-row definition)
      G[b,t,:] = d loss / d z[b,t,:] for t inside the window, zero elsewhere
      dH[b,t,:] = G[b,t,:] Ws                              chain rule through z = H_s W_s^T
      dW       += G[b]^T Hs[b]
    Returns dict(kl, logratio, gsq, lse_s, lse_t [B,T]; dH [B,T,d_s]; dW [V,d_s]), float64, and
    beside each gradient the sum of the absolute values of its terms, dH_abs = |G| |W_s| and
    dW_abs = |G|^T |H_s|: the scale against which a rounding of G is bounded; and dH_cond =
    (s P) |W_s|, dW_cond = (s P)^T |H_s| with P the student probabilities of the in-window rows
    and s = max(1, |E_p[z - u]|) per row: the scale against which an absolute perturbation of the
    centred difference (z_k - u_k) - E_p[z - u] inside g_k is bounded.
    """
    Hs64, Ws64, Ht64, Wt64 = widen(Hs), widen(Ws), widen(Ht), widen(Wt)
    B, T, ds = Hs64.shape
    V = Ws64.shape[0]
    assert Ws64.shape == (V, ds) and Ht64.shape[:2] == (B, T) and Wt64.shape == (V, Ht64.shape[2])
    tokens = _i32(tokens).reshape(B, T)
    window = _i32(window)
    rollout_len = _i32(rollout_len) if rollout_len is not None else np.full(B, T, np.int32)
    out = {k: np.zeros((B, T)) for k in ("kl", "logratio", "gsq", "lse_s", "lse_t")}
    dH = np.zeros((B, T, ds))
    dW = np.zeros((V, ds))
    dH_abs = np.zeros((B, T, ds))
    dW_abs = np.zeros((V, ds))
    dH_cond = np.zeros((B, T, ds))
    dW_cond = np.zeros((V, ds))
    for b in range(B):
        z = (Hs64[b] @ Ws64.T)[None]
        u = (Ht64[b] @ Wt64.T)[None]
        kl, c, gsq, ls, lt, G = _rows_f64_logits(z, u, tokens[b:b + 1], window[b:b + 1],
                                                 rollout_len[b:b + 1], grad_scale, grad_mode,
                                                 flags & FLAG_RANGE_FULL)
        for name, val in (("kl", kl), ("logratio", c), ("gsq", gsq), ("lse_s", ls), ("lse_t", lt)):
            out[name][b] = val[0]
        dH[b] = G[0] @ Ws64
        dW += G[0].T @ Hs64[b]
        dH_abs[b] = np.abs(G[0]) @ np.abs(Ws64)
        dW_abs += np.abs(G[0]).T @ np.abs(Hs64[b])
        inside = (np.arange(T) < min(window[b], rollout_len[b]))[:, None]
        sP = np.where(inside, np.exp(z[0] - ls[0][:, None]) *
                      np.maximum(1.0, np.abs(kl[0] + ls[0] - lt[0]))[:, None], 0.0)
        dH_cond[b] = sP @ np.abs(Ws64)
        dW_cond += sP.T @ np.abs(Hs64[b])
    out["dH"] = dH
    out["dW"] = dW
    out["dH_abs"] = dH_abs
    out["dW_abs"] = dW_abs
    out["dH_cond"] = dH_cond
    out["dW_cond"] = dW_cond
    return out


def lmhead_weight_cosine(Hs, Ws, Ht, Wt, tokens, rollout_len, candidates, grad_scale: float = 1.0,
                         grad_mode: int = MODE_FULL_KL):
    """Prefix-versus-full cosine of Section 4.2 in the space of the student's LM-head weight.

    For every candidate length L the prefix gradient is dW^(L) = sum over sequences and positions
    t < min(L, R_b) of g[b,t] h[b,t]^T, the full-horizon probe reference dW^full the same sum over
    t < R_b.  Literally: build both matrices, take <A,B> / (|A| |B|).  Returns
    dict(micro [K] = cosine after summing over the batch, macro [K] = mean over sequences of the
    per-sequence cosine, per_seq [B,K]).  A zero full norm gives cosine 1, a zero prefix norm 0.
    """
    Hs64, Ws64, Ht64, Wt64 = widen(Hs), widen(Ws), widen(Ht), widen(Wt)
    B, T, ds = Hs64.shape
    V = Ws64.shape[0]
    tokens = _i32(tokens).reshape(B, T)
    rollout_len = _i32(rollout_len) if rollout_len is not None else np.full(B, T, np.int32)
    cands = [int(L) for L in np.asarray(candidates).ravel()]

    def cos(a, b):
        na, nb = np.sqrt(np.sum(a * a)), np.sqrt(np.sum(b * b))
        if not nb > 0:
            return 1.0
        return float(np.sum(a * b) / (na * nb)) if na > 0 else 0.0

    full_b = np.zeros((B, V, ds))
    pre_b = np.zeros((len(cands), B, V, ds))
    for b in range(B):
        z = (Hs64[b] @ Ws64.T)[None]
        u = (Ht64[b] @ Wt64.T)[None]
        G = _rows_f64_logits(z, u, tokens[b:b + 1], rollout_len[b:b + 1], rollout_len[b:b + 1],
                             grad_scale, grad_mode, 0)[5][0]
        for t in range(T):
            if t < rollout_len[b]:
                outer = np.outer(G[t], Hs64[b, t])
                full_b[b] += outer
                for j, L in enumerate(cands):
                    if t < L:
                        pre_b[j, b] += outer
    per_seq = np.array([[cos(pre_b[j, b], full_b[b]) for j in range(len(cands))]
                        for b in range(B)]).reshape(B, len(cands))
    micro = np.array([cos(pre_b[j].sum(axis=0), full_b.sum(axis=0)) for j in range(len(cands))])
    return dict(micro=micro, macro=per_seq.mean(axis=0) if B else np.ones(len(cands)),
                per_seq=per_seq)
