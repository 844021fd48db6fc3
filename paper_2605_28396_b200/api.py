"""ctypes binding of the C ABI declared in ``include/adwin.h``: argument marshalling only.

Every step of the path runs in the CUDA library.  torch supplies device memory and the stream.
There is no CPU fallback: if the shared library is missing the first call raises.
"""
from __future__ import annotations

import ctypes
import math
from pathlib import Path
from types import SimpleNamespace

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libadwin_b200.so"

OK = 0
F32, BF16 = 0, 1
GRAD_FULL_KL, GRAD_SAMPLED = 0, 1
ZERO_TAIL, RANGE_FULL, FORCE_GENERIC, FORCE_STAGED = 1, 2, 4, 8
DEV_TOKEN_RANGE, DEV_NONFINITE, DEV_TIMEOUT, DEV_BOUNDS, DEV_WINDOW, DEV_WORKSPACE = 1, 2, 4, 8, 16, 32
ALIGN_DEGENERATE, ALIGN_NONE_ADMISSIBLE = 1, 2
DEFAULT_CANDIDATES = (64, 128, 256, 512, 1024, 2048)   # Section 5.1, Training Details
RHO_STAR = math.sqrt(2.0) / 2.0                          # Section 4.2, threshold equation

EXPORTS = ("adwin_version", "adwin_status_string", "adwin_workspace_bytes",
           "adwin_opd_kl_fwd_bwd", "adwin_window_reduce", "adwin_probe_align",
           "adwin_host_staging_bytes", "adwin_opd_kl_fwd_bwd_host",
           "adwin_no_alloc_max_sequences", "adwin_opd_kl_fwd_bwd_no_alloc",
           "adwin_return_to_go", "adwin_opd_kl_fwd_bwd_weighted", "adwin_teacher_drift",
           "adwin_drift_curves", "adwin_lmhead_workspace_bytes", "adwin_opd_kl_lmhead_fwd_bwd",
           "adwin_diag_set_wait_limit_ns", "adwin_lmhead_align_workspace_bytes",
           "adwin_lmhead_weight_align")

_lib = None


class AdwinError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(lib().adwin_status_string(code).decode())


def use_library(path=None):
    """Bind the calls to another build of the library (the bounds-checked flavour
    ``libadwin_b200_checked.so``), or back to the default one with ``path=None``."""
    global _lib, LIB_PATH
    LIB_PATH = Path(path) if path is not None else _PKG / "libadwin_b200.so"
    _lib = None


def lib():
    """Load libadwin_b200.so (built by ``build.py``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2605_28396_b200.build`; "
                "there is no fallback path")
        L = ctypes.CDLL(str(LIB_PATH))
        vp, i64, i32, f32, f64, sz = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32,
                                      ctypes.c_float, ctypes.c_double, ctypes.c_size_t)
        L.adwin_version.restype = ctypes.c_int
        L.adwin_status_string.restype = ctypes.c_char_p
        L.adwin_status_string.argtypes = [ctypes.c_int]
        L.adwin_workspace_bytes.restype = sz
        L.adwin_workspace_bytes.argtypes = [i64, i64, i64, ctypes.c_int, ctypes.c_int]
        L.adwin_opd_kl_fwd_bwd.restype = ctypes.c_int
        L.adwin_opd_kl_fwd_bwd.argtypes = [vp, vp, ctypes.c_int, i64, i64, i64, i64, vp, vp, vp,
                                           f32, ctypes.c_int, ctypes.c_int, vp, ctypes.c_int, i64,
                                           vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.adwin_window_reduce.restype = ctypes.c_int
        L.adwin_window_reduce.argtypes = [vp, vp, vp, vp, vp, i64, i64, vp, vp, vp]
        L.adwin_probe_align.restype = ctypes.c_int
        L.adwin_probe_align.argtypes = [vp, vp, vp, vp, vp, i64, i64, vp, i32, f64, vp, vp, vp,
                                        vp, vp, vp]
        L.adwin_host_staging_bytes.restype = sz
        L.adwin_host_staging_bytes.argtypes = [i64, i64, ctypes.c_int, ctypes.c_int, ctypes.c_int]
        L.adwin_opd_kl_fwd_bwd_host.restype = ctypes.c_int
        L.adwin_opd_kl_fwd_bwd_host.argtypes = [vp, vp, ctypes.c_int, i64, i64, i64, i64, vp, vp,
                                                vp, f32, ctypes.c_int, ctypes.c_int, vp,
                                                ctypes.c_int, i64, vp, vp, vp, vp, sz, i64, vp, vp]
        L.adwin_no_alloc_max_sequences.restype = i64
        L.adwin_opd_kl_fwd_bwd_no_alloc.restype = ctypes.c_int
        L.adwin_opd_kl_fwd_bwd_no_alloc.argtypes = [vp, vp, ctypes.c_int, i64, i64, i64, i64, vp,
                                                    vp, vp, f32, ctypes.c_int, ctypes.c_int, vp,
                                                    ctypes.c_int, i64, vp, vp, vp, vp, vp, vp, vp]
        L.adwin_return_to_go.restype = ctypes.c_int
        L.adwin_return_to_go.argtypes = [vp, vp, vp, i64, i64, f64, ctypes.c_int, vp, vp]
        L.adwin_opd_kl_fwd_bwd_weighted.restype = ctypes.c_int
        L.adwin_opd_kl_fwd_bwd_weighted.argtypes = [vp, vp, ctypes.c_int, i64, i64, i64, i64, vp,
                                                    vp, vp, vp, f32, ctypes.c_int, vp,
                                                    ctypes.c_int, i64, vp, vp, vp, vp, vp, vp, sz,
                                                    vp, vp]
        L.adwin_teacher_drift.restype = ctypes.c_int
        L.adwin_teacher_drift.argtypes = [vp, ctypes.c_int, i64, i64, i64, i64, vp, vp, vp, vp, vp,
                                          vp]
        L.adwin_drift_curves.restype = ctypes.c_int
        L.adwin_drift_curves.argtypes = [vp, vp, vp, i64, i64, vp, i32, vp, vp, vp, vp, vp]
        L.adwin_lmhead_workspace_bytes.restype = sz
        L.adwin_lmhead_workspace_bytes.argtypes = [i64, i64, i64, i64, i64, i64, ctypes.c_int,
                                                   ctypes.c_int]
        L.adwin_opd_kl_lmhead_fwd_bwd.restype = ctypes.c_int
        L.adwin_opd_kl_lmhead_fwd_bwd.argtypes = [vp, vp, vp, vp, i64, i64, i64, i64, i64, vp, vp,
                                                  vp, f32, ctypes.c_int, ctypes.c_int, vp,
                                                  ctypes.c_int, vp, vp, vp, vp, vp, vp, i64, vp,
                                                  sz, vp, vp]
        L.adwin_lmhead_align_workspace_bytes.restype = sz
        L.adwin_lmhead_align_workspace_bytes.argtypes = [i64, i64, i64, i64, i64, i64, i32]
        L.adwin_lmhead_weight_align.restype = ctypes.c_int
        L.adwin_lmhead_weight_align.argtypes = [vp, vp, vp, vp, i64, i64, i64, i64, i64, vp, vp,
                                                vp, i32, f64, ctypes.c_int, vp, vp, vp, vp, vp,
                                                vp, i64, vp, sz, vp, vp]
        L.adwin_diag_set_wait_limit_ns.restype = None
        L.adwin_diag_set_wait_limit_ns.argtypes = [ctypes.c_uint64]
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(device):
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def _dtype_code(dt):
    if dt == torch.float32:
        return F32
    if dt == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {dt}")


def _check(rc):
    if rc != OK:
        raise AdwinError(rc)


def adwin_workspace_bytes(B, T, V, dtype=BF16, flags=0) -> int:
    return int(lib().adwin_workspace_bytes(B, T, V, dtype, flags))


def adwin_opd_kl_fwd_bwd(student, teacher, tokens, window, rollout_len=None, *, grad_scale=1.0,
                         grad_mode=GRAD_FULL_KL, flags=0, grad=None, grad_dtype=None,
                         want_gsq=True, want_lse=False, out=None, workspace=None, dev_status=None,
                         row_coef=None):
    """Windowed per-token OPD divergence, forward + backward (see include/adwin.h).

    student, teacher: [B,T,V] CUDA tensors (fp32 or bf16), last dim contiguous, rows at a uniform
    stride.  ``grad``: a [B,T,V] tensor to write into, or None with ``grad_dtype`` set to have one
    allocated (uninitialised outside the window unless ZERO_TAIL), or both None for no gradient.
    Returns a namespace with kl, logratio, gsq, lse_s, lse_t, grad, dev_status (device tensors).
    Nothing is synchronised; read ``dev_status`` (or call ``raise_on_dev_status``) after a sync.
    With ``row_coef`` (see ``adwin_opd_kl_fwd_bwd_weighted``) the call goes to that entry point.
    """
    assert student.is_cuda and teacher.is_cuda and student.shape == teacher.shape
    assert student.dim() == 3 and student.dtype == teacher.dtype
    B, T, V = student.shape
    dev = student.device

    def row_stride(x):
        assert x.stride(2) == 1 or V == 1, "last dim must be contiguous"
        ld = x.stride(1) if T > 1 else (x.stride(0) if B > 1 else V)
        assert B <= 1 or T <= 1 or x.stride(0) == T * ld, "rows must sit at one uniform stride"
        return ld

    ld = row_stride(student)
    assert row_stride(teacher) == ld, "student and teacher must share the row stride"
    if grad is None and grad_dtype is not None:
        grad = torch.empty((B, T, V), dtype=grad_dtype, device=dev)
    ld_grad = row_stride(grad) if grad is not None else 0
    o = out if out is not None else SimpleNamespace()
    f32 = dict(dtype=torch.float32, device=dev)
    if getattr(o, "kl", None) is None:
        o.kl = torch.empty((B, T), **f32)
        o.logratio = torch.empty((B, T), **f32)
        o.gsq = torch.empty((B, T), **f32) if want_gsq else None
        o.lse_s = torch.empty((B, T), **f32) if want_lse else None
        o.lse_t = torch.empty((B, T), **f32) if want_lse else None
    o.grad = grad
    wsb = adwin_workspace_bytes(B, T, V, _dtype_code(student.dtype), flags)
    if workspace is None:
        workspace = torch.empty(wsb, dtype=torch.uint8, device=dev)
    if dev_status is None:
        dev_status = torch.zeros(1, dtype=torch.int32, device=dev)
    o.dev_status = dev_status
    o.workspace = workspace
    gdt = _dtype_code(grad.dtype) if grad is not None else 0
    if row_coef is None:
        rc = lib().adwin_opd_kl_fwd_bwd(
            _ptr(student), _ptr(teacher), _dtype_code(student.dtype), B, T, V, ld, _ptr(tokens),
            _ptr(window), _ptr(rollout_len), float(grad_scale), int(grad_mode), int(flags),
            _ptr(grad), gdt, ld_grad, _ptr(o.kl), _ptr(o.logratio), _ptr(o.gsq), _ptr(o.lse_s),
            _ptr(o.lse_t), _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream(dev))
    else:
        assert row_coef.shape == (B, T) and row_coef.dtype == torch.float32
        assert row_coef.is_contiguous() and row_coef.device == dev
        rc = lib().adwin_opd_kl_fwd_bwd_weighted(
            _ptr(student), _ptr(teacher), _dtype_code(student.dtype), B, T, V, ld, _ptr(tokens),
            _ptr(window), _ptr(rollout_len), _ptr(row_coef), float(grad_scale), int(flags),
            _ptr(grad), gdt, ld_grad, _ptr(o.kl), _ptr(o.logratio), _ptr(o.gsq), _ptr(o.lse_s),
            _ptr(o.lse_t), _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream(dev))
    _check(rc)
    return o


def adwin_opd_kl_fwd_bwd_weighted(student, teacher, tokens, window, rollout_len, row_coef, **kw):
    """Sampled-token gradient with ``row_coef[b,t]`` in place of c_t (Eq. 3; see include/adwin.h).
    Same arguments and result as ``adwin_opd_kl_fwd_bwd`` (``grad_mode`` is fixed)."""
    kw.pop("grad_mode", None)
    return adwin_opd_kl_fwd_bwd(student, teacher, tokens, window, rollout_len, row_coef=row_coef,
                                **kw)


def adwin_return_to_go(logratio, window, rollout_len=None, gamma=0.0, flags=0, out=None):
    """Discounted return-to-go of the per-token costs over each sequence's processed range (Eq. 3):
    returns a [B,T] float32 tensor, zero outside the range."""
    assert logratio.dim() == 2 and logratio.dtype == torch.float32 and logratio.is_contiguous()
    B, T = logratio.shape
    if out is None:
        out = torch.empty_like(logratio)
    _check(lib().adwin_return_to_go(_ptr(logratio), _ptr(window), _ptr(rollout_len), B, T,
                                    float(gamma), int(flags), _ptr(out), _stream(logratio.device)))
    return out


def raise_on_dev_status(dev_status, allow=0):
    """Synchronising read of the device status word; raises on bits outside ``allow``."""
    bits = int(dev_status.item())
    if bits & ~allow:
        names = {1: "TOKEN_RANGE", 2: "NONFINITE", 4: "TIMEOUT", 8: "BOUNDS", 16: "WINDOW",
                 32: "WORKSPACE"}
        raise RuntimeError("adwin device status: " +
                           "|".join(n for b, n in names.items() if bits & b))
    return bits


def adwin_window_reduce(kl, logratio, gsq, window, rollout_len=None):
    """Per-sequence and per-batch windowed sums: returns (seq_out [B,4], batch_out [4]) float64."""
    B, T = kl.shape
    dev = kl.device
    seq = torch.empty((B, 4), dtype=torch.float64, device=dev)
    batch = torch.empty(4, dtype=torch.float64, device=dev)
    _check(lib().adwin_window_reduce(_ptr(kl), _ptr(logratio), _ptr(gsq), _ptr(window),
                                     _ptr(rollout_len), B, T, _ptr(seq), _ptr(batch),
                                     _stream(dev)))
    return seq, batch


def adwin_probe_align(kl, logratio, gsq, window, rollout_len=None, candidates=None, rho_star=0.0):
    """Prefix-versus-full alignment audit.  ``candidates``: int32 CUDA tensor or None (paper list)."""
    B, T = kl.shape
    dev = kl.device
    K = 6 if candidates is None else int(candidates.numel())
    f64 = dict(dtype=torch.float64, device=dev)
    o = SimpleNamespace(
        seq_stats=torch.empty((B, K + 1, 4), **f64), seq_full=torch.empty((B, 3), **f64),
        batch_stats=torch.empty((K + 1, 5), **f64),
        L_next=torch.zeros(1, dtype=torch.int32, device=dev),
        flags=torch.zeros(1, dtype=torch.int32, device=dev))
    _check(lib().adwin_probe_align(_ptr(kl), _ptr(logratio), _ptr(gsq), _ptr(window),
                                   _ptr(rollout_len), B, T, _ptr(candidates), K, float(rho_star),
                                   _ptr(o.seq_stats), _ptr(o.seq_full), _ptr(o.batch_stats),
                                   _ptr(o.L_next), _ptr(o.flags), _stream(dev)))
    return o


def adwin_host_staging_bytes(rows_per_stage, V, dtype, grad_dtype, with_grad=True) -> int:
    return int(lib().adwin_host_staging_bytes(rows_per_stage, V, dtype, grad_dtype,
                                              1 if with_grad else 0))


def adwin_opd_kl_fwd_bwd_host(student, teacher, tokens, window, rollout_len=None, *, device,
                              grad=None, grad_scale=1.0, grad_mode=GRAD_FULL_KL, flags=0,
                              rows_per_stage=256, want_gsq=True, out=None, staging=None,
                              dev_status=None):
    """Host-buffer form: every tensor argument lives in (preferably pinned) host memory.

    Returns a namespace with host tensors kl, logratio, gsq, grad and the device status word.
    Asynchronous: synchronise the current stream of ``device`` before reading the outputs.
    """
    assert not student.is_cuda and not teacher.is_cuda and student.shape == teacher.shape
    B, T, V = student.shape
    assert student.is_contiguous() and teacher.is_contiguous()
    dev = torch.device(device)
    o = out if out is not None else SimpleNamespace()
    if getattr(o, "kl", None) is None:
        pin = dict(dtype=torch.float32, pin_memory=True)
        o.kl = torch.empty((B, T), **pin)
        o.logratio = torch.empty((B, T), **pin)
        o.gsq = torch.empty((B, T), **pin) if want_gsq else None
    o.grad = grad
    dt = _dtype_code(student.dtype)
    gdt = _dtype_code(grad.dtype) if grad is not None else dt
    need = adwin_host_staging_bytes(rows_per_stage, V, dt, gdt, grad is not None)
    if staging is None:
        staging = torch.empty(need, dtype=torch.uint8, device=dev)
    if dev_status is None:
        dev_status = torch.zeros(1, dtype=torch.int32, device=dev)
    o.dev_status, o.staging = dev_status, staging
    with torch.cuda.device(dev):
        rc = lib().adwin_opd_kl_fwd_bwd_host(
            _ptr(student), _ptr(teacher), dt, B, T, V, V, _ptr(tokens), _ptr(window),
            _ptr(rollout_len), float(grad_scale), int(grad_mode), int(flags), _ptr(grad), gdt, V,
            _ptr(o.kl), _ptr(o.logratio), _ptr(o.gsq), _ptr(staging), staging.numel(),
            int(rows_per_stage), _ptr(dev_status), _stream(dev))
    _check(rc)
    return o


def adwin_no_alloc_max_sequences() -> int:
    return int(lib().adwin_no_alloc_max_sequences())


def adwin_opd_kl_fwd_bwd_no_alloc(student, teacher, tokens, window, rollout_len, *, grad, kl,
                                  logratio, gsq, dev_status, grad_scale=1.0,
                                  grad_mode=GRAD_FULL_KL, flags=0, lse_s=None, lse_t=None):
    """The same pass through the entry point that needs no workspace and allocates nothing.

    For callers that own every buffer up front and may not allocate: all inputs AND outputs are
    passed in (this wrapper creates no tensor either), the row map lives in a fixed array inside
    the library.  B is limited to ``adwin_no_alloc_max_sequences()``; calls must stay ordered on
    one stream (they share that array).  ``grad`` may be None.  Returns None; raises AdwinError.
    """
    B, T, V = student.shape
    ld = student.stride(1) if T > 1 else (student.stride(0) if B > 1 else V)
    ld_grad = 0
    if grad is not None:
        ld_grad = grad.stride(1) if T > 1 else (grad.stride(0) if B > 1 else V)
    _check(lib().adwin_opd_kl_fwd_bwd_no_alloc(
        _ptr(student), _ptr(teacher), _dtype_code(student.dtype), B, T, V, ld, _ptr(tokens),
        _ptr(window), _ptr(rollout_len), float(grad_scale), int(grad_mode), int(flags), _ptr(grad),
        _dtype_code(grad.dtype) if grad is not None else 0, ld_grad, _ptr(kl), _ptr(logratio),
        _ptr(gsq), _ptr(lse_s), _ptr(lse_t), _ptr(dev_status), _stream(student.device)))


def adwin_teacher_drift(teacher, tokens, rollout_len=None, dev_status=None):
    """Teacher entropy (nats) and rank of the sampled token per position (Section 3.1).
    Returns a namespace with entropy [B,T] float32, rank [B,T] int32, dev_status."""
    assert teacher.is_cuda and teacher.dim() == 3
    B, T, V = teacher.shape
    dev = teacher.device
    assert teacher.stride(2) == 1 or V == 1, "last dim must be contiguous"
    ld = teacher.stride(1) if T > 1 else (teacher.stride(0) if B > 1 else V)
    assert B <= 1 or T <= 1 or teacher.stride(0) == T * ld, "rows must sit at one uniform stride"
    o = SimpleNamespace()
    o.entropy = torch.empty((B, T), dtype=torch.float32, device=dev)
    o.rank = torch.empty((B, T), dtype=torch.int32, device=dev)
    o.dev_status = dev_status if dev_status is not None else torch.zeros(1, dtype=torch.int32,
                                                                         device=dev)
    _check(lib().adwin_teacher_drift(_ptr(teacher), _dtype_code(teacher.dtype), B, T, V, ld,
                                     _ptr(tokens), _ptr(rollout_len), _ptr(o.entropy),
                                     _ptr(o.rank), _ptr(o.dev_status), _stream(dev)))
    return o


def adwin_drift_curves(entropy, rank, rollout_len=None, ks=(1, 5, 20)):
    """Top-k survival and mean branching factor per position over the batch (Section 3.1).
    Returns a namespace with worst_rank [B,T] int32, survival [K,T] float64, bf_mean [T] float64,
    n_active [T] int32."""
    B, T = entropy.shape
    dev = entropy.device
    ks_t = ks if torch.is_tensor(ks) else torch.tensor(list(ks), dtype=torch.int32, device=dev)
    K = int(ks_t.numel())
    o = SimpleNamespace()
    o.worst_rank = torch.empty((B, T), dtype=torch.int32, device=dev)
    o.survival = torch.empty((K, T), dtype=torch.float64, device=dev)
    o.bf_mean = torch.empty(T, dtype=torch.float64, device=dev)
    o.n_active = torch.empty(T, dtype=torch.int32, device=dev)
    _check(lib().adwin_drift_curves(_ptr(entropy), _ptr(rank), _ptr(rollout_len), B, T,
                                    _ptr(ks_t), K, _ptr(o.worst_rank), _ptr(o.survival),
                                    _ptr(o.bf_mean), _ptr(o.n_active), _stream(dev)))
    return o


def adwin_lmhead_workspace_bytes(B, T, V, d_s, d_t, max_rows=0, flags=0, with_grad=True) -> int:
    return int(lib().adwin_lmhead_workspace_bytes(B, T, V, d_s, d_t, int(max_rows), int(flags),
                                                  1 if with_grad else 0))


def adwin_opd_kl_lmhead_fwd_bwd(hidden_student, w_student, hidden_teacher, w_teacher, tokens,
                                window, rollout_len=None, *, grad_scale=1.0,
                                grad_mode=GRAD_FULL_KL, flags=0, grad_hidden=None, grad_w=None,
                                want_gsq=True, want_lse=False, max_rows=0, workspace=None,
                                dev_status=None):
    """Fused LM-head form: policies given as hidden states times output embeddings (adwin.h).

    hidden_* [B,T,d] and w_* [V,d] bf16 contiguous device tensors.  grad_hidden ([B,T,d_s], bf16 or
    fp32) and grad_w ([V,d_s] fp32) are caller-allocated and optional.  Returns a namespace with
    kl, logratio, gsq, lse_s, lse_t, dev_status, workspace.
    """
    B, T, ds = hidden_student.shape
    V = w_student.shape[0]
    dt = hidden_teacher.shape[2]
    dev = hidden_student.device
    for t in (hidden_student, w_student, hidden_teacher, w_teacher):
        if t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise TypeError("hidden states and LM heads must be contiguous bf16 tensors")
    if w_student.shape != (V, ds) or hidden_teacher.shape[:2] != (B, T) or \
            w_teacher.shape != (V, dt):
        raise ValueError("shape mismatch")
    for g in (grad_hidden, grad_w):
        if g is not None and not g.is_contiguous():
            raise ValueError("gradient tensors must be contiguous")
    kl = torch.empty((B, T), dtype=torch.float32, device=dev)
    logratio = torch.empty((B, T), dtype=torch.float32, device=dev)
    gsq = torch.empty((B, T), dtype=torch.float32, device=dev) if want_gsq else None
    lse_s = torch.empty((B, T), dtype=torch.float32, device=dev) if want_lse else None
    lse_t = torch.empty((B, T), dtype=torch.float32, device=dev) if want_lse else None
    with_grad = grad_hidden is not None or grad_w is not None
    need = adwin_lmhead_workspace_bytes(B, T, V, ds, dt, max_rows, flags, with_grad)
    if workspace is None:
        workspace = torch.empty(need + 1024, dtype=torch.uint8, device=dev)
    off = (-workspace.data_ptr()) % 1024
    ws_ptr = ctypes.c_void_p(workspace.data_ptr() + off)
    ws_bytes = workspace.numel() - off
    if dev_status is None:
        dev_status = torch.zeros(1, dtype=torch.int32, device=dev)
    gh_dtype = _dtype_code(grad_hidden.dtype) if grad_hidden is not None else F32
    if grad_w is not None and grad_w.dtype != torch.float32:
        raise TypeError("grad_w must be float32")
    _check(lib().adwin_opd_kl_lmhead_fwd_bwd(
        _ptr(hidden_student), _ptr(w_student), _ptr(hidden_teacher), _ptr(w_teacher), B, T, V, ds,
        dt, _ptr(tokens), _ptr(window), _ptr(rollout_len), float(grad_scale), int(grad_mode),
        int(flags), _ptr(grad_hidden), gh_dtype, _ptr(grad_w), _ptr(kl), _ptr(logratio),
        _ptr(gsq), _ptr(lse_s), _ptr(lse_t), int(max_rows), ws_ptr, ws_bytes, _ptr(dev_status),
        _stream(dev)))
    return SimpleNamespace(kl=kl, logratio=logratio, gsq=gsq, lse_s=lse_s, lse_t=lse_t,
                           dev_status=dev_status, workspace=workspace)


def adwin_diag_set_wait_limit_ns(ns: int) -> None:
    """Diagnostic: limit of the kernels' handshake waits for the launches that follow (0 = default)."""
    lib().adwin_diag_set_wait_limit_ns(int(ns))


def adwin_lmhead_weight_align(hidden_student, w_student, hidden_teacher, w_teacher, tokens,
                              rollout_len=None, candidates=None, rho_star=0.0, *,
                              grad_mode=GRAD_FULL_KL, max_rows=0, workspace=None, dev_status=None):
    """Section 4.2's prefix/full cosine in the space of the student's LM-head weight (adwin.h).

    candidates: a host sequence of ascending multiples of 64, or None for the paper's list.
    Returns a namespace with batch_stats [K,4] (rho_w, snr, admissible, n_tokens), L_next, flags,
    kl, logratio, gsq, dev_status, candidates.
    """
    B, T, ds = hidden_student.shape
    V = w_student.shape[0]
    dt = hidden_teacher.shape[2]
    dev = hidden_student.device
    for t in (hidden_student, w_student, hidden_teacher, w_teacher):
        if t.dtype != torch.bfloat16 or not t.is_contiguous():
            raise TypeError("hidden states and LM heads must be contiguous bf16 tensors")
    cands = list(DEFAULT_CANDIDATES) if candidates is None else [int(x) for x in candidates]
    K = len(cands)
    carr = (ctypes.c_int32 * max(K, 1))(*cands)
    kl = torch.empty((B, T), dtype=torch.float32, device=dev)
    logratio = torch.empty((B, T), dtype=torch.float32, device=dev)
    gsq = torch.empty((B, T), dtype=torch.float32, device=dev)
    stats = torch.empty((K, 4), dtype=torch.float64, device=dev)
    L_next = torch.zeros(1, dtype=torch.int32, device=dev)
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    need = int(lib().adwin_lmhead_align_workspace_bytes(B, T, V, ds, dt, int(max_rows), K))
    if workspace is None:
        workspace = torch.empty(need + 1024, dtype=torch.uint8, device=dev)
    off = (-workspace.data_ptr()) % 1024
    if dev_status is None:
        dev_status = torch.zeros(1, dtype=torch.int32, device=dev)
    _check(lib().adwin_lmhead_weight_align(
        _ptr(hidden_student), _ptr(w_student), _ptr(hidden_teacher), _ptr(w_teacher), B, T, V, ds,
        dt, _ptr(tokens), _ptr(rollout_len), ctypes.cast(carr, ctypes.c_void_p), K,
        float(rho_star), int(grad_mode), _ptr(kl), _ptr(logratio), _ptr(gsq), _ptr(stats),
        _ptr(L_next), _ptr(flags), int(max_rows), ctypes.c_void_p(workspace.data_ptr() + off),
        workspace.numel() - off, _ptr(dev_status), _stream(dev)))
    return SimpleNamespace(batch_stats=stats, L_next=L_next, flags=flags, kl=kl, logratio=logratio,
                           gsq=gsq, dev_status=dev_status, candidates=cands, workspace=workspace)
