"""Comparison rules between the CUDA path and the float64 oracle (used by the -m gpu tests).

Tolerances (relative) on the arithmetic: 1e-5 for fp32 logits, 2e-3 for bf16 logits (fp32
accumulation).  A gradient stored as bf16 is additionally rounded once at the store: bf16 keeps 8
significant bits, so its unit roundoff is 2^-8 = 3.9e-3 (relative, worst case just above a power
of two), more than the 2e-3 allowed to the arithmetic; the store rounding is therefore budgeted
separately as `store` = 2^-8 for a bf16 gradient and 0 for an fp32 one.  A purely relative test is
undefined where a reference entry crosses zero or underflows, so every rule carries a floor scaled
by the row:
  gradient entry   |a-b| <= (rtol+store)*|b| + rtol*max_k|g_ref[row]|,
  gradient row     ||a-b||_2 <= (rtol+store)*||b||_2
  fp32 gradient from bf16 logits: additionally ||a-b||_2 <= 1e-4*||b||_2 (regression guard: the
                   fp32 arithmetic on exactly representable inputs is far better than 2e-3)
  kl, logratio     |a-b| <= rtol*|b| + rtol*max(1, |lse_s - lse_t|)
  gsq              |a-b| <= rtol_q*|b| + tiny.  rtol_q = 1e-4 where the gradient is written (the
                   norm is summed from the fp32 gradient entries themselves); 1e-3 on rows whose
                   gradient is not written: there the norm comes from the single-sweep moment form
                   sum e^2 (delta - E_p delta)^2 = B2 - 2 c0 B1 + c0^2 B0 in fp32, whose conditioning
                   (a few tens to hundreds on ordinary rows) multiplies the ~1e-6 accumulation
                   error.  On a peaked row whose sampled token is not the peak the conditioning
                   reaches 1/(1-p_max)^2; where a test passes the oracle's `gsq_scale` (the sum of
                   the magnitudes of the terms the one-sweep form adds and subtracts) the rule
                   becomes |a-b| <= rtol_q*|b| + 64 ulp * gsq_scale
  windowed sums    |a-b| <= 1e-4 * max(|b|, 1e-3 * sum|terms|)
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import adwin_oracle as O
from paper_2605_28396_b200 import api, synth

RTOL = {torch.float32: 1e-5, torch.bfloat16: 2e-3}
STORE = {torch.float32: 0.0, torch.bfloat16: 2.0 ** -8, None: 0.0}
RTOL_GSQ = 1e-4
RTOL_GSQ_SINGLE_SWEEP = 1e-3
RTOL_SUM = 1e-4


def rtol_for(in_dtype, grad_dtype=None):
    """Arithmetic tolerance: set by the logits' dtype (the accumulation is fp32 either way)."""
    return RTOL[in_dtype]


def oracle_batch(batch, rows=None, **kw):
    """Run the oracle on the stored values of a Batch (or of selected sequences)."""
    s = synth.bits_for_oracle(batch.student)
    t = synth.bits_for_oracle(batch.teacher)
    return O.opd_kl_fwd_bwd(s, t, batch.tokens.cpu().numpy(), batch.window.cpu().numpy(),
                            batch.rollout_len.cpu().numpy(), **kw)


GSQ_SCALE_ULPS = 64


def check_scalars(got, ref, rtol, processed_mask, name="", grad_mask=None, gsq_scale=None,
                  rtol_gsq_grad=None):
    """got: namespace of device tensors; ref: oracle dict; mask: [B,T] bool of processed rows;
    grad_mask: rows whose gradient was written (their gsq is summed from the gradient);
    gsq_scale: oracle's term scale of the one-sweep gsq, for the rows outside grad_mask."""
    kl = got.kl.double().cpu().numpy()
    c = got.logratio.double().cpu().numpy()
    floor = rtol * np.maximum(1.0, np.abs(ref["lse_s"] - ref["lse_t"]))
    m = processed_mask
    for a, b, nm in ((kl, ref["kl"], "kl"), (c, ref["logratio"], "logratio")):
        valid = m & np.isfinite(b)
        err = np.abs(a - b)[valid]
        lim = (rtol * np.abs(b) + floor)[valid]
        assert (err <= lim).all(), f"{name}{nm}: worst err/lim {np.max(err / lim):.3g}"
        assert (a[~m] == 0).all(), f"{name}{nm}: rows outside the processed range must be 0"
        nanref = m & ~np.isfinite(b)
        assert np.isnan(a[nanref]).all()
    if getattr(got, "gsq", None) is not None:
        q = got.gsq.double().cpu().numpy()
        b = ref["gsq"]
        valid = m & np.isfinite(b)
        err = np.abs(q - b)[valid]
        rq = np.full(b.shape, RTOL_GSQ_SINGLE_SWEEP)
        if grad_mask is not None:
            rq[grad_mask] = RTOL_GSQ if rtol_gsq_grad is None else rtol_gsq_grad
        lim_all = rq * np.abs(b) + 1e-30
        if gsq_scale is not None:
            extra = GSQ_SCALE_ULPS * 2.0 ** -23 * np.asarray(gsq_scale)
            if grad_mask is not None:
                extra = np.where(grad_mask, 0.0, extra)
            lim_all = lim_all + extra
        lim = lim_all[valid]
        assert (err <= lim).all(), f"{name}gsq: worst err/lim {np.max(err / lim):.3g}"
        assert (q[~m] == 0).all()
    if getattr(got, "lse_s", None) is not None:
        for a, b in ((got.lse_s, ref["lse_s"]), (got.lse_t, ref["lse_t"])):
            a = a.double().cpu().numpy()
            assert (np.abs(a - b)[m] <= 1e-6 * np.maximum(1.0, np.abs(b))[m]).all()


def check_grad_rows(got_rows, ref_rows, rtol, name="", store=0.0, guard=None):
    """got_rows, ref_rows: [n,V] float64 arrays of written gradient rows."""
    a, b = got_rows, ref_rows
    finite = np.isfinite(b).all(axis=1)
    a, b = a[finite], b[finite]
    if a.size == 0:
        return 0.0
    rowmax = np.abs(b).max(axis=1, keepdims=True)
    err = np.abs(a - b)
    lim = (rtol + store) * np.abs(b) + rtol * rowmax + 1e-300
    worst = float(np.max(err / lim))
    assert worst <= 1.0, f"{name}grad entries: worst err/lim {worst:.3g}"
    n2 = np.linalg.norm(a - b, axis=1)
    d2 = np.linalg.norm(b, axis=1)
    ratio = float(np.max(n2 / (d2 + 1e-300)))
    assert (n2 <= (rtol + store) * d2 + 1e-300).all(), f"{name}grad rows: worst {ratio:.3g}"
    if guard is not None:
        assert (n2 <= guard * d2 + 1e-300).all(), f"{name}grad rows (guard): worst {ratio:.3g}"
    return worst


def check_sums(got, ref, terms_abs):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    lim = RTOL_SUM * np.maximum(np.abs(ref), 1e-3 * np.asarray(terms_abs)) + 1e-300
    assert (np.abs(got - ref) <= lim).all(), f"sums: {got} vs {ref}"


def processed_mask(window, rollout_len, T, range_full=False):
    w = np.asarray(window)
    r = np.asarray(rollout_len)
    lim = r if range_full else np.minimum(w, r)
    return np.arange(T)[None, :] < lim[:, None]
