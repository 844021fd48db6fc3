"""Full-size parity in the launch configuration the benchmark times: every processed row.

The sampled-row tests touch a few rows per sequence; these run the oracle over every in-window row
of config 3 (per-token scalars of all 15 360 rows, the gradient on a few hundred rows of every
sequence) and over two whole rollouts of config 4, one sequence at a time so that the float64 rows
fit in host memory.  What only a full-size run exercises is covered here: the persistent clusters'
row schedule, the ring phases over thousands of rows, the metadata ring's wrap-around.
"""
import numpy as np
import pytest
import torch

from oracle import adwin_oracle as O
from paper_2605_28396_b200 import api, synth
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def oracle_rows(batch, b, ts, want_grad, want_scale=False):
    """Oracle on positions ts of sequence b, gathered into one sequence that is all window."""
    idx = torch.as_tensor(ts, device=DEV)
    s = synth.bits_for_oracle(batch.student[b, idx].unsqueeze(0))
    t = synth.bits_for_oracle(batch.teacher[b, idx].unsqueeze(0))
    tok = batch.tokens[b, idx].unsqueeze(0).cpu().numpy()
    win = np.array([len(ts)], np.int32)
    ref = O.opd_kl_fwd_bwd(s, t, tok, win, None, want_grad=want_grad)
    if want_scale:
        ref["gsq_scale"] = O.gsq_term_scale(s, t, tok, win, None)
    return ref


def scalar_view(got, b, ts):
    idx = torch.as_tensor(ts, device=DEV)
    sub = type("S", (), {})()
    sub.kl, sub.logratio, sub.gsq = (x[b, idx].unsqueeze(0) for x in (got.kl, got.logratio, got.gsq))
    sub.lse_s, sub.lse_t = got.lse_s[b, idx].unsqueeze(0), got.lse_t[b, idx].unsqueeze(0)
    return sub


def test_config3_every_in_window_row_against_the_oracle():
    batch = synth.make_batch(3, device=DEV)
    B, T, V = batch.shape
    grad = torch.full((B, T, V), 7.0, dtype=torch.bfloat16, device=DEV)
    got = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                   batch.rollout_len, grad=grad, want_lse=True)
    torch.cuda.synchronize()
    api.raise_on_dev_status(got.dev_status)
    w = batch.window.cpu().numpy()
    rng = np.random.default_rng(33)
    n_rows = 0
    for b in range(B):
        n = int(w[b])
        ts = np.arange(n)
        ref = oracle_rows(batch, b, ts, want_grad=False)
        ones = np.ones((1, n), dtype=bool)
        P.check_scalars(scalar_view(got, b, ts), ref, 2e-3, ones, name=f"seq {b}: ", grad_mask=ones)
        n_rows += n
        # the gradient: the first and last 64 rows of the window and 64 rows in between
        pick = sorted(set(range(min(64, n))) | set(range(max(0, n - 64), n)) |
                      {int(x) for x in rng.integers(0, n, size=64)})
        gref = oracle_rows(batch, b, pick, want_grad=True)
        g = grad[b, torch.as_tensor(pick, device=DEV)].double().cpu().numpy()
        P.check_grad_rows(g, gref["grad"][0], 2e-3, name=f"seq {b}: ", store=2.0 ** -8)
        assert (grad[b, n:] == 7.0).all()
    assert n_rows == 15360


def test_config4_two_whole_rollouts_and_the_conditioning_of_the_single_sweep_norm():
    """Read-only probe pass at full size; every position of two rollouts against the oracle.
    The squared gradient norm of these rows comes from the single-sweep moment form, whose error
    is the fp32 accumulation error times the conditioning of sum e^2 (delta - E delta)^2 about the
    sampled token: 1e-3 relative plus 64 ulp of the oracle's term scale (the second part matters
    on peaked rows whose sampled token is not the peak).  The worst relative error and the worst
    conditioning met are printed."""
    batch = synth.make_batch(4, device=DEV, ragged_rollout=True, fill_all_rows=False)
    got = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                   batch.rollout_len, flags=api.RANGE_FULL, want_lse=True)
    torch.cuda.synchronize()
    api.raise_on_dev_status(got.dev_status)
    r = batch.rollout_len.cpu().numpy()
    order = np.argsort(r)
    worst, worst_cond, n_over, n_all = 0.0, 0.0, 0, 0
    for b in (int(order[0]), int(order[len(order) // 2])):   # the shortest and a median rollout
        n = int(r[b])
        ts = np.arange(n)
        ref = oracle_rows(batch, b, ts, want_grad=False, want_scale=True)
        P.check_scalars(scalar_view(got, b, ts), ref, 2e-3, np.ones((1, n), dtype=bool),
                        name=f"seq {b}: ", gsq_scale=ref["gsq_scale"])
        q = got.gsq[b, :n].double().cpu().numpy()
        rel = np.abs(q - ref["gsq"][0]) / ref["gsq"][0]
        cond = ref["gsq_scale"][0] / ref["gsq"][0]
        worst = max(worst, float(rel.max()))
        worst_cond = max(worst_cond, float(cond.max()))
        n_over += int((rel > P.RTOL_GSQ_SINGLE_SWEEP).sum())
        n_all += n
        assert (got.kl[b, n:] == 0).all()
    print(f"single-sweep gsq over {n_all} rows: worst relative error {worst:.3e}, "
          f"{n_over} rows above {P.RTOL_GSQ_SINGLE_SWEEP:g}, worst conditioning {worst_cond:.3g}")
