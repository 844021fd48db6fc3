"""GPU parity of the discounted return-to-go (Eq. 3) and of the sampled-token gradient that takes
it as its per-position coefficient, against the float64 oracle."""
from types import SimpleNamespace

import numpy as np
import pytest
import torch

from oracle import adwin_oracle as O
from paper_2605_28396_b200 import api, synth
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PATHS = {"staged": api.FORCE_STAGED, "generic": api.FORCE_GENERIC, "default": 0}


def _check_rtg(got, c64, window, rollout, gamma, flags):
    want = O.return_to_go(c64, window, rollout, gamma, flags)
    a = got.double().cpu().numpy()
    # fp64 sums rounded once to fp32: 2^-24 of the value, plus the order of the fp64 sums
    lim = 1e-6 * np.abs(want) + 1e-12 * np.abs(c64).sum(axis=1, keepdims=True)
    assert (np.abs(a - want) <= lim).all(), np.max(np.abs(a - want) / np.maximum(lim, 1e-300))
    return want


@pytest.mark.parametrize("gamma", [0.0, 0.5, 0.99, 1.0])
@pytest.mark.parametrize("T", [1, 7, 1000, 8192])
def test_return_to_go_matches_the_definition(gamma, T):
    g = torch.Generator().manual_seed(11 + T)
    B = 6
    c = (torch.randn((B, T), generator=g) * 1.5 + 0.1).to(DEV)
    window = torch.tensor([T, T // 2, 0, max(1, T // 3), T, 1], dtype=torch.int32)
    rollout = torch.tensor([T, T, T, max(1, T // 5), (T * 9) // 10, T], dtype=torch.int32)
    c64 = c.double().cpu().numpy()
    for flags in (0, api.RANGE_FULL):
        got = api.adwin_return_to_go(c, window.to(DEV), rollout.to(DEV), gamma, flags)
        want = _check_rtg(got, c64, window.numpy(), rollout.numpy(), gamma, flags)
        if gamma == 0.0:                                   # the token-local case is exact
            np.testing.assert_array_equal(got.cpu().numpy().astype(np.float64), want)
    got = api.adwin_return_to_go(c, window.to(DEV), None, gamma)      # rollout_len = NULL => T
    _check_rtg(got, c64, window.numpy(), None, gamma, 0)


def test_return_to_go_rejects_bad_arguments():
    c = torch.zeros((2, 4), device=DEV)
    w = torch.tensor([4, 4], dtype=torch.int32, device=DEV)
    for gamma in (-0.1, 1.5, float("nan")):
        with pytest.raises(Exception):
            api.adwin_return_to_go(c, w, None, gamma)
    with pytest.raises(Exception):
        api.adwin_return_to_go(c, w, None, 0.5, flags=api.ZERO_TAIL)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("in_cfg,g_dt", [(2, torch.bfloat16), (2, torch.float32),
                                         (1, torch.float32)])
def test_two_pass_future_coupled_gradient(path, in_cfg, g_dt):
    """Read-only pass for the costs, return-to-go, then the weighted gradient pass."""
    gamma, alpha, sentinel = 0.9, -0.5, 7.0
    batch = synth.make_batch(in_cfg, device=DEV, B=3, T=20, V=4096, ragged_rollout=True)
    batch.window = torch.tensor([20, 9, 4], dtype=torch.int32, device=DEV)
    batch.rollout_len = torch.tensor([20, 20, 3], dtype=torch.int32, device=DEV)
    B, T, V = batch.shape
    w, r = batch.window.cpu().numpy(), batch.rollout_len.cpu().numpy()
    first = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                     batch.rollout_len, flags=PATHS[path])
    rtg = api.adwin_return_to_go(first.logratio, batch.window, batch.rollout_len, gamma)
    grad = torch.full((B, T, V), sentinel, dtype=g_dt, device=DEV)
    got = api.adwin_opd_kl_fwd_bwd_weighted(batch.student, batch.teacher, batch.tokens,
                                            batch.window, batch.rollout_len, rtg,
                                            grad_scale=alpha, flags=PATHS[path], grad=grad,
                                            want_lse=True)
    torch.cuda.synchronize()
    api.raise_on_dev_status(first.dev_status)
    api.raise_on_dev_status(got.dev_status)

    rtol = P.rtol_for(batch.student.dtype, g_dt)
    ref = P.oracle_batch(batch, want_grad=False)
    mask = P.processed_mask(w, r, T, False)
    # (i) the per-row scalars of the weighted pass are those of the row
    got_scalars = SimpleNamespace(kl=got.kl, logratio=got.logratio, gsq=None, lse_s=got.lse_s,
                                  lse_t=got.lse_t)
    P.check_scalars(got_scalars, ref, rtol, mask)
    # (ii) return-to-go: same inputs through the oracle, and end to end from the oracle's costs
    c_gpu = first.logratio.double().cpu().numpy()
    _check_rtg(rtg, c_gpu, w, r, gamma, 0)
    G_ref = O.return_to_go(ref["logratio"], w, r, gamma)
    span = np.abs(ref["logratio"] * mask).sum(axis=1, keepdims=True)
    floor = rtol * np.maximum(1.0, np.abs(ref["lse_s"] - ref["lse_t"])).max()
    assert (np.abs(rtg.double().cpu().numpy() - G_ref) <= rtol * span + T * floor).all()
    # (iii) the gradient with exactly the coefficients the kernel was given
    z64 = batch.student.double().cpu().numpy()
    coef = rtg.double().cpu().numpy()
    tokens = batch.tokens.cpu().numpy()
    g = got.grad.double().cpu().numpy()
    q = got.gsq.double().cpu().numpy()
    rows, want_rows, want_q = [], [], []
    for b in range(B):
        for t in range(T):
            if mask[b, t]:
                gr, gq = O.row_weighted(z64[b, t], int(tokens[b, t]), alpha, coef[b, t])
                rows.append(g[b, t])
                want_rows.append(gr)
                want_q.append(gq)
    P.check_grad_rows(np.stack(rows), np.stack(want_rows), rtol, store=P.STORE[g_dt])
    want_q = np.array(want_q)
    assert (np.abs(q[mask] - want_q) <= P.RTOL_GSQ * want_q + 1e-30).all()
    assert (g[~mask] == sentinel).all() and (q[~mask] == 0).all()


def test_weighted_pass_with_the_costs_as_coefficients_is_the_sampled_mode():
    """gamma = 0: G_t = c_t, so the weighted entry point must reproduce ADWIN_GRAD_SAMPLED."""
    batch = synth.make_batch(2, device=DEV, B=2, T=10, V=8192)
    batch.window = torch.tensor([10, 6], dtype=torch.int32, device=DEV)
    plain = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                     batch.rollout_len, grad_mode=api.GRAD_SAMPLED,
                                     grad_dtype=torch.float32, flags=api.ZERO_TAIL)
    rtg = api.adwin_return_to_go(plain.logratio, batch.window, batch.rollout_len, 0.0)
    again = api.adwin_opd_kl_fwd_bwd_weighted(batch.student, batch.teacher, batch.tokens,
                                              batch.window, batch.rollout_len, rtg,
                                              grad_dtype=torch.float32, flags=api.ZERO_TAIL)
    torch.cuda.synchronize()
    assert torch.equal(plain.grad, again.grad) and torch.equal(plain.gsq, again.gsq)


def test_config3_full_size_two_pass_path_on_sampled_rows():
    """The return-to-go path at the size the bench times it (B=16, T=2048, V=151936): the scan
    against the oracle on every sequence, the weighted gradient on sampled rows."""
    gamma, alpha = 0.9, 1.0
    batch = synth.make_batch(3, device=DEV)
    B, T, V = batch.shape
    w, r = batch.window.cpu().numpy(), batch.rollout_len.cpu().numpy()
    first = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                     batch.rollout_len)
    rtg = api.adwin_return_to_go(first.logratio, batch.window, batch.rollout_len, gamma)
    sentinel = 7.0
    grad = torch.full((B, T, V), sentinel, dtype=torch.bfloat16, device=DEV)
    got = api.adwin_opd_kl_fwd_bwd_weighted(batch.student, batch.teacher, batch.tokens,
                                            batch.window, batch.rollout_len, rtg,
                                            grad_scale=alpha, grad=grad)
    torch.cuda.synchronize()
    api.raise_on_dev_status(got.dev_status)
    _check_rtg(rtg, first.logratio.double().cpu().numpy(), w, r, gamma, 0)
    rng = np.random.default_rng(4)
    coef = rtg.double().cpu().numpy()
    tokens = batch.tokens.cpu().numpy()
    rows, want, want_q = [], [], []
    for b in range(B):
        for t in sorted({0, int(w[b]) - 1} | {int(x) for x in rng.integers(0, int(w[b]), 2)}):
            g, q = O.row_weighted(batch.student[b, t].double().cpu().numpy(), int(tokens[b, t]),
                                  alpha, coef[b, t])
            rows.append((b, t))
            want.append(g)
            want_q.append(q)
    bs = torch.tensor([b for b, _ in rows], device=DEV)
    ts = torch.tensor([t for _, t in rows], device=DEV)
    P.check_grad_rows(grad[bs, ts].double().cpu().numpy(), np.stack(want), 2e-3, store=2.0 ** -8)
    q = got.gsq[bs, ts].double().cpu().numpy()
    assert (np.abs(q - np.array(want_q)) <= P.RTOL_GSQ * np.array(want_q) + 1e-30).all()
    for b in range(B):
        assert (grad[b, int(w[b]):] == sentinel).all()
