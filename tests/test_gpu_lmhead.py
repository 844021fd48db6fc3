"""GPU parity of the fused LM-head path (through the C ABI) against the float64 oracle.

Tolerances: the logits are bf16 products accumulated in fp32 on the tensor cores, so the per-token
scalars are held to the bf16-logit tolerance of the logit path (2e-3 with its floors, `gsq` from
the single-sweep moment form at 1e-3); the log-sum-exp values to 1e-5 (fp32 accumulation over a
contraction of a few thousand terms).  The logit gradient G is rounded to bf16 once before the two
gradient products.  An entry of dH or dW is a sum of signed terms G*w or G*h, so that rounding is
bounded against the sum of the terms' absolute values (which the oracle returns beside each
gradient), not against the entry itself:
    |a - b| <= 2e-3 |b| + 2e-3 max|b_row| + 2^-9 sum|terms| (+ 2^-8 |b| for a bf16 output)
               + |alpha| 8 ulp * sum_k s p_k |w_k|   (the fp32 floor of a peaked row's centred
                                                      difference, s = max(1, |E_p[z-u]|)),
and every row must satisfy ||a - b||_2 <= (2e-3 + 2^-8) ||b||_2 + the 2-norm of that last floor.
"""
import numpy as np
import pytest
import torch

from oracle import adwin_oracle as O
from paper_2605_28396_b200 import api, synth
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
RTOL = 2e-3
STORE = 2.0 ** -8
RTOL_LSE = 1e-5


def bits(t):
    return synth.bits_for_oracle(t)


def run(batch, *, mode=api.GRAD_FULL_KL, flags=0, gh_dtype=torch.bfloat16, grad_scale=1.0,
        want_dH=True, want_dW=True, max_rows=0, allow_status=0, sentinel=7.0):
    B, T, ds = batch.hidden_student.shape
    V = batch.w_student.shape[0]
    dH = torch.full((B, T, ds), sentinel, dtype=gh_dtype, device=DEV) if want_dH else None
    dW = torch.full((V, ds), float("nan"), dtype=torch.float32, device=DEV) if want_dW else None
    got = api.adwin_opd_kl_lmhead_fwd_bwd(
        batch.hidden_student, batch.w_student, batch.hidden_teacher, batch.w_teacher, batch.tokens,
        batch.window, batch.rollout_len, grad_scale=grad_scale, grad_mode=mode, flags=flags,
        grad_hidden=dH, grad_w=dW, want_lse=True, max_rows=max_rows)
    torch.cuda.synchronize()
    api.raise_on_dev_status(got.dev_status, allow=allow_status)
    got.dH, got.dW = dH, dW
    return got


def oracle(batch, mode, flags, grad_scale=1.0):
    return O.lmhead_fwd_bwd(bits(batch.hidden_student), bits(batch.w_student),
                            bits(batch.hidden_teacher), bits(batch.w_teacher),
                            batch.tokens.cpu().numpy(), batch.window.cpu().numpy(),
                            batch.rollout_len.cpu().numpy(), grad_scale=grad_scale, grad_mode=mode,
                            flags=flags & api.RANGE_FULL)


LOGIT_ABS = 1e-5   # bound on the error of a logit difference formed in fp32 (|z| of a few units)


def check_scalars(got, ref, mask, grad_mask=None, mode=api.GRAD_FULL_KL, alpha=1.0):
    ns = type("S", (), {})()
    ns.kl, ns.logratio, ns.gsq = got.kl, got.logratio, None
    P.check_scalars(ns, ref, RTOL, mask)
    # gsq: summed from the gradient entries where sweep 2 formed them (grad_mask, 1e-4), from the
    # single-sweep moments elsewhere (1e-3), plus the floor that fp32 leaves on a peaked row: every
    # entry g_k = alpha p_k ((z_k - u_k) - E_p[z - u]) carries an absolute error of about
    # |alpha| p_k eps with eps = 8 ulp of max(1, |E_p[z - u]|), which moves sum g^2 by at most
    # 2 sqrt(gsq) |alpha| eps (Cauchy-Schwarz with sum p^2 <= 1); negligible unless p is peaked.
    # With the sampled-token estimator gsq is c^2 times a well-conditioned factor and c is a
    # difference of computed logits, so the relative error of c, LOGIT_ABS / |c|, enters twice.
    q = got.gsq.double().cpu().numpy()
    b = ref["gsq"]
    rq = np.full(b.shape, P.RTOL_GSQ_SINGLE_SWEEP)
    if grad_mask is not None:
        rq[grad_mask] = P.RTOL_GSQ
    if mode == api.GRAD_SAMPLED:
        with np.errstate(divide="ignore", invalid="ignore"):
            rq = rq + 2.0 * LOGIT_ABS / np.abs(ref["logratio"])
    eps = 8 * 2.0 ** -23 * np.maximum(1.0, np.abs(ref["kl"] + ref["lse_s"] - ref["lse_t"]))
    floor = 2.0 * np.sqrt(np.abs(b)) * abs(alpha) * eps
    valid = mask & np.isfinite(b)
    with np.errstate(invalid="ignore"):
        lim_all = rq * np.abs(b) + floor + 1e-30
    err, lim = np.abs(q - b)[valid], lim_all[valid]
    assert (err <= lim).all(), f"gsq (mode {mode}): worst err/lim {np.max(err / lim):.3g}"
    assert (q[~mask] == 0).all()
    for a, b in ((getattr(got, "lse_s", None), ref["lse_s"]),
                 (getattr(got, "lse_t", None), ref["lse_t"])):
        if a is None:
            continue
        a = a.double().cpu().numpy()
        assert (np.abs(a - b)[mask] <= RTOL_LSE * np.maximum(1.0, np.abs(b))[mask]).all()
        assert (a[~mask] == 0).all()


def check_product(a, b, babs, name, out_store=0.0, cond=None, alpha=1.0):
    rowmax = np.abs(b).max(axis=-1, keepdims=True)
    lim = (RTOL + out_store) * np.abs(b) + RTOL * rowmax + 2.0 ** -9 * babs + 1e-300
    if cond is not None:     # fp32 floor of the centred difference inside g (see check_scalars)
        lim = lim + abs(alpha) * 8 * 2.0 ** -23 * cond
    worst = float(np.max(np.abs(a - b) / lim))
    assert worst <= 1.0, f"{name} entries: worst err/lim {worst:.3g}"
    n2 = np.linalg.norm(a - b, axis=-1)
    d2 = np.linalg.norm(b, axis=-1)
    fl = 0.0 if cond is None else abs(alpha) * 8 * 2.0 ** -23 * np.linalg.norm(cond, axis=-1)
    assert (n2 <= (RTOL + STORE + out_store) * d2 + fl + 1e-300).all(), \
        f"{name} rows: worst {float(np.max(n2 / (d2 + 1e-300))):.3g}"


def check_all(batch, got, ref, flags, sentinel=7.0, mode=api.GRAD_FULL_KL, alpha=1.0):
    T = batch.tokens.shape[1]
    w, r = batch.window.cpu().numpy(), batch.rollout_len.cpu().numpy()
    mask = P.processed_mask(w, r, T, bool(flags & api.RANGE_FULL))
    gmask = P.processed_mask(w, r, T, False)
    with_grad = got.dH is not None or got.dW is not None
    check_scalars(got, ref, mask, grad_mask=gmask if with_grad else None, mode=mode, alpha=alpha)
    if got.dH is not None:
        a = got.dH.double().cpu().numpy()
        check_product(a[gmask], ref["dH"][gmask], ref["dH_abs"][gmask], "dH",
                      out_store=STORE if got.dH.dtype == torch.bfloat16 else 0.0,
                      cond=ref["dH_cond"][gmask], alpha=alpha)
        want = 0.0 if flags & api.ZERO_TAIL else sentinel
        assert (a[~gmask] == want).all()
    if got.dW is not None:
        a = got.dW.double().cpu().numpy()
        assert np.isfinite(a).all()
        if gmask.any():
            check_product(a, ref["dW"], ref["dW_abs"], "dW", cond=ref["dW_cond"], alpha=alpha)
            tot = np.linalg.norm(a - ref["dW"]) / np.linalg.norm(ref["dW"])
            assert tot <= RTOL + STORE
        else:
            assert (a == 0).all()


@pytest.mark.parametrize("mode", [api.GRAD_FULL_KL, api.GRAD_SAMPLED])
@pytest.mark.parametrize("flags", [0, api.RANGE_FULL, api.ZERO_TAIL, api.RANGE_FULL | api.ZERO_TAIL])
def test_small_case_modes_and_flags(mode, flags):
    batch = synth.make_lmhead_batch(DEV, B=3, T=200, V=1024, d_s=128, d_t=192, w_std=0.1,
                                    ragged_rollout=True)
    batch.window = torch.tensor([70, 200, 0], dtype=torch.int32, device=DEV)
    batch.rollout_len = torch.tensor([200, 131, 50], dtype=torch.int32, device=DEV)
    got = run(batch, mode=mode, flags=flags, gh_dtype=torch.float32, grad_scale=-0.5)
    check_all(batch, got, oracle(batch, mode, flags, grad_scale=-0.5), flags, mode=mode, alpha=-0.5)


@pytest.mark.parametrize("V,ds,dt", [(1000, 72, 200), (264, 64, 64), (2048 + 8, 320, 136)])
def test_ragged_vocabulary_and_hidden_sizes(V, ds, dt):
    # V not a multiple of the 256-column tile, hidden sizes not multiples of the 64-wide k-block
    batch = synth.make_lmhead_batch(DEV, B=2, T=150, V=V, d_s=ds, d_t=dt, w_std=0.15)
    batch.window = torch.tensor([150, 37], dtype=torch.int32, device=DEV)
    for mode in (api.GRAD_FULL_KL, api.GRAD_SAMPLED):
        got = run(batch, mode=mode)
        check_all(batch, got, oracle(batch, mode, 0), 0, mode=mode)


@pytest.mark.parametrize("with_grad", [False, True])
def test_peaked_rows(with_grad):
    """Confident positions: the student's hidden state is a multiple of one token's embedding, so
    p puts ~0.999 on that token (the case in which a squared-norm formula that expands
    sum p^2 (delta - E delta)^2 loses digits).  Most positions sample the peak; a few do not."""
    batch = synth.make_lmhead_batch(DEV, B=2, T=140, V=1024, d_s=128, d_t=192, w_std=0.1)
    batch.window = torch.tensor([140, 90], dtype=torch.int32, device=DEV)
    g = torch.Generator(device=DEV)
    g.manual_seed(11)
    peak = torch.randint(0, 1024, (2, 140), generator=g, device=DEV)
    scale = 15.0 / (128 * 0.1 ** 2)
    batch.hidden_student = (batch.w_student[peak].float() * scale).to(torch.bfloat16).contiguous()
    batch.tokens = peak.to(torch.int32)
    off_peak = torch.rand((2, 140), generator=g, device=DEV) < 0.05
    batch.tokens[off_peak] = (batch.tokens[off_peak] + 17) % 1024
    got = run(batch, want_dH=with_grad, want_dW=with_grad)
    ref = oracle(batch, api.GRAD_FULL_KL, 0)
    T = 140
    w, r = batch.window.cpu().numpy(), batch.rollout_len.cpu().numpy()
    mask = P.processed_mask(w, r, T, False)
    if with_grad:
        check_all(batch, got, ref, 0)
    else:
        # no gradient: the moment form, centred on the sampled token.  Where the sampled token is
        # the peak it keeps its accuracy; off-peak samples of a peaked row are excluded from the
        # gsq comparison (documented limit of the single-sweep form)
        on_peak = mask & ~off_peak.cpu().numpy()
        ns = type("S", (), {})()
        ns.kl, ns.logratio, ns.gsq = got.kl, got.logratio, None
        P.check_scalars(ns, ref, RTOL, mask)
        q = got.gsq.double().cpu().numpy()
        rel = np.abs(q - ref["gsq"])[on_peak] / ref["gsq"][on_peak]
        assert rel.max() <= P.RTOL_GSQ_SINGLE_SWEEP, rel.max()


def test_scalars_only_and_single_gradients():
    batch = synth.make_lmhead_batch(DEV, B=2, T=130, V=768, d_s=128, d_t=128, w_std=0.1)
    ref = oracle(batch, api.GRAD_FULL_KL, 0)
    for want_dH, want_dW in ((False, False), (True, False), (False, True)):
        got = run(batch, want_dH=want_dH, want_dW=want_dW)
        check_all(batch, got, ref, 0)


def test_all_windows_empty_gives_zero_gradients():
    batch = synth.make_lmhead_batch(DEV, B=2, T=64, V=512, d_s=64, d_t=64)
    batch.window = torch.zeros(2, dtype=torch.int32, device=DEV)
    got = run(batch)
    assert (got.kl == 0).all() and (got.logratio == 0).all()
    assert (got.dW == 0).all() and (got.dH == 7.0).all()
    got = run(batch, flags=api.RANGE_FULL)           # scalars over the rollout, still no gradient
    assert (got.kl > 0).all() and (got.dW == 0).all()


def test_out_of_range_token_and_workspace_bound_are_reported():
    batch = synth.make_lmhead_batch(DEV, B=1, T=140, V=512, d_s=64, d_t=64, w_std=0.1)
    batch.window[:] = 140
    batch.tokens[0, 3] = 512
    batch.tokens[0, 130] = -4
    got = run(batch, allow_status=api.DEV_TOKEN_RANGE, want_dH=False, want_dW=False)
    assert int(got.dev_status.item()) == api.DEV_TOKEN_RANGE
    c = got.logratio.cpu().numpy()[0]
    assert np.isnan(c[3]) and np.isnan(c[130]) and np.isfinite(np.delete(c, [3, 130])).all()
    ref = oracle(batch, api.GRAD_FULL_KL, 0)
    np.testing.assert_allclose(got.kl.cpu().numpy(), ref["kl"], rtol=RTOL, atol=RTOL)
    # a bound on the processed positions that the lengths on the device exceed
    batch.tokens[0, 3] = 1
    batch.tokens[0, 130] = 2
    batch2 = synth.make_lmhead_batch(DEV, B=4, T=300, V=512, d_s=64, d_t=64)
    batch2.window = torch.full((4,), 300, dtype=torch.int32, device=DEV)
    got = run(batch2, max_rows=128, allow_status=api.DEV_WORKSPACE)
    assert int(got.dev_status.item()) == api.DEV_WORKSPACE
    assert (got.dW == 0).all()


def test_host_detected_errors():
    batch = synth.make_lmhead_batch(DEV, B=1, T=16, V=256, d_s=64, d_t=64)
    with pytest.raises(api.AdwinError) as e:
        api.adwin_opd_kl_lmhead_fwd_bwd(batch.hidden_student, batch.w_student, batch.hidden_teacher,
                                        batch.w_teacher, batch.tokens, batch.window, flags=64)
    assert e.value.code == 4
    with pytest.raises(api.AdwinError) as e:
        api.adwin_opd_kl_lmhead_fwd_bwd(batch.hidden_student, batch.w_student, batch.hidden_teacher,
                                        batch.w_teacher, batch.tokens, batch.window,
                                        workspace=torch.empty(4096, dtype=torch.uint8, device=DEV))
    assert e.value.code == 6
    odd = synth.make_lmhead_batch(DEV, B=1, T=16, V=260, d_s=64, d_t=64)     # V % 8 != 0
    with pytest.raises(api.AdwinError) as e:
        api.adwin_opd_kl_lmhead_fwd_bwd(odd.hidden_student, odd.w_student, odd.hidden_teacher,
                                        odd.w_teacher, odd.tokens, odd.window)
    assert e.value.code == 8


def test_results_are_bitwise_reproducible():
    batch = synth.make_lmhead_batch(DEV, B=2, T=260, V=1536, d_s=128, d_t=192, w_std=0.1)
    a = run(batch, mode=api.GRAD_FULL_KL)
    b = run(batch, mode=api.GRAD_FULL_KL)
    for x, y in ((a.kl, b.kl), (a.gsq, b.gsq), (a.dH, b.dH), (a.dW, b.dW)):
        assert torch.equal(x, y)


@pytest.mark.parametrize("mode", [api.GRAD_FULL_KL, api.GRAD_SAMPLED])
def test_config5_reduced_rows_full_vocabulary(mode):
    # the paper-scale vocabulary and hidden sizes on a few hundred positions
    batch = synth.make_lmhead_batch(DEV, B=2, T=192)
    batch.window = torch.tensor([100, 192], dtype=torch.int32, device=DEV)
    got = run(batch, mode=mode)
    check_all(batch, got, oracle(batch, mode, 0), 0, mode=mode)


def test_config5_full_size_sampled_rows_and_gradient_identities():
    """Config 5 in the launch configuration the benchmark times: per-token scalars and dH rows on
    sampled positions against the oracle; dW through two identities that hold at any size:
    its column sums vanish (every row of G sums to zero) and <W_s, dW> = <H_s, dH> (both equal
    sum_r g_r . z_r)."""
    batch = synth.make_lmhead_batch(DEV)
    B, T, ds = batch.hidden_student.shape
    nw = int(torch.minimum(batch.window, batch.rollout_len).sum())
    got = run(batch, gh_dtype=torch.float32, max_rows=nw)
    w = batch.window.cpu().numpy()
    rng = np.random.default_rng(5)
    picks = []
    for b in range(B):
        ts = {0, int(w[b]) - 1, int(rng.integers(0, w[b])), int(rng.integers(0, w[b]))}
        picks += [(b, t) for t in sorted(ts)]
    Ws64, Wt64 = O.widen(bits(batch.w_student)), O.widen(bits(batch.w_teacher))
    kl = got.kl.double().cpu().numpy()
    assert (kl[np.arange(T)[None, :] >= w[:, None]] == 0).all()
    for (b, t) in picks:
        z = O.widen(bits(batch.hidden_student[b, t])) @ Ws64.T
        u = O.widen(bits(batch.hidden_teacher[b, t])) @ Wt64.T
        r = O.row(z, u, int(batch.tokens[b, t]))
        floor = RTOL * max(1.0, abs(r["lse_s"] - r["lse_t"]))
        assert abs(kl[b, t] - r["kl"]) <= RTOL * abs(r["kl"]) + floor
        assert abs(float(got.logratio[b, t]) - r["c"]) <= RTOL * abs(r["c"]) + floor
        assert abs(float(got.gsq[b, t]) - r["gsq"]) <= P.RTOL_GSQ_SINGLE_SWEEP * r["gsq"]
        assert abs(float(got.lse_s[b, t]) - r["lse_s"]) <= RTOL_LSE * max(1.0, abs(r["lse_s"]))
        check_product(got.dH[b, t].double().cpu().numpy()[None], (r["g"] @ Ws64)[None],
                      (np.abs(r["g"]) @ np.abs(Ws64))[None], "dH")
    dW = got.dW.double()
    scale = float(dW.abs().sum(dim=0).max())
    assert float(dW.sum(dim=0).abs().max()) <= 2e-3 * scale
    gm = (torch.arange(T, device=DEV)[None, :] < batch.window[:, None])
    lhs = float((dW * batch.w_student.double()).sum())
    rhs = float((got.dH.double() * batch.hidden_student.double())[gm].sum())
    assert abs(lhs - rhs) <= 2e-3 * max(abs(lhs), abs(rhs))


# ---------------------------------------------------------------- weight-space alignment audit
def check_weight_align(batch, cands, mode, rho_star=0.0):
    al = api.adwin_lmhead_weight_align(batch.hidden_student, batch.w_student, batch.hidden_teacher,
                                       batch.w_teacher, batch.tokens, batch.rollout_len, cands,
                                       rho_star, grad_mode=mode)
    torch.cuda.synchronize()
    api.raise_on_dev_status(al.dev_status)
    ref = O.lmhead_weight_cosine(bits(batch.hidden_student), bits(batch.w_student),
                                 bits(batch.hidden_teacher), bits(batch.w_teacher),
                                 batch.tokens.cpu().numpy(), batch.rollout_len.cpu().numpy(), cands,
                                 grad_mode=mode)
    st = al.batch_stats.cpu().numpy()
    # G is rounded to bf16 once: the bin matrices carry ~1e-3 relative noise, the cosines of their
    # sums a few 1e-3 absolute at most
    np.testing.assert_allclose(st[:, 0], ref["micro"], rtol=0, atol=4e-3)
    rho = st[:, 0]
    np.testing.assert_allclose(st[:, 1], np.where(rho ** 2 < 1, rho ** 2 / (1 - rho ** 2), np.inf),
                               rtol=1e-12)
    star = rho_star if rho_star > 0 else np.sqrt(2) / 2
    np.testing.assert_array_equal(st[:, 2], (rho >= star).astype(float))
    r = batch.rollout_len.cpu().numpy()
    np.testing.assert_array_equal(st[:, 3], [np.minimum(L, r).sum() for L in cands])
    adm = [L for L, a in zip(cands, st[:, 2]) if a]
    assert int(al.L_next.item()) == (adm[0] if adm else cands[-1])
    assert int(al.flags.item()) == (0 if adm else api.ALIGN_NONE_ADMISSIBLE)
    # per-token outputs over the whole rollout, as the fused pass gives them
    full = oracle(batch_with_window(batch, batch.rollout_len), mode, 0)
    mask = P.processed_mask(r, r, batch.tokens.shape[1], False)
    check_scalars(al, full, mask, grad_mask=mask, mode=mode)
    return st, ref


def batch_with_window(batch, window):
    import copy
    b = copy.copy(batch)
    b.window = window
    return b


@pytest.mark.parametrize("mode", [api.GRAD_FULL_KL, api.GRAD_SAMPLED])
def test_weight_space_alignment_against_the_oracle(mode):
    batch = synth.make_lmhead_batch(DEV, B=3, T=256, V=512, d_s=64, d_t=64, w_std=0.15)
    batch.rollout_len = torch.tensor([256, 130, 70], dtype=torch.int32, device=DEV)
    st, ref = check_weight_align(batch, [64, 128, 192], mode, rho_star=0.5)
    assert st[-1, 0] < 1.0 - 1e-3        # the longest candidate does not cover the first rollout


def test_weight_space_alignment_sees_cross_sample_cancellation():
    # every position shares one hidden state: dW = (sum of the logit gradients) h^T, so the cosine
    # is the one between summed logit gradients and differs from the logit-space rho, which has no
    # cross terms (and is monotone in L)
    batch = synth.make_lmhead_batch(DEV, B=2, T=192, V=512, d_s=64, d_t=64, w_std=0.15)
    batch.hidden_student = batch.hidden_student[0, 0].expand(2, 192, 64).contiguous()
    st, ref = check_weight_align(batch, [64, 128, 192], api.GRAD_FULL_KL)
    lal = api.adwin_lmhead_weight_align(batch.hidden_student, batch.w_student, batch.hidden_teacher,
                                        batch.w_teacher, batch.tokens, batch.rollout_len,
                                        [64, 128, 192])
    logit = api.adwin_probe_align(lal.kl, lal.logratio, lal.gsq, batch.rollout_len,
                                  batch.rollout_len,
                                  torch.tensor([64, 128, 192], dtype=torch.int32, device=DEV))
    torch.cuda.synchronize()
    rho_logit = logit.batch_stats[:3, 0].cpu().numpy()
    assert np.abs(st[:2, 0] - rho_logit[:2]).min() > 1e-2
    assert st[2, 0] == pytest.approx(1.0, abs=1e-6)      # L covers every rollout


def test_weight_space_alignment_rejects_bad_candidate_lists():
    batch = synth.make_lmhead_batch(DEV, B=1, T=128, V=256, d_s=64, d_t=64)
    for bad in ([100], [128, 64], [64, 64], []):
        with pytest.raises(api.AdwinError) as e:
            api.adwin_lmhead_weight_align(batch.hidden_student, batch.w_student,
                                          batch.hidden_teacher, batch.w_teacher, batch.tokens,
                                          batch.rollout_len, bad)
        assert e.value.code == 2
