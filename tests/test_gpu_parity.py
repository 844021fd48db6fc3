"""GPU parity: the CUDA path (through the C ABI) against the float64 oracle, element by element."""
import math

import numpy as np
import pytest
import torch

from oracle import adwin_oracle as O
from paper_2605_28396_b200 import api, synth
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PATHS = {"staged": api.FORCE_STAGED, "generic": api.FORCE_GENERIC, "default": 0}


def run_and_check(batch, *, grad_dtype, grad_mode=api.GRAD_FULL_KL, flags=0, grad_scale=1.0,
                  allow_status=0, sentinel=7.0, rtol_gsq_grad=None):
    B, T, V = batch.shape
    grad = None
    if grad_dtype is not None:
        grad = torch.full((B, T, V), sentinel, dtype=grad_dtype, device=batch.student.device)
    got = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                   batch.rollout_len, grad_scale=grad_scale, grad_mode=grad_mode,
                                   flags=flags, grad=grad, want_lse=True)
    torch.cuda.synchronize()
    api.raise_on_dev_status(got.dev_status, allow=allow_status)
    oflags = flags & (api.ZERO_TAIL | api.RANGE_FULL)
    ref = P.oracle_batch(batch, grad_scale=grad_scale, grad_mode=grad_mode, flags=oflags,
                         want_grad=grad is not None,
                         grad_init=None if grad is None else np.full((B, T, V), sentinel))
    rtol = P.rtol_for(batch.student.dtype, grad_dtype)
    w, r = batch.window.cpu().numpy(), batch.rollout_len.cpu().numpy()
    mask = P.processed_mask(w, r, T, bool(flags & api.RANGE_FULL))
    gmask = P.processed_mask(w, r, T, False) if grad is not None else None
    P.check_scalars(got, ref, rtol, mask, grad_mask=gmask, rtol_gsq_grad=rtol_gsq_grad)
    if grad is not None:
        g = got.grad.double().cpu().numpy()
        wmask = P.processed_mask(w, r, T, False)
        guard = 1e-4 if (grad_dtype == torch.float32 and grad_mode == api.GRAD_FULL_KL) else None
        P.check_grad_rows(g[wmask], ref["grad"][wmask], rtol, store=P.STORE[grad_dtype],
                          guard=guard)
        # rows outside the window: untouched (sentinel) or exactly zero with ZERO_TAIL
        want = 0.0 if flags & api.ZERO_TAIL else sentinel
        assert (g[~wmask] == want).all()
    return got, ref


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode", [api.GRAD_FULL_KL, api.GRAD_SAMPLED])
def test_config1_fp32(path, mode):
    batch = synth.make_batch(1, device=DEV)
    run_and_check(batch, grad_dtype=torch.float32, grad_mode=mode, flags=PATHS[path])


@pytest.mark.parametrize("path", PATHS)
def test_config2_bf16_full_size(path):
    batch = synth.make_batch(2, device=DEV)
    run_and_check(batch, grad_dtype=torch.bfloat16, flags=PATHS[path])


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("mode", [api.GRAD_FULL_KL, api.GRAD_SAMPLED])
def test_config3_reduced_T_full_vocab(path, mode):
    batch = synth.make_batch(3, device=DEV, B=4, T=48)           # windows 6,12,24,48
    run_and_check(batch, grad_dtype=torch.bfloat16, grad_mode=mode, flags=PATHS[path])


@pytest.mark.parametrize("path", PATHS)
def test_config4_probe_reduced_with_ragged_rollouts(path):
    batch = synth.make_batch(4, device=DEV, B=4, T=64, ragged_rollout=True)
    got, ref = run_and_check(batch, grad_dtype=None, flags=api.RANGE_FULL | PATHS[path])
    cands = torch.tensor([4, 8, 16, 32, 64], dtype=torch.int32, device=DEV)
    al = api.adwin_probe_align(got.kl, got.logratio, got.gsq, batch.window, batch.rollout_len,
                               cands, 0.0)
    torch.cuda.synchronize()
    w, r = batch.window.cpu().numpy(), batch.rollout_len.cpu().numpy()
    # (i) same per-token inputs through the oracle's audit: sums agree to float64 rounding
    same = O.probe_align(got.kl.cpu().numpy(), got.logratio.cpu().numpy(), got.gsq.cpu().numpy(),
                         w, r, cands.cpu().numpy(), math.sqrt(2) / 2)
    np.testing.assert_allclose(al.seq_stats.cpu().numpy(), same["seq_stats"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(al.seq_full.cpu().numpy(), same["seq_full"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(al.batch_stats.cpu().numpy(), same["batch_stats"], rtol=1e-12)
    assert int(al.L_next.item()) == same["L_next"] and int(al.flags.item()) == same["flags"]
    # (ii) end to end against the oracle run from the logits
    e2e = O.probe_align(ref["kl"], ref["logratio"], ref["gsq"], w, r, cands.cpu().numpy(),
                        math.sqrt(2) / 2)
    np.testing.assert_allclose(al.batch_stats.cpu().numpy()[:, :2], e2e["batch_stats"][:, :2],
                               rtol=P.RTOL_SUM)
    near = np.abs(e2e["batch_stats"][:-1, 0] - math.sqrt(2) / 2).min() <= 1e-6
    assert int(al.L_next.item()) == e2e["L_next"] or near


@pytest.mark.parametrize("path", PATHS)
def test_range_full_with_gradient_inside_window_only(path):
    batch = synth.make_batch(2, device=DEV, B=3, T=40, V=4096, ragged_rollout=True)
    batch.window = torch.tensor([5, 17, 0], dtype=torch.int32, device=DEV)
    batch.rollout_len = torch.tensor([40, 17, 9], dtype=torch.int32, device=DEV)
    run_and_check(batch, grad_dtype=torch.bfloat16, flags=api.RANGE_FULL | PATHS[path])
    run_and_check(batch, grad_dtype=torch.float32,
                  flags=api.RANGE_FULL | api.ZERO_TAIL | PATHS[path])


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("in_dt,g_dt", [(1, torch.bfloat16), (1, torch.float32),
                                        (2, torch.float32), (2, torch.bfloat16)])
def test_dtype_combinations_and_grad_scale(path, in_dt, g_dt):
    batch = synth.make_batch(in_dt, device=DEV, B=2, T=12, V=8192)
    batch.window = torch.tensor([12, 5], dtype=torch.int32, device=DEV)
    for mode in (api.GRAD_FULL_KL, api.GRAD_SAMPLED):
        run_and_check(batch, grad_dtype=g_dt, grad_mode=mode, grad_scale=-0.125,
                      flags=PATHS[path] | api.ZERO_TAIL)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("in_dt,g_dt", [(2, torch.bfloat16), (1, torch.float32), (2, None)])
def test_sampled_token_far_below_the_row_maximum(path, in_dt, g_dt):
    """Rows whose sampled token has a vanishing probability (the staged kernel's shared reference
    overflows there and the row is redone with a running maximum), next to ordinary rows."""
    batch = synth.make_batch(in_dt, device=DEV, B=2, T=6, V=8192)
    batch.window = torch.tensor([6, 4], dtype=torch.int32, device=DEV)
    for (b, t, gap_s, gap_t) in [(0, 1, 90.0, 0.0), (0, 3, 0.0, 120.0), (1, 2, 60.0, 70.0),
                                 (1, 5, 200.0, 200.0)]:
        y = int(batch.tokens[b, t])
        batch.student[b, t, y] = batch.student[b, t].float().max() - gap_s
        batch.teacher[b, t, y] = batch.teacher[b, t].float().max() - gap_t
    flags = PATHS[path] | (api.RANGE_FULL if g_dt is None else 0)
    run_and_check(batch, grad_dtype=g_dt, flags=flags)
    run_and_check(batch, grad_dtype=g_dt, grad_mode=api.GRAD_SAMPLED, flags=flags)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("in_dt,g_dt,shift", [(1, torch.float32, 8.0), (2, torch.bfloat16, 50.0),
                                              (2, torch.bfloat16, 1000.0), (2, None, 1000.0)])
def test_teacher_rows_shifted_by_a_constant(path, in_dt, g_dt, shift):
    """The divergence does not depend on a constant added to a logit row.  The kernels work with
    z - u in fp32, whose rounding grows with such an offset (offset * 2^-24 against differences of
    order one): an offset of 8 must stay inside the fp32 tolerance of 1e-5 (an offset of 50
    already costs 1.3e-5 on a gradient row in any fp32 evaluation of z - u), one of 1000 inside
    the bf16 tolerance."""
    batch = synth.make_batch(in_dt, device=DEV, B=2, T=10, V=8192)
    batch.window = torch.tensor([10, 6], dtype=torch.int32, device=DEV)
    batch.teacher = (batch.teacher.float() + shift).to(batch.teacher.dtype)
    # With the offset of 1000 the squared norm of a written gradient row is held to the arithmetic
    # tolerance of the dtype instead of 1e-4: the staged kernel forms coef*(z-u) - coef*E_p[z-u]
    # uncentred, which costs offset * 2^-24 = 6e-5 relative on every entry there.
    for mode in (api.GRAD_FULL_KL, api.GRAD_SAMPLED):
        run_and_check(batch, grad_dtype=g_dt, grad_mode=mode, flags=PATHS[path],
                      rtol_gsq_grad=2e-3 if shift >= 1000.0 else None)


@pytest.mark.parametrize("g_dt", [torch.bfloat16, None])
def test_teacher_logits_outside_the_range_of_the_polynomial_exponential(g_dt):
    """The staged kernel takes the exponential of the first teacher pair of every 16-byte piece
    from a polynomial that is only valid on a clamped range: entries far below the reference must
    still count as nil, and one far above it must still send the row to the safe path."""
    batch = synth.make_batch(2, device=DEV, B=2, T=5, V=8192)
    batch.window = torch.tensor([5, 3], dtype=torch.int32, device=DEV)
    first_pair = torch.arange(0, 8192, 8, device=DEV)
    batch.teacher[0, 1, first_pair[5:400]] = -3.0e4            # far below: 2^x underflows
    batch.teacher[0, 1, first_pair[5:400] + 1] = -250.0
    batch.teacher[1, 0, first_pair[::7]] = -1.0e3
    uy = float(batch.teacher[0, 3, int(batch.tokens[0, 3])])
    batch.teacher[0, 3, first_pair[17]] = uy + 96.0              # far above, polynomial position
    uy = float(batch.teacher[1, 2, int(batch.tokens[1, 2])])
    batch.teacher[1, 2, first_pair[900] + 1] = uy + 71.0         # just inside the clamp
    flags = api.RANGE_FULL if g_dt is None else 0
    run_and_check(batch, grad_dtype=g_dt, flags=flags)
    run_and_check(batch, grad_dtype=g_dt, grad_mode=api.GRAD_SAMPLED, flags=flags)


@pytest.mark.parametrize("V", [1, 2, 7, 8, 9, 1001, 4100, 65537])
def test_odd_vocab_sizes(V):
    batch = synth.make_batch(2, device=DEV, B=2, T=6, V=V)
    batch.window = torch.tensor([6, 3], dtype=torch.int32, device=DEV)
    run_and_check(batch, grad_dtype=torch.bfloat16)
    run_and_check(batch, grad_dtype=None)


@pytest.mark.parametrize("V", [409600, 1048576])
def test_vocabulary_beyond_what_tensor_memory_holds(V):
    """The staged kernel parks the streamed chunks of a row slice in tensor memory between its
    sweeps when they fit (up to 5 chunks + the resident slots per CTA, with clusters of up to 4);
    larger rows go back to fetching those chunks a second time through the shared-memory ring.
    Both sizes here are beyond the limit (the paper-scale vocabulary is inside it)."""
    batch = synth.make_batch(3, device=DEV, B=1, T=5, V=V)
    batch.window = torch.tensor([4], dtype=torch.int32, device=DEV)
    for mode in (api.GRAD_FULL_KL, api.GRAD_SAMPLED):
        run_and_check(batch, grad_dtype=torch.bfloat16, grad_mode=mode, flags=api.FORCE_STAGED)


@pytest.mark.parametrize("path", PATHS)
def test_padded_row_stride(path):
    B, T, V, ld = 2, 5, 4096, 4096 + 64
    base = synth.make_batch(2, device=DEV, B=B, T=T, V=ld)
    batch = synth.Batch(base.student[..., :V], base.teacher[..., :V],
                        torch.randint(0, V, (B, T), dtype=torch.int32, device=DEV),
                        torch.tensor([5, 2], dtype=torch.int32, device=DEV), base.rollout_len, 2)
    grad = torch.full((B, T, ld), 3.0, dtype=torch.bfloat16, device=DEV)
    got = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                   batch.rollout_len, grad=grad[..., :V], flags=PATHS[path])
    torch.cuda.synchronize()
    ref = O.opd_kl_fwd_bwd(synth.bits_for_oracle(batch.student.contiguous()),
                           synth.bits_for_oracle(batch.teacher.contiguous()),
                           batch.tokens.cpu().numpy(), batch.window.cpu().numpy(), None)
    mask = P.processed_mask(batch.window.cpu().numpy(), np.array([T, T]), T)
    P.check_scalars(got, ref, 2e-3, mask)
    g = grad.double().cpu().numpy()
    P.check_grad_rows(g[..., :V][mask], ref["grad"][mask], 2e-3, store=2.0 ** -8)
    assert (g[..., V:] == 3.0).all()                     # padding columns never written


def test_unaligned_row_stride_runs_through_the_generic_kernel():
    B, T, V, ld = 2, 4, 1000, 1003                       # rows not 16-byte aligned
    base = synth.make_batch(2, device=DEV, B=B, T=T, V=ld)
    s, t = base.student[..., :V], base.teacher[..., :V]
    tok = torch.randint(0, V, (B, T), dtype=torch.int32, device=DEV)
    win = torch.tensor([4, 4], dtype=torch.int32, device=DEV)
    gbuf = torch.zeros((B, T, ld), dtype=torch.float32, device=DEV)
    got = api.adwin_opd_kl_fwd_bwd(s, t, tok, win, None, grad=gbuf[..., :V])
    torch.cuda.synchronize()
    ref = O.opd_kl_fwd_bwd(synth.bits_for_oracle(s.contiguous()),
                           synth.bits_for_oracle(t.contiguous()), tok.cpu().numpy(),
                           win.cpu().numpy(), None)
    mask = np.ones((B, T), dtype=bool)
    P.check_scalars(got, ref, 2e-3, mask)
    P.check_grad_rows(gbuf[..., :V].double().cpu().numpy()[mask], ref["grad"][mask], 2e-3)


@pytest.mark.parametrize("path", PATHS)
def test_degenerate_windows(path):
    batch = synth.make_batch(2, device=DEV, B=4, T=8, V=4096)
    batch.window = torch.tensor([0, 8, 100, 3], dtype=torch.int32, device=DEV)     # W=0, W>T
    batch.rollout_len = torch.tensor([8, 0, 5, 8], dtype=torch.int32, device=DEV)  # R=0, W>R
    got, _ = run_and_check(batch, grad_dtype=torch.bfloat16, flags=PATHS[path])
    seq, tot = api.adwin_window_reduce(got.kl, got.logratio, got.gsq, batch.window,
                                       batch.rollout_len)
    torch.cuda.synchronize()
    assert seq[:, 3].tolist() == [0.0, 0.0, 5.0, 3.0] and tot[3].item() == 8.0
    batch.window[:] = 0                                                            # nothing at all
    got, _ = run_and_check(batch, grad_dtype=torch.bfloat16, flags=PATHS[path])
    assert (got.kl == 0).all()


@pytest.mark.parametrize("path", PATHS)
def test_device_detected_conditions_set_status_bits(path):
    batch = synth.make_batch(2, device=DEV, B=2, T=6, V=4096)
    batch.tokens[0, 1] = 4096
    batch.tokens[1, 0] = -3
    got, ref = run_and_check(batch, grad_dtype=torch.bfloat16, flags=PATHS[path],
                             allow_status=api.DEV_TOKEN_RANGE)
    assert int(got.dev_status.item()) & api.DEV_TOKEN_RANGE
    assert torch.isnan(got.logratio[0, 1]) and torch.isnan(got.logratio[1, 0])
    assert torch.isfinite(got.kl).all()
    # invalid lengths are clamped and reported, never dereferenced out of range
    batch = synth.make_batch(2, device=DEV, B=3, T=6, V=4096)
    batch.window = torch.tensor([-2, 4, 6], dtype=torch.int32, device=DEV)
    batch.rollout_len = torch.tensor([6, -1, 9], dtype=torch.int32, device=DEV)
    got = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                   batch.rollout_len, flags=PATHS[path])
    torch.cuda.synchronize()
    assert int(got.dev_status.item()) & api.DEV_WINDOW
    assert (got.kl[0] == 0).all() and (got.kl[1] == 0).all() and (got.kl[2] != 0).all()


@pytest.mark.parametrize("path", PATHS)
def test_bitwise_reproducible(path):
    batch = synth.make_batch(3, device=DEV, B=2, T=16, V=151936)
    outs = []
    for _ in range(3):
        g = torch.zeros(batch.shape, dtype=torch.bfloat16, device=DEV)
        got = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                       batch.rollout_len, grad=g, flags=PATHS[path])
        torch.cuda.synchronize()
        outs.append((got.kl.clone(), got.logratio.clone(), got.gsq.clone(), g))
    for o in outs[1:]:
        for a, b in zip(outs[0], o):
            assert torch.equal(a, b)


def test_window_reduce_against_oracle():
    batch = synth.make_batch(2, device=DEV, B=6, T=64, V=4096, ragged_rollout=True)
    got, ref = run_and_check(batch, grad_dtype=torch.bfloat16)
    seq, tot = api.adwin_window_reduce(got.kl, got.logratio, got.gsq, batch.window,
                                       batch.rollout_len)
    torch.cuda.synchronize()
    w, r = batch.window.cpu().numpy(), batch.rollout_len.cpu().numpy()
    s_same, t_same = O.window_reduce(got.kl.cpu().numpy(), got.logratio.cpu().numpy(),
                                     got.gsq.cpu().numpy(), w, r)
    np.testing.assert_allclose(seq.cpu().numpy(), s_same, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(tot.cpu().numpy(), t_same, rtol=1e-13, atol=1e-13)
    s_ref, t_ref = O.window_reduce(ref["kl"], ref["logratio"], ref["gsq"], w, r)
    mask = P.processed_mask(w, r, 64)
    terms = [np.abs(ref[k] * mask).sum() for k in ("kl", "logratio", "gsq")] + [0.0]
    P.check_sums(tot.cpu().numpy(), t_ref, terms)
    seq2, tot2 = api.adwin_window_reduce(got.kl, got.logratio, None, batch.window, None)
    torch.cuda.synchronize()
    assert (seq2[:, 2] == 0).all() and tot2[2].item() == 0


def test_probe_align_default_candidates_and_flags():
    B, T = 5, 4096
    g = torch.Generator(device=DEV).manual_seed(5)
    gsq = torch.rand((B, T), device=DEV, generator=g)
    kl = torch.rand((B, T), device=DEV, generator=g)
    c = torch.randn((B, T), device=DEV, generator=g)
    win = torch.full((B,), 256, dtype=torch.int32, device=DEV)
    rl = torch.tensor([4096, 3000, 100, 2048, 64], dtype=torch.int32, device=DEV)
    al = api.adwin_probe_align(kl, c, gsq, win, rl)
    torch.cuda.synchronize()
    ref = O.probe_align(kl.cpu().numpy(), c.cpu().numpy(), gsq.cpu().numpy(), win.cpu().numpy(),
                        rl.cpu().numpy(), np.array(api.DEFAULT_CANDIDATES, np.int32), api.RHO_STAR)
    np.testing.assert_allclose(al.batch_stats.cpu().numpy(), ref["batch_stats"], rtol=1e-12)
    np.testing.assert_allclose(al.seq_stats.cpu().numpy(), ref["seq_stats"], rtol=1e-12)
    assert int(al.L_next.item()) == ref["L_next"] and int(al.flags.item()) == ref["flags"]
    # nothing admissible / degenerate norms
    gsq0 = torch.zeros((B, T), device=DEV)
    al = api.adwin_probe_align(kl, c, gsq0, win, rl)
    torch.cuda.synchronize()
    assert int(al.flags.item()) & api.ALIGN_DEGENERATE and int(al.L_next.item()) == 64
    gsq1 = torch.zeros((B, T), device=DEV)
    gsq1[:, 60] = 1.0
    gsq1[:, 3000:] = 100.0
    al = api.adwin_probe_align(kl, c, gsq1, win, None, rho_star=0.9)
    torch.cuda.synchronize()
    assert int(al.flags.item()) & api.ALIGN_NONE_ADMISSIBLE and int(al.L_next.item()) == 2048


@pytest.mark.parametrize("flags", [0, api.RANGE_FULL | api.ZERO_TAIL])
def test_host_buffer_entry_point_matches_device_entry_point(flags):
    batch = synth.make_batch(2, device="cpu", B=3, T=70, V=8192, ragged_rollout=True)
    batch.window = torch.tensor([70, 9, 33], dtype=torch.int32)
    batch.rollout_len = torch.tensor([70, 40, 20], dtype=torch.int32)
    pin = lambda x: x.contiguous().pin_memory()
    s_h, t_h, tok_h = pin(batch.student), pin(batch.teacher), pin(batch.tokens)
    g_h = torch.full(batch.shape, 5.0, dtype=torch.bfloat16).pin_memory()
    got = api.adwin_opd_kl_fwd_bwd_host(s_h, t_h, tok_h, batch.window, batch.rollout_len,
                                        device=DEV, grad=g_h, flags=flags, rows_per_stage=16,
                                        grad_scale=0.5)
    torch.cuda.synchronize()
    assert int(got.dev_status.item()) == 0
    dgrad = torch.full(batch.shape, 5.0, dtype=torch.bfloat16, device=DEV)
    ref = api.adwin_opd_kl_fwd_bwd(batch.student.to(DEV), batch.teacher.to(DEV),
                                   batch.tokens.to(DEV), batch.window.to(DEV),
                                   batch.rollout_len.to(DEV), grad=dgrad, flags=flags,
                                   grad_scale=0.5)
    torch.cuda.synchronize()
    # same kernels on the same values: only the staging layout differs
    assert torch.allclose(got.kl, ref.kl.cpu(), rtol=1e-6, atol=1e-7)
    assert torch.allclose(got.logratio, ref.logratio.cpu(), rtol=1e-6, atol=1e-7)
    assert torch.allclose(got.gsq, ref.gsq.cpu(), rtol=1e-5, atol=1e-12)
    assert torch.equal(g_h, dgrad.cpu())
    with pytest.raises(api.AdwinError):
        api.adwin_opd_kl_fwd_bwd_host(s_h, t_h, tok_h, torch.tensor([-1, 2, 3], dtype=torch.int32),
                                      None, device=DEV)


def _oracle_on_rows(batch, rows, **kw):
    """Oracle on selected (b, t) rows only: each row becomes a one-token sequence inside its window."""
    bs = torch.tensor([b for b, _ in rows], device=batch.student.device)
    ts = torch.tensor([t for _, t in rows], device=batch.student.device)
    s = synth.bits_for_oracle(batch.student[bs, ts].unsqueeze(1))
    t = synth.bits_for_oracle(batch.teacher[bs, ts].unsqueeze(1))
    tok = batch.tokens[bs, ts].unsqueeze(1).cpu().numpy()
    return O.opd_kl_fwd_bwd(s, t, tok, np.ones(len(rows), np.int32), None, **kw)


def _sample_rows(limits, per_seq, rng):
    """First, last and a few random processed rows of every sequence."""
    rows = []
    for b, n in enumerate(limits):
        if n <= 0:
            continue
        ts = {0, int(n) - 1} | {int(x) for x in rng.integers(0, int(n), size=per_seq)}
        rows += [(b, t) for t in sorted(ts)]
    return rows


def test_config3_full_size_in_the_bench_launch_configuration_on_sampled_rows():
    """The workload bench.py times, at full size, with the oracle on sampled rows plus the
    properties that hold at any size (untouched tail, zeroed scalars, reproducible sums)."""
    batch = synth.make_batch(3, device=DEV)
    B, T, V = batch.shape
    sentinel = 7.0
    grad = torch.full((B, T, V), sentinel, dtype=torch.bfloat16, device=DEV)
    got = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                   batch.rollout_len, grad=grad)
    torch.cuda.synchronize()
    api.raise_on_dev_status(got.dev_status)
    w = batch.window.cpu().numpy()
    rows = _sample_rows(w, 2, np.random.default_rng(3))
    ref = _oracle_on_rows(batch, rows)
    bs = torch.tensor([b for b, _ in rows], device=DEV)
    ts = torch.tensor([t for _, t in rows], device=DEV)
    sub = type("S", (), {})()
    sub.kl, sub.logratio, sub.gsq = (x[bs, ts].unsqueeze(1) for x in (got.kl, got.logratio, got.gsq))
    ones = np.ones((len(rows), 1), dtype=bool)
    P.check_scalars(sub, ref, 2e-3, ones, grad_mask=ones)
    P.check_grad_rows(grad[bs, ts].double().cpu().numpy(), ref["grad"][:, 0], 2e-3, store=2.0 ** -8)
    for b in range(B):                                   # rows past the window: never touched
        assert (grad[b, int(w[b]):] == sentinel).all()
        assert (got.kl[b, int(w[b]):] == 0).all() and (got.gsq[b, int(w[b]):] == 0).all()
    seq, tot = api.adwin_window_reduce(got.kl, got.logratio, got.gsq, batch.window, batch.rollout_len)
    torch.cuda.synchronize()
    mask = torch.arange(T, device=DEV)[None, :] < batch.window[:, None]
    want = (got.kl.double() * mask).sum()
    assert abs(tot[0].item() - want.item()) <= 1e-9 * abs(want.item())
    assert tot[3].item() == float(w.sum()) and torch.isfinite(got.kl).all() and (got.kl[mask] > -1e-4).all()


def test_config4_full_size_probe_pass_on_sampled_rows():
    """Delayed full-rollout probe at full size (B=8, T=8192, V=151936, ragged rollouts): one pass
    without a gradient, then the alignment audit; oracle on sampled rows, audit against the oracle's
    audit of the same per-token scalars."""
    batch = synth.make_batch(4, device=DEV, ragged_rollout=True, fill_all_rows=False)
    B, T, V = batch.shape
    got = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                   batch.rollout_len, flags=api.RANGE_FULL)
    torch.cuda.synchronize()
    api.raise_on_dev_status(got.dev_status)
    w, r = batch.window.cpu().numpy(), batch.rollout_len.cpu().numpy()
    rows = _sample_rows(r, 3, np.random.default_rng(4))
    ref = _oracle_on_rows(batch, rows, want_grad=False)
    bs = torch.tensor([b for b, _ in rows], device=DEV)
    ts = torch.tensor([t for _, t in rows], device=DEV)
    sub = type("S", (), {})()
    sub.kl, sub.logratio, sub.gsq = (x[bs, ts].unsqueeze(1) for x in (got.kl, got.logratio, got.gsq))
    P.check_scalars(sub, ref, 2e-3, np.ones((len(rows), 1), dtype=bool))
    for b in range(B):
        assert (got.kl[b, int(r[b]):] == 0).all()
    al = api.adwin_probe_align(got.kl, got.logratio, got.gsq, batch.window, batch.rollout_len)
    torch.cuda.synchronize()
    same = O.probe_align(got.kl.cpu().numpy(), got.logratio.cpu().numpy(), got.gsq.cpu().numpy(),
                         w, r, np.array(api.DEFAULT_CANDIDATES, np.int32), api.RHO_STAR)
    np.testing.assert_allclose(al.batch_stats.cpu().numpy(), same["batch_stats"], rtol=1e-12)
    np.testing.assert_allclose(al.seq_stats.cpu().numpy(), same["seq_stats"], rtol=1e-12, atol=1e-12)
    assert int(al.L_next.item()) == same["L_next"] and int(al.flags.item()) == same["flags"]
    rho = al.batch_stats[:, 0].cpu().numpy()
    assert (np.diff(rho[:-1]) >= -1e-12).all() and (rho <= 1 + 1e-12).all()
