"""GPU parity of the teacher-drift diagnostics (Section 3.1) against the float64 oracle: ranks and
survival counts bit-exact, entropies within the tolerance of the logits' dtype."""
import numpy as np
import pytest
import torch

from oracle import adwin_oracle as O
from paper_2605_28396_b200 import api, synth
from tests import parity as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _oracle_rows(teacher, tokens, rollout):
    u64 = teacher.double().cpu().numpy()
    tok = tokens.cpu().numpy()
    B, T, _ = u64.shape
    H = np.zeros((B, T))
    r = np.zeros((B, T), dtype=np.int64)
    for b in range(B):
        for t in range(int(rollout[b])):
            H[b, t], r[b, t] = O.teacher_drift_row(u64[b, t], int(tok[b, t]))
    return H, r


def _check(batch, ks=(1, 2, 5, 50)):
    B, T, V = batch.shape
    R = batch.rollout_len.cpu().numpy()
    got = api.adwin_teacher_drift(batch.teacher, batch.tokens, batch.rollout_len)
    cur = api.adwin_drift_curves(got.entropy, got.rank, batch.rollout_len, ks)
    torch.cuda.synchronize()
    api.raise_on_dev_status(got.dev_status)
    H, r = _oracle_rows(batch.teacher, batch.tokens, R)
    rtol = P.rtol_for(batch.teacher.dtype)
    a = got.entropy.double().cpu().numpy()
    # H = lse - E_q[u]: absolute accuracy is set by the scale of the log-sum-exp
    assert (np.abs(a - H) <= rtol * np.maximum(1.0, np.abs(H))).all(), np.abs(a - H).max()
    np.testing.assert_array_equal(got.rank.cpu().numpy(), r)          # integer work: exact
    mask = np.arange(T)[None, :] < R[:, None]
    assert (a[~mask] == 0).all()
    worst = np.maximum.accumulate(np.where(mask, r, 0), axis=1)
    np.testing.assert_array_equal(cur.worst_rank.cpu().numpy(), worst)
    S = cur.survival.cpu().numpy()
    for j, k in enumerate(ks):
        np.testing.assert_array_equal(S[j], O.topk_survival(r, R, k))  # counts over B: exact
    n = mask.sum(axis=0)
    np.testing.assert_array_equal(cur.n_active.cpu().numpy(), n)
    bf = np.where(mask, np.exp(H), 0.0).sum(axis=0) / np.maximum(n, 1)
    np.testing.assert_allclose(cur.bf_mean.cpu().numpy(), bf, rtol=5 * rtol * max(1.0, H.max()))


@pytest.mark.parametrize("cfg,V", [(1, 4096), (2, 32000), (3, 151936)])
def test_drift_on_the_configs(cfg, V):
    batch = synth.make_batch(cfg, device=DEV, B=3, T=24, V=V, ragged_rollout=True)
    batch.rollout_len = torch.tensor([24, 0, 13], dtype=torch.int32, device=DEV)
    _check(batch)


@pytest.mark.parametrize("V", [1, 2, 9, 1001, 4100])
def test_drift_on_odd_vocabularies_and_strides(V):
    base = synth.make_batch(2, device=DEV, B=2, T=6, V=V + 3)
    batch = synth.Batch(base.student[..., :V], base.teacher[..., :V],
                        torch.randint(0, V, (2, 6), dtype=torch.int32, device=DEV), base.window,
                        torch.tensor([6, 4], dtype=torch.int32, device=DEV), 2)
    _check(batch, ks=(1, 3))


def test_drift_with_ties_peaks_and_a_token_out_of_range():
    batch = synth.make_batch(2, device=DEV, B=2, T=5, V=8192)
    batch.teacher[0, 0, :] = 1.5                               # uniform: H = log V, every rank 1
    batch.teacher[0, 1, :] = -40.0
    batch.teacher[0, 1, 77] = 30.0                             # one-hot: H ~ 0
    batch.tokens[0, 1] = 77
    batch.teacher[1, 2, 100:110] = 25.0                        # ten-way tie at the top
    batch.tokens[1, 2] = 105
    _check(batch)
    got = api.adwin_teacher_drift(batch.teacher, batch.tokens, batch.rollout_len)
    assert abs(float(got.entropy[0, 0]) - np.log(8192)) < 1e-4 and int(got.rank[0, 0]) == 1
    assert int(got.rank[1, 2]) == 1
    batch.tokens[1, 3] = 8192
    bad = api.adwin_teacher_drift(batch.teacher, batch.tokens, batch.rollout_len)
    torch.cuda.synchronize()
    assert int(bad.dev_status.item()) == 1 and int(bad.rank[1, 3]) == 0


def test_drift_curves_over_many_rollouts_and_long_horizons():
    g = torch.Generator().manual_seed(5)
    B, T = 300, 3000
    rank = torch.randint(1, 2000, (B, T), generator=g, dtype=torch.int32)
    R = torch.randint(0, T + 1, (B,), generator=g, dtype=torch.int32)
    rank = torch.where(torch.arange(T)[None, :] < R[:, None], rank, torch.zeros_like(rank))
    H = torch.rand((B, T), generator=g) * 3
    ks = (1, 100, 1000, 1999)
    cur = api.adwin_drift_curves(H.to(DEV), rank.to(DEV), R.to(DEV), ks)
    torch.cuda.synchronize()
    r = rank.numpy().astype(np.int64)
    for j, k in enumerate(ks):
        want = (np.maximum.accumulate(r, axis=1) <= k).mean(axis=0)
        np.testing.assert_allclose(cur.survival[j].cpu().numpy(), want, rtol=0, atol=1e-15)
    np.testing.assert_array_equal(cur.worst_rank.cpu().numpy(), np.maximum.accumulate(r, axis=1))


def test_config3_full_size_drift_on_sampled_rows():
    """The drift pass at the size the bench times it (B=16, T=2048, V=151936): entropy and rank
    against the oracle on sampled rows, the curves against the same ranks on the host."""
    batch = synth.make_batch(3, device=DEV)
    B, T, V = batch.shape
    ks = (1, 5, 20)
    got = api.adwin_teacher_drift(batch.teacher, batch.tokens, batch.rollout_len)
    cur = api.adwin_drift_curves(got.entropy, got.rank, batch.rollout_len, ks)
    torch.cuda.synchronize()
    api.raise_on_dev_status(got.dev_status)
    rng = np.random.default_rng(8)
    tok = batch.tokens.cpu().numpy()
    for b in range(B):
        for t in sorted({0, T - 1} | {int(x) for x in rng.integers(0, T, 2)}):
            H, r = O.teacher_drift_row(batch.teacher[b, t].double().cpu().numpy(), int(tok[b, t]))
            assert abs(float(got.entropy[b, t]) - H) <= 2e-3 * max(1.0, abs(H))
            assert int(got.rank[b, t]) == r
    ranks = got.rank.cpu().numpy().astype(np.int64)
    R = batch.rollout_len.cpu().numpy()
    np.testing.assert_array_equal(cur.worst_rank.cpu().numpy(), np.maximum.accumulate(ranks, axis=1))
    for j, k in enumerate(ks):
        np.testing.assert_array_equal(cur.survival[j].cpu().numpy(), O.topk_survival(ranks, R, k))
    assert (cur.n_active.cpu().numpy() == B).all()
    bf = np.exp(got.entropy.double().cpu().numpy()).mean(axis=0)
    np.testing.assert_allclose(cur.bf_mean.cpu().numpy(), bf, rtol=1e-12)
