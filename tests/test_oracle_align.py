"""Pins of the oracle's alignment audit (Section 4.2): rho, SNR, threshold, L_next, macro/micro."""
import math
from pathlib import Path

import numpy as np
import pytest

from oracle import adwin_oracle as O

RNG = np.random.default_rng(99)
GOLDEN = Path(__file__).parent / "golden" / "paper_constants.txt"


def golden():
    out = {}
    for line in GOLDEN.read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            k, v = line.split("=")
            out[k.strip()] = v.strip()
    return out


def align(gsq, W, R, cands, rho_star=math.sqrt(2) / 2, kl=None, c=None):
    gsq = np.asarray(gsq, dtype=np.float64)
    kl = np.zeros_like(gsq) if kl is None else kl
    c = np.zeros_like(gsq) if c is None else c
    return O.probe_align(kl, c, gsq, np.asarray(W, np.int32), np.asarray(R, np.int32),
                         np.asarray(cands, np.int32), rho_star)


def test_threshold_constants_from_the_paper():
    g = golden()
    rho_star = math.sqrt(2) / 2
    assert round(rho_star, 3) == float(g["rho_star_printed"])
    # uniform per-token energy over T=4: Q(L)=L, so rho(2) = sqrt(1/2) = rho*: SNR = 1, admissible
    out = align(np.ones((1, 4)), [4], [4], [1, 2, 3], rho_star)
    bs = out["batch_stats"]
    assert bs[1, 0] == pytest.approx(rho_star, rel=1e-15)
    assert bs[1, 2] == pytest.approx(float(g["snr_at_rho_star"]), rel=1e-12)
    assert bs[0, 3] == 0.0 and bs[2, 3] == 1.0
    assert [int(x) for x in g["candidates"].split()] == [64, 128, 256, 512, 1024, 2048]


def test_inclusive_threshold_and_shortest_admissible():
    # rho(L) = sqrt(L/T); choose rho_star exactly representable as one of them
    T = 16
    gs = np.ones((1, T))
    out = align(gs, [T], [T], [4, 9, 12, 16], rho_star=0.75)     # rho(9) = 0.75 exactly
    assert out["batch_stats"][1, 0] == 0.75 and out["batch_stats"][1, 3] == 1.0
    assert out["L_next"] == 9 and out["flags"] == 0
    out = align(gs, [T], [T], [16, 12, 9, 4], rho_star=0.75)     # unsorted list: still the shortest
    assert out["L_next"] == 9
    out = align(gs, [T], [T], [1, 2, 3], rho_star=0.75)          # none admissible: largest + flag
    assert out["L_next"] == 3 and out["flags"] & O.ALIGN_NONE_ADMISSIBLE


def test_rho_monotone_in_unit_interval_and_one_at_full_length():
    B, T = 5, 64
    gs = RNG.uniform(0, 1, (B, T))
    R = RNG.integers(1, T + 1, B)
    W = np.minimum(R, 8)
    cands = [1, 2, 4, 8, 16, 32, 64, 128]
    out = align(gs, W, R, cands)
    rho = out["batch_stats"][:len(cands), 0]
    assert (np.diff(rho) >= 0).all() and rho[0] >= 0 and rho[-1] <= 1
    assert out["batch_stats"][6, 0] == 1.0 and out["batch_stats"][7, 0] == 1.0     # L >= max R
    assert (out["seq_stats"][:, 6, 3] == 1.0).all()
    for b in range(B):   # rho_b = 1 as soon as L >= R_b
        for j, L in enumerate(cands):
            if L >= R[b]:
                assert out["seq_stats"][b, j, 3] == 1.0


def test_snr_formula():
    gs = RNG.uniform(0, 1, (3, 20))
    out = align(gs, [5, 5, 5], [20, 20, 20], [3, 7, 11])
    for j in range(4):
        r = out["batch_stats"][j, 0]
        assert out["batch_stats"][j, 2] == pytest.approx(r * r / (1 - r * r), rel=1e-12)
    out = align(gs, [5, 5, 5], [20, 20, 20], [20])
    assert math.isinf(out["batch_stats"][0, 2])


def test_macro_differs_from_micro_on_a_constructed_case():
    # seq 0: all energy in the first token; seq 1: small energy spread evenly over 4 tokens.
    gs = np.array([[100.0, 0, 0, 0], [1.0, 1.0, 1.0, 1.0]])
    out = align(gs, [1, 1], [4, 4], [1])
    micro, macro = out["batch_stats"][0, 0], out["batch_stats"][0, 1]
    assert micro == pytest.approx(math.sqrt(101.0 / 104.0), rel=1e-14)
    assert macro == pytest.approx((1.0 + 0.5) / 2, rel=1e-14)
    assert macro < micro                                       # Figure 5: macro stays below micro


def test_prefix_sums_windows_slot_and_token_counts():
    B, T = 3, 10
    kl = RNG.uniform(0, 1, (B, T)); c = RNG.normal(0, 1, (B, T)); gs = RNG.uniform(0, 1, (B, T))
    W = [2, 10, 7]
    R = [10, 4, 7]
    cands = [3, 6]
    out = align(gs, W, R, cands, kl=kl, c=c)
    for b in range(B):
        for j, L in enumerate(cands + [W[b]]):
            n = min(L, R[b])
            assert out["seq_stats"][b, j, 0] == pytest.approx(gs[b, :n].sum(), rel=1e-14)
            assert out["seq_stats"][b, j, 1] == pytest.approx(kl[b, :n].sum(), rel=1e-14)
            assert out["seq_stats"][b, j, 2] == pytest.approx(c[b, :n].sum(), rel=1e-12, abs=1e-14)
        assert out["seq_full"][b, 0] == pytest.approx(gs[b, :R[b]].sum(), rel=1e-14)
        assert out["seq_full"][b, 1] == pytest.approx(kl[b, :R[b]].sum(), rel=1e-14)
    assert out["batch_stats"][0, 4] == 3 + 3 + 3
    assert out["batch_stats"][1, 4] == 6 + 4 + 6
    assert out["batch_stats"][2, 4] == 2 + 4 + 7


def test_degenerate_zero_full_norm():
    gs = np.zeros((2, 5)); gs[1, :] = 1.0
    out = align(gs, [2, 2], [5, 5], [2])
    assert out["flags"] & O.ALIGN_DEGENERATE
    assert out["seq_stats"][0, 0, 3] == 1.0
    assert out["seq_stats"][1, 0, 3] == pytest.approx(math.sqrt(0.4))


@pytest.mark.parametrize("mode", [O.MODE_FULL_KL, O.MODE_SAMPLED])
def test_closed_form_equals_literal_dot_product_cosine(mode):
    # Materialise the gradient of every rollout position, mask it to the prefix, and take the
    # cosine from the dot product; it must equal sqrt(Q(L)/Q_full) built from per-token gsq.
    B, T, V = 3, 9, 12
    z = RNG.normal(0, 2, (B, T, V)).astype(np.float32)
    u = (z + RNG.normal(0, 1, (B, T, V))).astype(np.float32)
    y = RNG.integers(0, V, (B, T)).astype(np.int32)
    R = np.array([9, 5, 7], dtype=np.int32)
    W = np.array([9, 9, 9], dtype=np.int32)
    full = O.opd_kl_fwd_bwd(z, u, y, W, R, grad_mode=mode, flags=O.FLAG_RANGE_FULL | O.FLAG_ZERO_TAIL)
    cands = [1, 3, 6, 9]
    out = O.probe_align(full["kl"], full["logratio"], full["gsq"], W, R,
                        np.array(cands, np.int32), math.sqrt(2) / 2)
    for j, L in enumerate(cands):
        micro, per_seq = O.literal_cosine(full["grad"], R, L)
        assert out["batch_stats"][j, 0] == pytest.approx(micro, rel=1e-12)
        np.testing.assert_allclose(out["seq_stats"][:, j, 3], per_seq, rtol=1e-12)
        assert out["batch_stats"][j, 1] == pytest.approx(per_seq.mean(), rel=1e-12)
