"""The bounds-checked build flavour (-DADWIN_CHECKED) on the small and odd-shaped parity cases.

A memory checker is not available where these tests run, so the library has a flavour in which
every index the kernels form by hand is tested before the access and a violation raises
ADWIN_DEV_BOUNDS instead of touching memory.  Here the cases with ragged tails, degenerate
windows, padded strides and the overflow fallback run through that flavour: the status word must
stay clear (the helpers raise on any bit) and the results must equal the ordinary build's bit for
bit.
"""
import pytest
import torch

from paper_2605_28396_b200 import api, build, synth
from tests import test_gpu_lmhead as L
from tests import test_gpu_parity as G

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture()
def checked_library():
    path = build.build(checked=True)
    api.use_library(path)
    try:
        yield path
    finally:
        api.use_library(None)


@pytest.mark.parametrize("V", [1, 7, 9, 1001, 4100, 65537])
def test_odd_vocabularies(checked_library, V):
    G.test_odd_vocab_sizes(V)


@pytest.mark.parametrize("path", G.PATHS)
def test_degenerate_windows_padded_strides_and_overflow_fallback(checked_library, path):
    G.test_degenerate_windows(path)
    G.test_padded_row_stride(path)
    G.test_range_full_with_gradient_inside_window_only(path)
    G.test_sampled_token_far_below_the_row_maximum(path, 2, torch.bfloat16)
    G.test_config3_reduced_T_full_vocab(path, api.GRAD_FULL_KL)


def test_teacher_drift_and_return_to_go(checked_library):
    from tests import test_gpu_drift as D
    from tests import test_gpu_rtg as R
    for name in dir(D):
        if name.startswith("test_") and "full_size" not in name:
            fn = getattr(D, name)
            if fn.__code__.co_argcount == 0:
                fn()
    for name in dir(R):
        if name.startswith("test_") and "full_size" not in name:
            fn = getattr(R, name)
            if fn.__code__.co_argcount == 0:
                fn()


def test_fused_lm_head_small_and_ragged(checked_library):
    L.test_small_case_modes_and_flags(api.GRAD_FULL_KL, api.RANGE_FULL)
    L.test_ragged_vocabulary_and_hidden_sizes(1000, 72, 200)
    L.test_all_windows_empty_gives_zero_gradients()


def test_results_equal_the_ordinary_build_bit_for_bit():
    batch = synth.make_batch(3, device=DEV, B=4, T=48)
    lm = synth.make_lmhead_batch(DEV, B=2, T=150, V=1000, d_s=72, d_t=200, w_std=0.15)
    outs = []
    for checked in (False, True):
        api.use_library(build.build(checked=True) if checked else None)
        try:
            grad = torch.zeros(batch.shape, dtype=torch.bfloat16, device=DEV)
            a = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                         batch.rollout_len, grad=grad)
            b = api.adwin_opd_kl_fwd_bwd(batch.student, batch.teacher, batch.tokens, batch.window,
                                         batch.rollout_len, flags=api.RANGE_FULL)
            dW = torch.zeros((1000, 72), dtype=torch.float32, device=DEV)
            c = api.adwin_opd_kl_lmhead_fwd_bwd(lm.hidden_student, lm.w_student, lm.hidden_teacher,
                                                lm.w_teacher, lm.tokens, lm.window, lm.rollout_len,
                                                grad_w=dW)
            torch.cuda.synchronize()
            for o in (a, b, c):
                api.raise_on_dev_status(o.dev_status)
            outs.append((grad, a.kl, a.gsq, b.kl, b.gsq, dW, c.kl, c.gsq))
        finally:
            api.use_library(None)
    for x, y in zip(*outs):
        assert torch.equal(x, y)
